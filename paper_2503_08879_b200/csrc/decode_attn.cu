// Step 4: append the new token to the recent window, then attention of every query head over its view
// of the reduced cache (sink + its own selected segment + window).
//
// Flash-decoding layout: the L rows of a KV head are cut into n_splits partitions; one CTA per
// (partition, KV head, batch entry) streams its K and V rows once, straight from global memory into
// tensor-core fragments, and keeps a running softmax.  Per 16-row tile of a warp
//   S^T = Q K^T   heads (padded to 16) x 8 rows per mma; lane (g, c) loads 16-byte pieces of rows g and
//                 g+8 and the query fragment uses the same column permutation, so no shuffle or shared
//                 memory is needed to form the fragments;
//   O^T += V^T P  head_dim x heads; the lane that owns logits of rows {2c, 2c+1, 2c+8, 2c+9} for head g
//                 (the accumulator layout of the first product) is exactly the lane that must supply
//                 those rows' weights for head g as the B fragment, and it loads the same four V rows
//                 at 16 columns of its own, pairing two rows per register with a byte permute.
// Every head masks the rows of the other heads' segments.  The partition results (max, sum, O) go to
// scratch; the CTA that arrives last for a KV head (one atomic ticket, no waiting) merges them by
// log-sum-exp and writes bf16 output.  The new token's row is taken from k_new / v_new by whichever
// lane would have read the window slot it replaces, and the CTA owning that slot stores it.
#include "common.cuh"

namespace sagekv {

constexpr int kDecodeThreads = kDecodeWarps * 32;

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

__device__ __forceinline__ uint32_t reg_of(const uint4 &v, int i) {
  return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

__global__ void __launch_bounds__(kDecodeThreads) decode_attn_kernel(const DecodeParams p) {
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  const bool append = p.k_new != nullptr;

  int step = 0, slot = -1;
  if (append) {
    step = *reinterpret_cast<const volatile int32_t *>(p.d_step);
    slot = p.S + p.n_sel + step % p.ring_len;
  }

  const uint16_t *Kh = p.Kc + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride;
  const uint16_t *Vh = p.Vc + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride;
  const uint16_t *kn = append ? p.k_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  const uint16_t *vn = append ? p.v_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;

  // A fragments of Q: head g in row g of the tile, rows 8..15 are padding
  uint4 qf[4];
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) qf[jj] = make_uint4(0u, 0u, 0u, 0u);
  if (g < p.G) {
    const uint16_t *qrow = p.q + ((int64_t)b * p.H_q + kvh * p.G + g) * kHeadDim;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) qf[jj] = *reinterpret_cast<const uint4 *>(qrow + jj * 32 + c * 8);
  }
  // rows head g may look at: sink, its own segment, the window
  const int seg_lo = p.S + g * p.k_q, seg_hi = seg_lo + p.k_q, win_lo = p.S + p.n_sel;

  float m_run = -INFINITY;   // running max of head g (log2 units), equal in the 4 lanes of a group
  float l_run = 0.f;         // this lane's share of the running sum of head g
  float acc[8][4];           // O^T: [m-tile][(d_a,h 2c), (d_a,h 2c+1), (d_b,h 2c), (d_b,h 2c+1)]
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;

  const int split_lo = split * p.iters * kDecodeTile;
  for (int it = 0; it < p.iters; ++it) {
    const int base = split_lo + it * kDecodeTile + warp * 16;
    if (base >= p.L) break;    // warp-uniform
    // ---- loads: K rows g, g+8 (4 pieces each); V rows 2c, 2c+1, 2c+8, 2c+9 (2 pieces each) ----
    uint4 ka[4], kb[4], vv[4][2];
    {
      const int r0 = min(base + g, p.L - 1), r1 = min(base + g + 8, p.L - 1);
      const uint16_t *pa = (r0 == slot ? kn : Kh + (int64_t)r0 * p.cs.token_stride) + c * 8;
      const uint16_t *pb = (r1 == slot ? kn : Kh + (int64_t)r1 * p.cs.token_stride) + c * 8;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        ka[jj] = ld_v4(pa + jj * 32);
        kb[jj] = ld_v4(pb + jj * 32);
      }
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int r = min(base + 2 * c + (s & 1) + (s >> 1) * 8, p.L - 1);
        const uint16_t *pv = (r == slot ? vn : Vh + (int64_t)r * p.cs.token_stride) + g * 8;
        vv[s][0] = ld_v4(pv);
        vv[s][1] = ld_v4(pv + 64);
      }
    }
    // ---- S^T = Q K^T for rows base..base+7 (s0,s1) and base+8..base+15 (s2,s3) ----
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      mma_bf16_16816(s0, s1, z0, z1, qf[jj].x, 0u, qf[jj].y, 0u, ka[jj].x, ka[jj].y);
      mma_bf16_16816(s0, s1, z0, z1, qf[jj].z, 0u, qf[jj].w, 0u, ka[jj].z, ka[jj].w);
      mma_bf16_16816(s2, s3, z2, z3, qf[jj].x, 0u, qf[jj].y, 0u, kb[jj].x, kb[jj].y);
      mma_bf16_16816(s2, s3, z2, z3, qf[jj].z, 0u, qf[jj].w, 0u, kb[jj].z, kb[jj].w);
    }
    float sv[4] = {s0 * p.scale_log2, s1 * p.scale_log2, s2 * p.scale_log2, s3 * p.scale_log2};
    float tile_max = -INFINITY;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int r = base + 2 * c + (s & 1) + (s >> 1) * 8;
      const bool vis = g < p.G && r < p.L && (r < p.S || r >= win_lo || (r >= seg_lo && r < seg_hi));
      sv[s] = vis ? sv[s] : -INFINITY;
      tile_max = fmaxf(tile_max, sv[s]);
    }
    tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 1));
    tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 2));
    const float m_new = fmaxf(m_run, tile_max);
    const float m_safe = m_new == -INFINITY ? 0.f : m_new;
    const float alpha = fast_exp2(m_run - m_safe);      // 0 while nothing has been seen
    float pw[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) pw[s] = fast_exp2(sv[s] - m_safe);
    // the weights enter the second product as bf16; sum the rounded values so numerator and denominator agree
    const uint32_t pb0 = pack_bf16x2(pw[0], pw[1]), pb1 = pack_bf16x2(pw[2], pw[3]);
    l_run = l_run * alpha + (__uint_as_float(pb0 << 16) + __uint_as_float(pb0 & 0xffff0000u)) +
            (__uint_as_float(pb1 << 16) + __uint_as_float(pb1 & 0xffff0000u));
    m_run = m_new;
    // rescale factors of heads 2c and 2c+1 live in the lanes of groups 2c and 2c+1
    const float al0 = __shfl_sync(0xffffffffu, alpha, (2 * c) * 4);
    const float al1 = __shfl_sync(0xffffffffu, alpha, (2 * c + 1) * 4);
    // ---- O^T += V^T P ----
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const int piece = mt >> 2, reg = mt & 3;           // columns 8g + 2*reg (+1) of piece 0, 64 + ... of piece 1
      const uint32_t v0 = reg_of(vv[0][piece], reg), v1 = reg_of(vv[1][piece], reg);
      const uint32_t v2 = reg_of(vv[2][piece], reg), v3 = reg_of(vv[3][piece], reg);
      acc[mt][0] *= al0; acc[mt][1] *= al1; acc[mt][2] *= al0; acc[mt][3] *= al1;
      mma_bf16_16816(acc[mt][0], acc[mt][1], acc[mt][2], acc[mt][3], prmt(v0, v1, 0x5410u), prmt(v0, v1, 0x7632u),
                     prmt(v2, v3, 0x5410u), prmt(v2, v3, 0x7632u), pb0, pb1);
    }
  }

  // ---- merge the warps of the CTA ----
  __shared__ float sm_m[kDecodeWarps][kMaxGroup], sm_l[kDecodeWarps][kMaxGroup];
  __shared__ float sm_o[kDecodeWarps][kMaxGroup][kHeadDim];
  __shared__ float sm_w[kMaxGroup * 64];   // merge weights of the last-arriving CTA
  __shared__ int sm_last;
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (c == 0) { sm_m[warp][g] = m_run; sm_l[warp][g] = l_run; }
  __syncthreads();
  {
    const int h0 = 2 * c, h1 = 2 * c + 1;
    float M0 = -INFINITY, M1 = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) { M0 = fmaxf(M0, sm_m[w][h0]); M1 = fmaxf(M1, sm_m[w][h1]); }
    const float f0 = M0 == -INFINITY ? 0.f : fast_exp2(sm_m[warp][h0] - M0);
    const float f1 = M1 == -INFINITY ? 0.f : fast_exp2(sm_m[warp][h1] - M1);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const int d_a = (mt >> 2) * 64 + g * 8 + (mt & 3) * 2;
      sm_o[warp][h0][d_a] = acc[mt][0] * f0;
      sm_o[warp][h1][d_a] = acc[mt][1] * f1;
      sm_o[warp][h0][d_a + 1] = acc[mt][2] * f0;
      sm_o[warp][h1][d_a + 1] = acc[mt][3] * f1;
    }
  }
  __syncthreads();
  // thread d owns column d of every head from here on
  const int d = tid;
  float o_cta[kMaxGroup], m_cta[kMaxGroup], l_cta[kMaxGroup];
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][h]);
    float l = 0.f, o = 0.f;
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) {
      l += M == -INFINITY ? 0.f : sm_l[w][h] * fast_exp2(sm_m[w][h] - M);
      o += sm_o[w][h][d];
    }
    m_cta[h] = M; l_cta[h] = l; o_cta[h] = o;
  }

  // the CTA that owns the replaced window slot stores the new token's row
  if (append && slot >= split_lo && slot < split_lo + p.iters * kDecodeTile && tid < 32) {
    const uint16_t *src = (lane < 16 ? kn : vn) + (lane & 15) * 8;
    uint16_t *dst = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                    (int64_t)slot * p.cs.token_stride + (lane & 15) * 8;
    st_v4(dst, ld_v4(src));
  }

  const int bk = b * p.H_kv + kvh;
  if (p.n_splits > 1) {
    float *part = p.partials + ((int64_t)bk * p.n_splits + split) * kPartialStride;
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h)
      if (h < p.G) part[h * kHeadDim + d] = o_cta[h];
    if (d < p.G) {
      part[kMaxGroup * kHeadDim + d] = m_cta[d];
      part[kMaxGroup * kHeadDim + kMaxGroup + d] = l_cta[d];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sm_last = atomicAdd(&p.tickets[bk], 1) == p.n_splits - 1;
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    // ---- last arrival for this KV head: log-sum-exp merge of all partitions ----
    const float *all = p.partials + (int64_t)bk * p.n_splits * kPartialStride;
    for (int h = 0; h < p.G; ++h) {
      float M = -INFINITY;
      for (int i = 0; i < p.n_splits; ++i) M = fmaxf(M, __ldcg(all + (int64_t)i * kPartialStride + kMaxGroup * kHeadDim + h));
      __syncthreads();                                   // sm_w of the previous head has been consumed
      float lsum = 0.f;
      for (int i0 = 0; i0 < p.n_splits; i0 += 64) {
        const int n = min(64, p.n_splits - i0);
        if (tid < n) {
          const float mi = __ldcg(all + (int64_t)(i0 + tid) * kPartialStride + kMaxGroup * kHeadDim + h);
          sm_w[tid] = (M == -INFINITY) ? 0.f : fast_exp2(mi - M);
        }
        __syncthreads();
        float o = 0.f;
        for (int i = 0; i < n; ++i) {
          const float *pi = all + (int64_t)(i0 + i) * kPartialStride;
          o += __ldcg(pi + h * kHeadDim + d) * sm_w[i];
          lsum += __ldcg(pi + kMaxGroup * kHeadDim + kMaxGroup + h) * sm_w[i];
        }
        o_cta[0] = i0 == 0 ? o : o_cta[0] + o;
        __syncthreads();
      }
      const float outv = lsum > 0.f ? o_cta[0] / lsum : 0.f;
      p.out[((int64_t)b * p.H_q + kvh * p.G + h) * kHeadDim + d] = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
      if (p.lse != nullptr && d == 0)
        p.lse[(int64_t)b * p.H_q + kvh * p.G + h] = lsum > 0.f ? (M + log2f(lsum)) * kLn2 : -INFINITY;
    }
    if (tid == 0) p.tickets[bk] = 0;
  } else {
    for (int h = 0; h < p.G; ++h) {
      const float outv = l_cta[h] > 0.f ? o_cta[h] / l_cta[h] : 0.f;
      p.out[((int64_t)b * p.H_q + kvh * p.G + h) * kHeadDim + d] = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
      if (p.lse != nullptr && d == 0)
        p.lse[(int64_t)b * p.H_q + kvh * p.G + h] = l_cta[h] > 0.f ? (m_cta[h] + log2f(l_cta[h])) * kLn2 : -INFINITY;
    }
  }
  // ---- the last KV head to finish advances the step counter ----
  if (tid == 0) {
    const int n_heads = p.B * p.H_kv;
    __threadfence();
    if (atomicAdd(&p.tickets[n_heads], 1) == n_heads - 1) {
      p.tickets[n_heads] = 0;
      if (append) *p.d_step = step + 1;
    }
  }
}

cudaError_t launch_decode(const DecodeParams &p, cudaStream_t stream) {
  dim3 grid(p.n_splits, p.H_kv, p.B);
  decode_attn_kernel<<<grid, kDecodeThreads, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace sagekv
