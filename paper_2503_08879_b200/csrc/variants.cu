// Kernels of the comparison paths that sit beside the four steps of the method:
//   - StreamLLM_R (Section 3.1 "Baselines", Appendix A.1): the sink + recent + last rows of a PRE-RoPE key cache,
//     each key rotated by its index inside the kept window while it is copied; values copied verbatim.
//   - the pooled reading of Step 2: the score rows of a KV head's G query heads summed into one row.
//   - a Quest-style comparator (Section 3.1 "Baselines"): per block of 16 tokens the element-wise minimum and
//     maximum of the keys (built once), and per decode step an upper bound of every block's attention logit.
// Both are plain streaming kernels (HBM-bound, no reuse): one warp per 256-byte row, 16-byte accesses.
#include "common.cuh"

namespace sagekv {

// ---- StreamLLM_R ---------------------------------------------------------------------------------------------
// Row r of the reduced cache (r < S: sink token r; otherwise token N - (S + R + 1) + r, i.e. the R recent tokens
// and the last one) gets  y[i] = x[i] cos(a_i) - x[i + 64] sin(a_i),  y[i + 64] = x[i + 64] cos(a_i) + x[i] sin(a_i),
// a_i = r * theta^(-2i/128): dimension i is paired with i + 64, as in the Llama and Qwen models.  Angles, sines
// and cosines are taken in double precision (positions reach thousands of radians at the low dimensions, and the
// kernel moves a few hundred rows), the products in double, one rounding to bf16 at the end.
__global__ void __launch_bounds__(256) compact_window_rope_kernel(const WindowRopeParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int L = p.S + p.R + 1;
  const int64_t n_rows = (int64_t)p.B * p.H_kv * L;
  const double log2_theta = log2((double)p.theta);
  for (int64_t it = (int64_t)blockIdx.x * 8 + warp; it < n_rows; it += (int64_t)gridDim.x * 8) {
    const int r = (int)(it % L);
    const int bk = (int)(it / L), b = bk / p.H_kv, kvh = bk - b * p.H_kv;
    const int64_t tok = r < p.S ? r : (int64_t)p.N - L + r;
    if (!SAGEKV_OK_INDEX(p.status, tok >= 0 && tok < p.N)) continue;
    const int64_t src = (int64_t)b * p.ks.batch_stride + (int64_t)kvh * p.ks.head_stride + tok * p.ks.token_stride;
    const int64_t dst = (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride + (int64_t)r * p.cs.token_stride;
    // lanes 0-15 hold dims 4*lane .. +3 and their partners 64 + 4*lane .. +3 of K; lanes 16-31 copy V (16 bytes each)
    if (lane < 16) {
      const uint2 lo = *reinterpret_cast<const uint2 *>(p.K + src + 4 * lane);
      const uint2 hi = *reinterpret_cast<const uint2 *>(p.K + src + 64 + 4 * lane);
      const uint32_t xl[2] = {lo.x, lo.y}, xh[2] = {hi.x, hi.y};
      uint32_t yl[2], yh[2];
#pragma unroll
      for (int w = 0; w < 2; ++w) {
        float ol[2], oh[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int i = 4 * lane + 2 * w + e;
          const double x1 = (double)__uint_as_float(((xl[w] >> (16 * e)) & 0xffffu) << 16);
          const double x2 = (double)__uint_as_float(((xh[w] >> (16 * e)) & 0xffffu) << 16);
          const double ang = (double)r * exp2(-(double)(2 * i) / (double)kHeadDim * log2_theta);
          double sn, cn;
          sincos(ang, &sn, &cn);
          ol[e] = (float)(x1 * cn - x2 * sn);
          oh[e] = (float)(x2 * cn + x1 * sn);
        }
        yl[w] = pack_bf16x2(ol[0], ol[1]);
        yh[w] = pack_bf16x2(oh[0], oh[1]);
      }
      *reinterpret_cast<uint2 *>(p.Kc + dst + 4 * lane) = make_uint2(yl[0], yl[1]);
      *reinterpret_cast<uint2 *>(p.Kc + dst + 64 + 4 * lane) = make_uint2(yh[0], yh[1]);
    } else {
      const int piece = (lane - 16) * 8;
      st_v4(p.Vc + dst + piece, ld_stream_v4(p.V + src + piece));
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *p.d_step = 0;
}

cudaError_t launch_compact_window_rope(const WindowRopeParams &p, int n_sm, cudaStream_t stream) {
  const int64_t n_rows = (int64_t)p.B * p.H_kv * (p.S + p.R + 1);
  int64_t blocks = (n_rows + 7) / 8;
  if (blocks > 4 * (int64_t)n_sm) blocks = 4 * (int64_t)n_sm;
  if (blocks < 1) blocks = 1;
  compact_window_rope_kernel<<<(unsigned)blocks, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

// ---- pooled scores -------------------------------------------------------------------------------------------
// pooled[b, g, i] = sum over j < G of scores[b, g*G + j, i], added in head order in fp32.
__global__ void __launch_bounds__(256) pool_scores_kernel(const float *scores, int64_t row_stride, float *pooled,
                                                          int64_t pooled_stride, int E, int G, int n_groups) {
  const int n_vec = E >> 2;
  for (int g = blockIdx.y; g < n_groups; g += gridDim.y) {
    const float *src = scores + (int64_t)g * G * row_stride;
    float *dst = pooled + (int64_t)g * pooled_stride;
    for (int v = blockIdx.x * 256 + threadIdx.x; v < n_vec; v += gridDim.x * 256) {
      float4 acc = *reinterpret_cast<const float4 *>(src + 4 * v);
      for (int j = 1; j < G; ++j) {
        const float4 x = *reinterpret_cast<const float4 *>(src + (int64_t)j * row_stride + 4 * v);
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
      }
      *reinterpret_cast<float4 *>(dst + 4 * v) = acc;
    }
    if (blockIdx.x == 0 && (int)threadIdx.x < E - 4 * n_vec) {
      const int i = 4 * n_vec + threadIdx.x;
      float acc = src[i];
      for (int j = 1; j < G; ++j) acc += src[(int64_t)j * row_stride + i];
      dst[i] = acc;
    }
  }
}

cudaError_t launch_pool_scores(const float *scores, int64_t row_stride, float *pooled, int64_t pooled_stride, int E, int G,
                               int n_groups, int n_sm, cudaStream_t stream) {
  if (E <= 0 || n_groups <= 0) return cudaSuccess;
  int bx = (E / 4 + 256 * 4 - 1) / (256 * 4);
  const int want = (4 * n_sm + n_groups - 1) / n_groups;
  if (bx > want) bx = want;
  if (bx < 1) bx = 1;
  pool_scores_kernel<<<dim3((unsigned)bx, (unsigned)(n_groups < 65535 ? n_groups : 65535)), 256, 0, stream>>>(
      scores, row_stride, pooled, pooled_stride, E, G, n_groups);
  return cudaGetLastError();
}

// ---- Quest-style block summaries -----------------------------------------------------------------------------
// One warp per block of 16 tokens of the eviction region: the two half-warps take alternate rows, 16 bytes (8
// dims) per lane, and are merged with one shuffle.  Minima and maxima of bf16 values are bf16 values: exact.
__device__ __forceinline__ void minmax_bf16x8(uint4 v, float (&lo)[8], float (&hi)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float a = __uint_as_float(w[i] << 16), b = __uint_as_float(w[i] & 0xffff0000u);
    lo[2 * i] = fminf(lo[2 * i], a); hi[2 * i] = fmaxf(hi[2 * i], a);
    lo[2 * i + 1] = fminf(lo[2 * i + 1], b); hi[2 * i + 1] = fmaxf(hi[2 * i + 1], b);
  }
}

__global__ void __launch_bounds__(256) quest_build_kernel(const uint16_t *K, sagekv_strides ks, uint16_t *kmin, uint16_t *kmax,
                                                          int S, int E, int n_blocks, int H_kv) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const uint16_t *Kh = K + (int64_t)b * ks.batch_stride + (int64_t)kvh * ks.head_stride + (int64_t)S * ks.token_stride;
  for (int blk = blockIdx.x * 8 + warp; blk < n_blocks; blk += gridDim.x * 8) {
    float lo[8], hi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { lo[i] = INFINITY; hi[i] = -INFINITY; }
    const int t0 = blk * kQuestBlock, t1 = min(E, t0 + kQuestBlock);
#pragma unroll
    for (int u = 0; u < kQuestBlock / 2; ++u) {
      const int t = t0 + 2 * u + (lane >> 4);
      if (t < t1) minmax_bf16x8(ld_stream_v4(Kh + (int64_t)t * ks.token_stride + (lane & 15) * 8), lo, hi);
    }
    uint32_t olo[4], ohi[4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      lo[i] = fminf(lo[i], __shfl_xor_sync(0xffffffffu, lo[i], 16));
      hi[i] = fmaxf(hi[i], __shfl_xor_sync(0xffffffffu, hi[i], 16));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) { olo[i] = pack_bf16x2(lo[2 * i], lo[2 * i + 1]); ohi[i] = pack_bf16x2(hi[2 * i], hi[2 * i + 1]); }
    const int64_t o = (((int64_t)b * H_kv + kvh) * n_blocks + blk) * kHeadDim + (lane & 15) * 8;
    if (lane < 16) st_v4(kmin + o, make_uint4(olo[0], olo[1], olo[2], olo[3]));
    else st_v4(kmax + o, make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]));
  }
}

cudaError_t launch_quest_build(const uint16_t *K, sagekv_strides ks, uint16_t *kmin, uint16_t *kmax, int S, int E, int H_kv,
                               int B, int n_sm, cudaStream_t stream) {
  const int n_blocks = (E + kQuestBlock - 1) / kQuestBlock;
  if (n_blocks <= 0) return cudaSuccess;
  int gx = (n_blocks + 7) / 8;
  const int want = (8 * n_sm + H_kv * B - 1) / (H_kv * B);
  if (gx > want) gx = want;
  quest_build_kernel<<<dim3((unsigned)gx, (unsigned)H_kv, (unsigned)B), 256, 0, stream>>>(K, ks, kmin, kmax, S, E, n_blocks, H_kv);
  return cudaGetLastError();
}

// u[b, h, blk] = scale * sum_c max(q[b,h,c] * kmin[b, h/G, blk, c], q[b,h,c] * kmax[...]), fp32.  A half-warp per block: lane l of
// it holds dims 8l .. 8l+7 of both summaries and adds its eight terms for each of the G heads, four shuffles sum the
// sixteen lanes.  The queries of the KV head sit in shared memory as fp32.
__global__ void __launch_bounds__(256) quest_bounds_kernel(const uint16_t *q, const uint16_t *kmin, const uint16_t *kmax, float *u,
                                                           int64_t u_stride, int n_blocks, int G, int H_q, int H_kv, float scale) {
  __shared__ float qs[kMaxGroup][kHeadDim];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, l16 = lane & 15;
  const int kvh = blockIdx.y, b = blockIdx.z;
  for (int i = threadIdx.x; i < G * kHeadDim; i += 256)
    qs[i >> 7][i & 127] = __uint_as_float((uint32_t)q[((int64_t)b * H_q + kvh * G) * kHeadDim + i] << 16);
  __syncthreads();
  const int64_t base = ((int64_t)b * H_kv + kvh) * n_blocks;
  for (int blk0 = (blockIdx.x * 8 + warp) * 2; blk0 < n_blocks; blk0 += gridDim.x * 16) {
    const int blk = blk0 + (lane >> 4);
    const bool have = blk < n_blocks;
    const int64_t o = (base + (have ? blk : blk0)) * kHeadDim + l16 * 8;
    const uint4 a = ld_stream_v4(kmin + o), c = ld_stream_v4(kmax + o);
    const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wc[4] = {c.x, c.y, c.z, c.w};
    float mn[8], mx[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mn[2 * i] = __uint_as_float(wa[i] << 16); mn[2 * i + 1] = __uint_as_float(wa[i] & 0xffff0000u);
      mx[2 * i] = __uint_as_float(wc[i] << 16); mx[2 * i + 1] = __uint_as_float(wc[i] & 0xffff0000u);
    }
    for (int h = 0; h < G; ++h) {
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float qv = qs[h][l16 * 8 + i];
        acc += fmaxf(qv * mn[i], qv * mx[i]);
      }
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
      if (l16 == 0 && have) u[((int64_t)b * H_q + kvh * G + h) * u_stride + blk] = acc * scale;
    }
  }
}

cudaError_t launch_quest_bounds(const uint16_t *q, const uint16_t *kmin, const uint16_t *kmax, float *u, int64_t u_stride,
                                int n_blocks, int G, int H_q, int H_kv, int B, float scale, int n_sm, cudaStream_t stream) {
  if (n_blocks <= 0) return cudaSuccess;
  int gx = (n_blocks + 15) / 16;
  const int want = (8 * n_sm + H_kv * B - 1) / (H_kv * B);
  if (gx > want) gx = want;
  quest_bounds_kernel<<<dim3((unsigned)gx, (unsigned)H_kv, (unsigned)B), 256, 0, stream>>>(q, kmin, kmax, u, u_stride, n_blocks, G,
                                                                                         H_q, H_kv, scale);
  return cudaGetLastError();
}

}  // namespace sagekv
