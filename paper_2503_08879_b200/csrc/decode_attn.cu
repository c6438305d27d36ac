// Step 4: append the new token to the recent window, then attention of every query head over its view
// of the reduced cache (sink + its own selected segment + window).
//
// Flash-decoding on thread-block clusters.  The L rows of one KV head are cut into 16-row tiles that are
// dealt evenly to the CTAs of one cluster.  Every warp owns two staging slots: it issues 16-byte cp.async
// copies for the K and V rows of its first two tiles at once (in flight together, no registers held),
// works on both tiles, and, when the partition is longer than the staging area, refills its own two
// slots for the next pass (no block-wide synchronisation: the slots belong to the warp).  Only beyond
// four passes does a head get more than one cluster.  Per pair of tiles:
//   S^T = Q K^T   heads (padded to 16) x 8 rows per mma.  Lane (g, c) reads 16-byte pieces of rows g and
//                 g+8; the query fragment uses the same column permutation, so fragments come straight
//                 from the staged rows with no transposition.
//   O^T += V^T P  head_dim x heads.  The accumulator layout of the first product puts the weights of rows
//                 {2c, 2c+1, 2c+8, 2c+9} for head g in lane (g, c), which is exactly the B fragment of the
//                 second; the lane reads the same four V rows at 16 columns of its own and pairs two rows
//                 per register with a byte permute.
// The staged rows are XOR-swizzled so that both access patterns are free of bank conflicts.  Every head
// masks the rows of the other heads' segments.  Warps are merged through shared memory, the CTAs of a
// cluster through distributed shared memory (each CTA finishes a slice of the 128 columns), so with one
// cluster per head nothing touches global scratch.  With several clusters per head the cluster results
// go to scratch and the CTA that arrives last (one atomic ticket, no waiting) merges them.
// The staged copy of the window row that the new token replaces is overwritten in shared memory from
// k_new / v_new once it has landed, and the CTA owning that row stores the new token into the cache.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace sagekv {

constexpr int kTileBytes = 16 * 256;           // 16 rows of K (or V)
constexpr int kResFloats = kMaxGroup * kHeadDim + 2 * kMaxGroup;

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

__device__ __forceinline__ uint32_t reg_of(const uint4 &v, int i) {
  return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// 16-byte piece `piece` of row `row` of a staged tile lives at piece ^ swz(row): rows g and g+1 land in
// different halves of the 128-byte bank window (K fragment reads), rows 2c apart in different quarters
// (V fragment reads).
__device__ __forceinline__ int swz(int row) { return ((row & 1) << 2) ^ (((row >> 1) & 3) << 1); }

__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// kPasses: the CTA's partition is longer than its staging area (false keeps the common case free of the pass loop)
template <bool kPasses>
__global__ void __launch_bounds__(kDecodeMaxWarps * 32) decode_attn_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char stage[];          // tiles: [K 4 KB | V 4 KB] each
  __shared__ __align__(16) float inbox_o[kMaxGroup * (kHeadDim + 16)];   // [source CTA][head][my columns], pushed by the peers; cluster size x columns <= 144
  __shared__ float2 inbox_ml[kDecodeMaxCluster * kMaxGroup];        // [source CTA][head] (max, sum)
  __shared__ float sm_m[kDecodeMaxWarps][kMaxGroup], sm_l[kDecodeMaxWarps][kMaxGroup];
  __shared__ int sm_last;

  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int ci = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;      // ci: CTA index within the head
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_warps = blockDim.x >> 5;
  const int g = lane >> 2, c = lane & 3;
  const bool append = p.k_new != nullptr;
  cluster.barrier_arrive();                              // waited for just before the first push into a peer

  // Programmatic dependent launch: until the wait returns, nothing that an earlier kernel on the stream may
  // still be writing is read (q, k_new, v_new, the step counter) and nothing at all is written.  In
  // prefetch mode the rows of the reduced cache are requested first: the caller has promised that the
  // kernel directly before this one does not write this layer's cache.  The successor is released only
  // after the wait, so at most one kernel runs ahead of its dependency.
  if (p.pdl_mode < 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  const uint16_t *Kh = p.Kc + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride;
  const uint16_t *Vh = p.Vc + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride;

  // tiles of this CTA: an even deal of the head's n_tiles over the gridDim.x CTAs
  const int n_tiles = (p.L + 15) >> 4;
  const int base_n = n_tiles / (int)gridDim.x, rem = n_tiles % (int)gridDim.x;
  const int first_tile = ci * base_n + min(ci, rem);
  const int my_tiles = base_n + (ci < rem ? 1 : 0);
  const int n_mine = warp < my_tiles ? (my_tiles - warp + n_warps - 1) / n_warps : 0;   // tiles of this warp

  // ---- issue the copies of this warp's first two tiles (its later tiles reuse the same two slots) ----
  const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(stage);
  auto issue_half = [&](int i, const uint16_t *src, uint32_t half) {   // K (half 0) or V (half 1) of this warp's i-th tile -> slot i & 1
    const int row0 = (first_tile + warp + i * n_warps) << 4;
    const uint32_t dst = stage_base + (warp + (i & 1) * n_warps) * 2 * kTileBytes + half * kTileBytes;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int flat = u * 32 + lane, row = flat >> 4, piece = flat & 15;
      const int r = min(row0 + row, p.L - 1);
      cp_async16(dst + row * 256 + ((piece ^ swz(row)) << 4), src + (int64_t)r * p.cs.token_stride + piece * 8);
    }
  };
  for (int i = 0; i < min(n_mine, 2); ++i) {
    issue_half(i, Kh, 0u);
    issue_half(i, Vh, 1u);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");

  if (p.pdl_mode >= 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  int step = 0, slot = -1;
  if (append) {
    step = *reinterpret_cast<const volatile int32_t *>(p.d_step);
    slot = p.S + p.n_sel + step % p.ring_len;
  }
  const uint16_t *kn = append ? p.k_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  const uint16_t *vn = append ? p.v_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;

  // the CTA that owns the replaced window slot stores the new token's row
  if (append && warp == 0) {
    const int st = slot >> 4;
    if (st >= first_tile && st < first_tile + my_tiles) {
      const uint16_t *src = (lane < 16 ? kn : vn) + (lane & 15) * 8;
      uint16_t *dst = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                      (int64_t)slot * p.cs.token_stride + (lane & 15) * 8;
      st_v4(dst, ld_v4(src));
    }
  }

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
  float acc[8][4];           // O^T: [m-tile][(d_a,h 2c), (d_a,h 2c+1), (d_a+1,h 2c), (d_a+1,h 2c+1)]
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;

  // A warp works on two tiles at once (twice as many independent mma chains, one softmax update) and,
  // when the partition is longer than the staging area, goes through its tiles in passes of two.
  for (int i0 = 0; i0 < (kPasses ? n_mine : min(n_mine, 2)); i0 += 2) {
    const int nt = min(2, n_mine - i0);                    // tiles of this pass
    // Later passes refill the warp's own two slots, K and V as separate copy groups: K as soon as the pass before
    // has taken its first product, V after its second.  Here the K rows are needed; the V group, committed
    // after them, may still be on its way.
    const bool more = kPasses && i0 + 2 < n_mine;          // a pass follows this one
    if (kPasses && i0 > 0) {
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncwarp();
    uint32_t tk[2], tv[2];
    int base[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      base[t] = (first_tile + warp + (i0 + (t < nt ? t : 0)) * n_warps) << 4;
      tk[t] = stage_base + (warp + (t < nt ? t : 0) * n_warps) * 2 * kTileBytes;
      tv[t] = tk[t] + kTileBytes;
      if (t < nt && slot >= base[t] && slot < base[t] + 16 && lane < 16) {   // the staged copy of the replaced row is stale: patch it (K here, V below)
        const int row = slot - base[t], piece = lane & 15;
        const uint4 nv = ld_v4(kn + piece * 8);
        const uint32_t dst = tk[t] + row * 256 + ((piece ^ swz(row)) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(nv.x), "r"(nv.y), "r"(nv.z), "r"(nv.w) : "memory");
      }
    }
    __syncwarp();
    // ---- S^T = Q K^T: per tile, rows base..base+7 -> sv[t][0..1], rows base+8..base+15 -> sv[t][2..3] ----
    float sv[2][4];
    {
      float z[2][4];
#pragma unroll
      for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) { sv[t][e] = 0.f; z[t][e] = 0.f; }
      const int sa = swz(g), sb = swz(g + 8);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (t < nt) {
            const uint4 ka = lds_v4(tk[t] + g * 256 + (((c + 4 * jj) ^ sa) << 4));
            const uint4 kb = lds_v4(tk[t] + (g + 8) * 256 + (((c + 4 * jj) ^ sb) << 4));
            mma_bf16_16816(sv[t][0], sv[t][1], z[t][0], z[t][1], qf[jj].x, 0u, qf[jj].y, 0u, ka.x, ka.y);
            mma_bf16_16816(sv[t][2], sv[t][3], z[t][2], z[t][3], qf[jj].x, 0u, qf[jj].y, 0u, kb.x, kb.y);
            mma_bf16_16816(sv[t][0], sv[t][1], z[t][0], z[t][1], qf[jj].z, 0u, qf[jj].w, 0u, ka.z, ka.w);
            mma_bf16_16816(sv[t][2], sv[t][3], z[t][2], z[t][3], qf[jj].z, 0u, qf[jj].w, 0u, kb.z, kb.w);
          }
        }
      }
    }
    if (more) {                                            // the K rows are in registers' past: refill them for the next pass
      __syncwarp();
      for (int i = i0 + 2; i < min(n_mine, i0 + 4); ++i) issue_half(i, Kh, 0u);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    float tile_max = -INFINITY;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int r = base[t] + 2 * c + (s & 1) + (s >> 1) * 8;
        const bool vis = t < nt && g < p.G && r < p.L && (r < p.S || r >= win_lo || (r >= seg_lo && r < seg_hi));
        sv[t][s] = vis ? sv[t][s] * p.scale_log2 : -INFINITY;
        tile_max = fmaxf(tile_max, sv[t][s]);
      }
    }
    tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 1));
    tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, 2));
    const float m_new = fmaxf(m_run, tile_max);
    const float m_safe = m_new == -INFINITY ? 0.f : m_new;
    if (kPasses && i0 > 0) {                              // a later pass: bring sum and accumulators to the new maximum
      const float alpha = fast_exp2(m_run - m_safe);
      l_run *= alpha;
      // the factors of heads 2c and 2c+1 live in the lanes of groups 2c and 2c+1
      const float al0 = __shfl_sync(0xffffffffu, alpha, (2 * c) * 4), al1 = __shfl_sync(0xffffffffu, alpha, (2 * c + 1) * 4);
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) { acc[mt][0] *= al0; acc[mt][1] *= al1; acc[mt][2] *= al0; acc[mt][3] *= al1; }
    }
    m_run = m_new;
    // the weights enter the second product as bf16; sum the rounded values so numerator and denominator agree
    uint32_t pb[2][2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      pb[t][0] = pack_bf16x2(fast_exp2(sv[t][0] - m_safe), fast_exp2(sv[t][1] - m_safe));
      pb[t][1] = pack_bf16x2(fast_exp2(sv[t][2] - m_safe), fast_exp2(sv[t][3] - m_safe));
      l_run += (__uint_as_float(pb[t][0] << 16) + __uint_as_float(pb[t][0] & 0xffff0000u)) +
               (__uint_as_float(pb[t][1] << 16) + __uint_as_float(pb[t][1] & 0xffff0000u));
    }
    // ---- O^T += V^T P: rows 2c, 2c+1, 2c+8, 2c+9 at columns 8g..8g+7 and 64+8g..64+8g+7 ----
    if (kPasses && i0 > 0) {                               // this pass's V group; the next pass's K group may stay pending
      if (more) {
        asm volatile("cp.async.wait_group 1;" ::: "memory");
      } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
    }
    __syncwarp();
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      if (t < nt && slot >= base[t] && slot < base[t] + 16 && lane >= 16) {
        const int row = slot - base[t], piece = lane & 15;
        const uint4 nv = ld_v4(vn + piece * 8);
        const uint32_t dst = tv[t] + row * 256 + ((piece ^ swz(row)) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(nv.x), "r"(nv.y), "r"(nv.z), "r"(nv.w) : "memory");
      }
    }
    __syncwarp();
    int vs[4];
    uint32_t voff[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int row = 2 * c + (s & 1) + (s >> 1) * 8;
      voff[s] = row * 256;
      vs[s] = swz(row);
    }
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        if (t < nt) {
          uint4 vv[4];
#pragma unroll
          for (int s = 0; s < 4; ++s) vv[s] = lds_v4(tv[t] + voff[s] + (((g + 8 * piece) ^ vs[s]) << 4));
#pragma unroll
          for (int reg = 0; reg < 4; ++reg) {
            const int mt = piece * 4 + reg;              // columns piece*64 + 8g + 2*reg (+1)
            const uint32_t v0 = reg_of(vv[0], reg), v1 = reg_of(vv[1], reg);
            const uint32_t v2 = reg_of(vv[2], reg), v3 = reg_of(vv[3], reg);
            mma_bf16_16816(acc[mt][0], acc[mt][1], acc[mt][2], acc[mt][3], prmt(v0, v1, 0x5410u),
                           prmt(v0, v1, 0x7632u), prmt(v2, v3, 0x5410u), prmt(v2, v3, 0x7632u), pb[t][0], pb[t][1]);
          }
        }
      }
    }
    if (more) {
      __syncwarp();
      for (int i = i0 + 2; i < min(n_mine, i0 + 4); ++i) issue_half(i, Vh, 1u);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }

  // ---- merge the warps of the CTA (the staging area is reused for the exchange) ----
  // Exchange order of the 8 x 128 values: idx = ((piece*8 + e)*8 + g)*8 + h for column piece*64 + g*8 + e,
  // so that the float2 stores of a half-warp (g 0..3, heads 2c, 2c+1) fall into 32 different banks.
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (c == 0) { sm_m[warp][g] = m_run; sm_l[warp][g] = l_run; }
  __syncthreads();                                       // also: every warp is done reading its tiles
  const int n_act = min(n_warps, my_tiles);              // warps that had a tile
  float *xo = reinterpret_cast<float *>(stage);          // [n_act][1024]
  if (warp < n_act) {
    const int h0 = 2 * c, h1 = 2 * c + 1;
    float M0 = -INFINITY, M1 = -INFINITY;
    for (int w = 0; w < n_act; ++w) { M0 = fmaxf(M0, sm_m[w][h0]); M1 = fmaxf(M1, sm_m[w][h1]); }
    const float f0 = M0 == -INFINITY ? 0.f : fast_exp2(sm_m[warp][h0] - M0);
    const float f1 = M1 == -INFINITY ? 0.f : fast_exp2(sm_m[warp][h1] - M1);
    float *mine = xo + warp * (kMaxGroup * kHeadDim) + g * 8 + h0;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const int pe = (mt >> 2) * 8 + (mt & 3) * 2;       // piece*8 + e of column d_a; d_a + 1 is the next e
      *reinterpret_cast<float2 *>(mine + pe * 64) = make_float2(acc[mt][0] * f0, acc[mt][1] * f1);
      *reinterpret_cast<float2 *>(mine + (pe + 1) * 64) = make_float2(acc[mt][2] * f0, acc[mt][3] * f1);
    }
  }
  __syncthreads();
  cluster.barrier_wait();                                // pairs with the arrive at kernel entry: every peer runs

  // ---- push this CTA's result to the peers: the owner of a column slice receives it from every CTA.
  // One thread sums four neighbouring columns of one head over the warps and sends them as one 16-byte store.
  const int cols = ((kHeadDim + cs - 1) / cs + 3) & ~3;  // columns each CTA of the cluster finishes: a multiple of 4, the last CTA may get fewer
  // A warp's 32 items are 8 column groups (g) x 4 heads at one (piece, e): their exchange addresses g*8 + h
  // fall into 32 different banks.
  for (int item = tid; item < 8 * 32; item += blockDim.x) {
    const int g8 = item & 7, h = ((item >> 3) & 3) + ((item >> 5) & 1) * 4, pg = item >> 6;   // pg = piece*2 + e0/4
    if (h < p.G) {
      const int col0 = (pg >> 1) * 64 + g8 * 8 + (pg & 1) * 4;
      const float *src = xo + (((pg >> 1) * 8 + (pg & 1) * 4) * 8 + g8) * 8 + h;             // column col0 + e: + 64*e
      float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int w = 0; w < n_act; ++w) {
        const float *sw = src + w * kMaxGroup * kHeadDim;
        o.x += sw[0]; o.y += sw[64]; o.z += sw[128]; o.w += sw[192];
      }
      const int owner = col0 / cols;
      *reinterpret_cast<float4 *>(cluster.map_shared_rank(inbox_o, owner) + (rank * kMaxGroup + h) * cols +
                                  (col0 - owner * cols)) = o;
    }
  }
  for (int h = warp; h < p.G; h += n_warps) {            // one warp per head, one lane per contributing warp
    const float mw = lane < n_act ? sm_m[lane][h] : -INFINITY;
    float M = mw;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    float l = (lane < n_act && M != -INFINITY) ? sm_l[lane][h] * fast_exp2(mw - M) : 0.f;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if (lane < cs) cluster.map_shared_rank(inbox_ml, lane)[rank * kMaxGroup + h] = make_float2(M, l);
  }
  cluster.sync();   // all pushes have landed; no shared memory of a peer is touched after this point

  // ---- finish columns [rank*cols, (rank+1)*cols) of every head from the inbox ----
  const int bk = b * p.H_kv + kvh;
  const int n_clusters = (int)gridDim.x / cs, cl = ci / cs;
  float *part = p.partials + ((int64_t)bk * n_clusters + cl) * kResFloats;
  for (int item = tid; item < p.G * cols; item += blockDim.x) {
    const int h = item / cols, lc = item - h * cols, col = rank * cols + lc;
    if (col >= kHeadDim) continue;
    float M = -INFINITY;
    for (int r = 0; r < cs; ++r) M = fmaxf(M, inbox_ml[r * kMaxGroup + h].x);
    float o = 0.f, l = 0.f;
    for (int r = 0; r < cs; ++r) {
      const float2 ml = inbox_ml[r * kMaxGroup + h];
      const float wgt = M == -INFINITY ? 0.f : fast_exp2(ml.x - M);
      o += inbox_o[(r * kMaxGroup + h) * cols + lc] * wgt;
      l += ml.y * wgt;
    }
    if (n_clusters == 1) {
      const float outv = l > 0.f ? o / l : 0.f;
      p.out[((int64_t)b * p.H_q + kvh * p.G + h) * kHeadDim + col] = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
      if (p.lse != nullptr && col == 0)
        p.lse[(int64_t)b * p.H_q + kvh * p.G + h] = l > 0.f ? (M + log2f(l)) * kLn2 : -INFINITY;
    } else {
      part[h * kHeadDim + col] = o;
      if (col == 0) {
        part[kMaxGroup * kHeadDim + h] = M;
        part[kMaxGroup * kHeadDim + kMaxGroup + h] = l;
      }
    }
  }

  bool head_done = rank == 0;                            // one CTA per head reports completion
  if (n_clusters > 1) {
    // ---- several clusters per head: the last CTA to arrive merges the cluster results ----
    __threadfence();
    __syncthreads();
    if (tid == 0) sm_last = atomicAdd(&p.tickets[bk], 1) == (int)gridDim.x - 1;
    __syncthreads();
    head_done = sm_last != 0;
    if (head_done) {
      __threadfence();
      const float *all = p.partials + (int64_t)bk * n_clusters * kResFloats;
      for (int item = tid; item < p.G * kHeadDim; item += blockDim.x) {
        const int h = item >> 7, col = item & 127;
        float M = -INFINITY;
        for (int i = 0; i < n_clusters; ++i) M = fmaxf(M, __ldcg(all + i * kResFloats + kMaxGroup * kHeadDim + h));
        float o = 0.f, l = 0.f;
        for (int i = 0; i < n_clusters; ++i) {
          const float *pi = all + i * kResFloats;
          const float wgt = M == -INFINITY ? 0.f : fast_exp2(__ldcg(pi + kMaxGroup * kHeadDim + h) - M);
          o += __ldcg(pi + h * kHeadDim + col) * wgt;
          l += __ldcg(pi + kMaxGroup * kHeadDim + kMaxGroup + h) * wgt;
        }
        const float outv = l > 0.f ? o / l : 0.f;
        p.out[((int64_t)b * p.H_q + kvh * p.G + h) * kHeadDim + col] = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
        if (p.lse != nullptr && col == 0)
          p.lse[(int64_t)b * p.H_q + kvh * p.G + h] = l > 0.f ? (M + log2f(l)) * kLn2 : -INFINITY;
      }
      if (tid == 0) p.tickets[bk] = 0;
    }
  }
  // ---- the last KV head to finish advances the step counter ----
  // (every CTA read the counter before it got here, so the update cannot reach a reader of this launch)
  if (append && head_done && tid == 0) {
    const int n_heads = p.B * p.H_kv;
    if (atomicAdd(&p.tickets[n_heads], 1) == n_heads - 1) {
      p.tickets[n_heads] = 0;
      *p.d_step = step + 1;
    }
  }
}

// How many clusters of each size can be resident at once when a CTA takes a whole SM (a cluster must fit into
// one GPC, so this is not n_sm / size: on this part 15 clusters of 8 but 22 of 6).  Filled by decode_setup.
static int g_cluster_cap[kDecodeMaxCluster + 1];

// Clusters of 8 CTAs, the portable limit.  (16-CTA clusters were tried: too few of them are co-resident on
// this part, so the grid ran in two waves.)
cudaError_t decode_setup() {
  cudaError_t e = cudaFuncSetAttribute(decode_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kDecodeMaxTiles * 2 * kTileBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(decode_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kDecodeMaxTiles * 2 * kTileBytes);
  if (e != cudaSuccess) return e;
  for (int c = 4; c <= kDecodeMaxCluster; ++c) {
    if (c == 7) continue;                                // never chosen (no more of them fit than of 8)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(c * 64), 1, 1);
    cfg.blockDim = dim3(kDecodeMaxWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = kDecodeMaxTiles * 2 * kTileBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, decode_attn_kernel<false>, &cfg) != cudaSuccess) {
      (void)cudaGetLastError();
      n = 0;                                             // unknown: this size is then not considered
    }
    g_cluster_cap[c] = n;
  }
  return cudaSuccess;
}

// Warps and staging bytes of a CTA that gets per_cta tiles
static void decode_cta_shape(int per_cta, int *n_warps, int *smem_bytes) {
  int w = (per_cta + 1) / 2;                                                     // two tiles per warp and pass
  if (per_cta > 2 * 9) w = kDecodeMaxTiles / 2;                                  // several passes: use every slot
  else if (w > 9) w = 9;
  if (w < 1) w = 1;
  *n_warps = w;
  *smem_bytes = (per_cta < 2 * w ? per_cta : 2 * w) * 2 * kTileBytes;
}

// Launch geometry for a reduced cache of L rows: one cluster per KV head whose CTAs go through their
// tiles in passes of (two tiles per warp); more clusters per head only beyond kDecodeMaxPasses passes.
// heads = batch x KV heads of the launch (0: not known).  When a CTA needs a whole SM and the heads do not fit
// at once as clusters of 8, smaller clusters are weighed: more of them are resident, each takes longer
// (measured on this part at L = 2049 and 4097: about 4.5 us + 0.1 us per tile of a CTA + 1 us per extra pass).
void decode_geometry(int L, int heads, int *n_clusters, int *cs, int *n_warps, int *smem_bytes) {
  const int n_tiles = (L + 15) / 16;
  int c = 1;
  while (c < kDecodeMaxCluster && c * 2 <= n_tiles) c <<= 1;                     // cluster size 1, 2, 4 or 8
  const int per_pass = kDecodeMaxTiles;                                          // tiles a CTA can stage at once
  const int nc = (n_tiles + c * per_pass * kDecodeMaxPasses - 1) / (c * per_pass * kDecodeMaxPasses);
  int per_cta = (n_tiles + c * nc - 1) / (c * nc);                               // most tiles a CTA gets
  decode_cta_shape(per_cta, n_warps, smem_bytes);
  if (c == kDecodeMaxCluster && nc == 1 && *smem_bytes > 12 * 2 * kTileBytes && heads > g_cluster_cap[c] &&
      g_cluster_cap[c] > 0) {
    float best = 0.f;
    int best_c = c;
    for (int cand = kDecodeMaxCluster; cand >= 4; --cand) {
      const int cap = g_cluster_cap[cand];
      if (cap <= 0 || n_tiles > cand * per_pass * kDecodeMaxPasses) continue;
      const int per = (n_tiles + cand - 1) / cand, passes = (per + per_pass - 1) / per_pass;
      const float cost = (float)((heads + cap - 1) / cap) * (4.5f + 0.1f * (float)per + (float)(passes - 1));
      if (cand == kDecodeMaxCluster || cost < best) { best = cost; best_c = cand; }
    }
    c = best_c;
    per_cta = (n_tiles + c - 1) / c;
    decode_cta_shape(per_cta, n_warps, smem_bytes);
  }
  *n_clusters = nc;
  *cs = c;
}

cudaError_t launch_decode(const DecodeParams &p, cudaStream_t stream) {
  int n_clusters, cs, n_warps, smem;
  decode_geometry(p.L, p.B * p.H_kv, &n_clusters, &cs, &n_warps, &smem);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_clusters * cs), (unsigned)p.H_kv, (unsigned)p.B);
  cfg.blockDim = dim3((unsigned)(n_warps * 32), 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.pdl_mode > 0 ? 2 : 1;
  const int n_tiles = (p.L + 15) / 16;
  const int per_cta = (n_tiles + n_clusters * cs - 1) / (n_clusters * cs);
  return per_cta > 2 * n_warps ? cudaLaunchKernelEx(&cfg, decode_attn_kernel<true>, p)
                               : cudaLaunchKernelEx(&cfg, decode_attn_kernel<false>, p);
}

}  // namespace sagekv
