// Step 4: append the new token to the recent window, then attention of every query head over its view
// of the reduced cache (sink + its own selected segment + window).
//
// Flash-decoding on thread-block clusters.  The L rows of one KV head are cut into 16-row tiles that are
// dealt evenly, as contiguous ranges, to the CTAs of one cluster.  A CTA brings its K and V tiles into shared
// memory with tensor copies (one 16-row x 64-column box per request, 128-byte swizzle, completion counted on
// an mbarrier), issued by a ninth warp that does nothing else.  The staging area has 50 slots of one tile
// (K or V) each.  All K tiles of the range are resident from the start; so are the V tiles while slots last,
// and the remaining V tiles take over the K slots as soon as the first product is done.  There is one pass:
//   S = K Q^T     16 rows x 8 heads per mma, a tile per warp in turn (the scores of all its tiles stay in
//                 registers).  A fragments come from the swizzled tile with ldmatrix, the query (B fragments)
//                 sits in registers.
//   softmax       ONE maximum per head over the whole CTA (two block barriers in all), so nothing is ever
//                 rescaled; the weights, rounded to bf16, go to shared memory for all tiles.
//   O^T = V^T P   split by COLUMNS: warp w accumulates columns 16w..16w+15 of all heads over all rows
//                 (transposing ldmatrix for V, the weights as B fragments).  The warps' results are
//                 disjoint, so nothing is exchanged or summed inside the CTA.
// Every head masks the rows of the other heads' segments.  The CTAs of a cluster are merged through
// distributed shared memory: each warp sends its 16 columns straight from registers into the inbox of the
// CTA that finishes those columns with asynchronous stores counted on that CTA's barrier (one way, no
// cluster barrier), and each CTA writes its slice of the 128 output columns.  With several clusters per
// head (caches beyond 44 tiles per CTA: a warp keeps the scores of at most six) the cluster results go to scratch and the CTA that arrives last
// (one atomic ticket, no waiting) merges them.
// The staged copy of the window row that the new token replaces is overwritten in shared memory from
// k_new / v_new once it has landed, and the CTA owning that row stores the new token into the cache.
// Every wait on a copy barrier is bounded: a wait that runs out sets kStatusWaitTimeout in the context's status
// word and the CTA runs on with whatever its shared memory holds, so every block and cluster barrier is still
// reached and the kernel ends; the output of such a launch is meaningless and the status word says so.
#include <cooperative_groups.h>
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "trace.cuh"

namespace cg = cooperative_groups;

namespace sagekv {

constexpr int kDecodeThreads = (kDecodeWarps + 1) * 32;   // eight consumer warps and the warp that issues the copies
constexpr int kConsumerThreads = kDecodeWarps * 32;
constexpr int kDecodeBaseCluster = 8;          // the cluster size tried first (the portable limit)
constexpr int kSlotBytes = 16 * 256;           // a slot of the staging area: 16 rows of K or of V
constexpr int kHalfBytes = 16 * 128;           // 16 rows x 64 columns: one box of the tensor copy
constexpr int kPHeadWords = 12;                // 32-bit words per (tile, head) of the weight buffer: 8 used, 4 spread the banks
constexpr int kPTileWords = kMaxGroup * kPHeadWords;
constexpr int kQkGroup = 3;                    // tiles of the first product a warp works on at once
constexpr int kQkTiles = (kDecodeMaxTiles + kDecodeWarps - 1) / kDecodeWarps;   // tiles a warp may get in the first product (6)
constexpr uint32_t kWaitLimit = 1u << 22;      // polls of a copy barrier before giving up (each poll already blocks for a while)

struct DecShared {
  // softmax weights: [tile][head][row pair g: rows 2g, 2g + 1]; the tensor-memory variant keeps its two small
  // operands here instead (12 KB of weights, 4 KB of queries, both in the 128-byte-swizzled operand layout, which
  // wants 1024-byte alignment: the struct sits behind the staging area, on such a boundary)
  alignas(1024) uint32_t P[kDecodeMaxTiles * kPTileWords];
  unsigned long long bar[5];                                   // K landed, early V landed, late V landed; scores ready, outputs ready (tensor-memory variant)
  unsigned long long inbox_bar;                                // every CTA's share for this CTA's columns has landed
  unsigned long long ml_bar;                                   // every CTA's (max, sum) pairs have landed (they travel ahead of the columns)
  int last;
  uint32_t tmem_base;                                          // tensor-memory variant: first column of the CTA's allocation
  int pad_[2];
  float warp_m[kDecodeWarps][kMaxGroup];                       // maxima of the warps' rows
  float warp_l[kDecodeWarps][kMaxGroup];                       // sums of the warps' (rounded) weights
  float2 inbox_ml[kDecodeMaxCluster][kMaxGroup];               // [source CTA][head] (max, sum)
  float inbox_o[(kHeadDim + 4 * kDecodeMaxCluster) * kMaxGroup];   // [source CTA][my column][head]; cluster size x columns <= 160
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// false: the wait ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// one box of a [batch, head, row, column] bf16 tensor -> shared memory; the copy reads this GPU's memory only
// (the cache rows are read once per call: they are marked evict-first in L2, so that the small operands every
// call reads after its dependency wait, q and the step counter, tend to stay there)
__device__ __forceinline__ void tensor_copy_4d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, int w, uint32_t bar,
                                               uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, fp32) = A(16x16, bf16, row) * B(16x8, bf16, col): the first link of an accumulator chain
__device__ __forceinline__ void mma_first(float &d0, float &d1, float &d2, float &d3, uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// Byte offset, inside a staged K or V tile (two 2 KB boxes: columns 0..63 and 64..127), of the 16-byte piece
// `piece` (0..15) of row `row` (0..15): the 128-byte swizzle of the tensor copy XORs the piece index within a
// 128-byte line with the line index modulo 8 (the boxes start on 1024-byte boundaries).
__device__ __forceinline__ uint32_t tile_offset(int row, int piece) {
  return (uint32_t)((piece >> 3) * kHalfBytes + row * 128 + (((piece & 7) ^ (row & 7)) << 4));
}

// keeps a value that was worked out early in a register, so that the work is not redone (later) where it is used
__device__ __forceinline__ void pin(uint32_t &x) { asm volatile("" : "+r"(x)); }
__device__ __forceinline__ void pin(int &x) { asm volatile("" : "+r"(x)); }

__device__ __forceinline__ void bar_sync(int id, int n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

// n_slots: slots of this launch's staging area (min(2 * most tiles of a CTA, kDecodeSlots)).
// kLong: a CTA may have more tiles than half the slots (part of V arrives late, a warp may have up to six tiles in
// the first product); false keeps the common case free of that.
template <bool kLong>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_attn_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const int n_slots) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t stage = (raw + 1023u) & ~1023u;                 // the slots: boxes on 1024-byte boundaries
  DecShared &sh = *reinterpret_cast<DecShared *>(smem_raw + (stage - raw) + (size_t)n_slots * kSlotBytes);

  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int ci = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;    // ci: CTA index within the head
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  const int h0 = 2 * c, h1 = 2 * c + 1;                           // the two heads a lane's accumulators belong to
  const bool producer = warp == kDecodeWarps;
  const bool append = p.k_new != nullptr;
  SAGEKV_TRACE_BEGIN
  SAGEKV_STAMP(0);

  // tiles of this CTA: an even deal of the head's n_tiles over the gridDim.x CTAs, contiguous ranges
  const int n_tiles = (p.L + 15) >> 4;
  const int base_n = n_tiles / (int)gridDim.x, rem = n_tiles % (int)gridDim.x;
  const int first_tile = ci * base_n + min(ci, rem);
  const int n = base_n + (ci < rem ? 1 : 0);                      // my tiles: K tile t in slot t
  // V tile t sits in slot n + t while slots last (the early ones, requested at once); the others (late) take
  // slot n + t - n_slots, a K slot, once the first product is done
  constexpr int kQk = kLong ? kQkTiles : kQkGroup;           // tiles of the first product a warp may have
  const int n_early = kLong ? min(n, n_slots - n) : n, n_late = n - n_early;
  auto v_slot = [&](int t) { return (!kLong || t < n_early) ? n + t : n + t - n_slots; };

  // columns each CTA of the cluster finishes: a multiple of 4, the last CTA may get fewer
  const int cols = ((kHeadDim + cs - 1) / cs + 3) & ~3;
  const int my_cols = max(0, min(cols, kHeadDim - rank * cols));
  const int n_pairs = (p.G + 1) >> 1;                             // head pairs in use

  const uint32_t kbar = smem_u32(&sh.bar[0]), vbar_e = smem_u32(&sh.bar[1]), vbar_l = smem_u32(&sh.bar[2]);
  const uint32_t inbox_bar = smem_u32(&sh.inbox_bar);
  const uint32_t ml_bar = smem_u32(&sh.ml_bar);
  if (tid == 0) {
    mbar_init(kbar, 1);
    mbar_init(vbar_e, 1);
    mbar_init(vbar_l, 1);
    mbar_init(inbox_bar, 1);
    mbar_init(ml_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    // from every CTA of the cluster: 8 bytes per (own column, head pair in use) and 64 bytes of (max, sum) pairs
    mbar_expect_tx(inbox_bar, (uint32_t)(cs * my_cols * n_pairs * 8));
    mbar_expect_tx(ml_bar, (uint32_t)(cs * 64));
  }
  __syncthreads();
  cluster.barrier_arrive();                              // waited for just before the first store into a peer: its barrier is set up

  // Programmatic dependent launch: until the wait returns, nothing that an earlier kernel on the stream may
  // still be writing is read (q, k_new, v_new, the step counter) and nothing at all is written to global
  // memory.  In prefetch mode the rows of the reduced cache are requested first: the caller has promised that
  // the kernel directly before this one does not write this layer's cache.  The successor is released only
  // after the wait, so at most one kernel runs ahead of its dependency.
  if (p.pdl_mode < 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }

  // ---- the warp that issues the copies: lane i takes requests i, i + 32, ... (two boxes per tile) ----
  if (producer) {
    uint64_t stream_policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
    auto issue = [&](const CUtensorMap *map, int t_lo, int t_hi, bool is_v, uint32_t bar) {   // tiles [t_lo, t_hi)
      if (lane == 0 && t_hi > t_lo) mbar_expect_tx(bar, (uint32_t)(t_hi - t_lo) * kSlotBytes);
      __syncwarp();
      for (int op = lane; op < (t_hi - t_lo) * 2; op += 32) {
        const int t = t_lo + (op >> 1), hf = op & 1;
        const uint32_t dst = stage + (uint32_t)((is_v ? v_slot(t) : t) * kSlotBytes + hf * kHalfBytes);
        tensor_copy_4d(dst, map, hf * 64, (first_tile + t) << 4, kvh, b, bar, stream_policy);
      }
    };
    // (In prefetch mode this warp never waits for the predecessor: it reads nothing of it, and what it requests
    // after barrier A comes after the consumers' wait.  It leaves the release of the successor to the consumers,
    // who give it after their wait: a release from here would let a second launch run ahead.)
    issue(&map_k, 0, n, false, kbar);
    issue(&map_v, 0, n_early, true, vbar_e);
    bar_sync(1, kDecodeThreads);                         // A: every consumer warp is done with the K slots
    if (kLong && n_late > 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // their reads (and a patched row) precede the refill
      issue(&map_v, n_early, n, true, vbar_l);
    }
    return;                                              // (its cluster arrival at entry stands; it takes part in nothing else)
  }

  // ---- everything that does not depend on the predecessor's results is worked out before the wait ----
  // The instructions after the wait form one long dependent chain per warp, so every address, mask and index
  // that can be known now is computed now and kept in a register.
  // (1) which of this lane's score elements are visible to their heads (sink, own segment, window): bit 4i + e
  //     for the warp's i-th tile, element e of the accumulator
  // Row order of the K fragments: A row m of the mma (m < 8) holds token 2m (m < 4) or 2m + 1, A row m + 8 the
  // other token of the pair (2m, 2m + 1).  So a lane's accumulators belong to two neighbouring tokens, whose
  // weights make one 32-bit word of the second product's B fragment, and the eight rows one ldmatrix phase
  // reads still fall into eight different bank groups of the swizzled tile.
  const int win_lo = p.S + p.n_sel;
  const int seg0_lo = p.S + (p.pooled ? 0 : h0 * p.k_q), seg0_hi = seg0_lo + p.k_q;
  const int seg1_lo = p.S + (p.pooled ? 0 : h1 * p.k_q), seg1_hi = seg1_lo + p.k_q;
  uint32_t vis = 0;
#pragma unroll
  for (int i = 0; i < kQk; ++i) {
    const int r0 = ((first_tile + warp + kDecodeWarps * i) << 4) + 2 * g;
    const int ra = r0 + (g >= 4 ? 1 : 0), rb = r0 + (g >= 4 ? 0 : 1);   // tokens of accumulator elements 0, 1 and 2, 3
    const bool va = ra < p.L, vb = rb < p.L;
    const bool sa = ra < p.S || ra >= win_lo, sb = rb < p.S || rb >= win_lo;
    vis |= (va && h0 < p.G && (sa || (ra >= seg0_lo && ra < seg0_hi)) ? 1u : 0u) << (4 * i);
    vis |= (va && h1 < p.G && (sa || (ra >= seg1_lo && ra < seg1_hi)) ? 2u : 0u) << (4 * i);
    vis |= (vb && h0 < p.G && (sb || (rb >= seg0_lo && rb < seg0_hi)) ? 4u : 0u) << (4 * i);
    vis |= (vb && h1 < p.G && (sb || (rb >= seg1_lo && rb < seg1_hi)) ? 8u : 0u) << (4 * i);
  }
  // (2) fragment addresses: K rows for the first product (ldmatrix), V for the second (transposing ldmatrix), the
  //     weight words this lane writes and reads
  const int mi = lane >> 3, l8 = lane & 7;
  const int arow = 2 * l8 + (((mi & 1) != 0) != (l8 >= 4) ? 1 : 0);
  uint32_t k_off[8];                                     // k-step ks of a tile: slot base + k_off[ks]
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) k_off[ks] = tile_offset(arow, 2 * ks + (mi >> 1));
  const uint16_t *q_lane = p.q + ((int64_t)b * p.H_q + kvh * p.G + min(g, p.G - 1)) * kHeadDim + 2 * c;   // this lane's first query element
  uint32_t v_off = tile_offset((mi >> 1) * 8 + l8, 2 * warp + (mi & 1));
  uint32_t pw_addr = smem_u32(sh.P) + (uint32_t)((h0 * kPHeadWords + g) * 4);   // + tile * kPTileWords * 4; head h1: + kPHeadWords * 4
  uint32_t pr_addr = smem_u32(sh.P) + (uint32_t)((g * kPHeadWords + c) * 4);    // + tile * kPTileWords * 4; rows 2c+8, 2c+9: + 16
  // (3) where this lane's results go: the owners of its two columns, as addresses in their shared memory
  const int col_a = 16 * warp + g, col_b = col_a + 8;
  const int own_a = col_a / cols, own_b = col_b / cols;
  uint32_t dst_a, dst_b, bar_a, bar_b, dst_ml = 0, bar_ml = 0;
  {
    const uint32_t inbox = smem_u32(sh.inbox_o);
    const uint32_t la = inbox + (uint32_t)(((rank * cols + (col_a - own_a * cols)) * kMaxGroup + h0) * 4);
    const uint32_t lb = inbox + (uint32_t)(((rank * cols + (col_b - own_b * cols)) * kMaxGroup + h0) * 4);
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst_a) : "r"(la), "r"(own_a));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst_b) : "r"(lb), "r"(own_b));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar_a) : "r"(inbox_bar), "r"(own_a));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar_b) : "r"(inbox_bar), "r"(own_b));
    if (warp == 0 && g < cs) {                           // lane (g, c) of warp 0 tells CTA g the (max, sum) of heads 2c, 2c+1
      const uint32_t lm = smem_u32(&sh.inbox_ml[rank][h0]);
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst_ml) : "r"(lm), "r"(g));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar_ml) : "r"(ml_bar), "r"(g));
    }
  }
  // (4) integer divisions cost a hundred instructions apiece: the ones the tail needs are done here, and the step
  //     counter is reduced modulo the ring length with a reciprocal worked out here
  int n_clusters = (int)gridDim.x / cs, cl = ci / cs;
  uint32_t ring_magic = 0xffffffffu / (uint32_t)max(p.ring_len, 1);
  pin(n_clusters); pin(cl); pin(ring_magic);
  // (5) the finishing stage: one thread per output value (own column lc, head fh)
  const int fin_items = my_cols * p.G, n_src = cs;
  int fin_lc = tid / p.G, fin_h = tid - fin_lc * p.G;
  uint16_t *fin_out = p.out + ((int64_t)b * p.H_q + kvh * p.G + fin_h) * kHeadDim + rank * cols + fin_lc;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) pin(k_off[ks]);
  asm volatile("" : "+l"(q_lane)); pin(v_off); pin(pw_addr); pin(pr_addr); pin(dst_a); pin(dst_b); pin(bar_a); pin(bar_b); pin(dst_ml); pin(bar_ml);
  pin(vis); pin(fin_lc); pin(fin_h); asm volatile("" : "+l"(fin_out));

  SAGEKV_STAMP(1);
  if (p.pdl_mode >= 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  SAGEKV_STAMP(2);

  // What the predecessor may have written is read now, all requests issued back to back (query first: the first
  // product needs it; the step counter last: only the patch of the replaced row needs it), so the round trips to
  // L2 overlap instead of queueing behind one another.
  uint32_t qb[8][2];                      // B fragments of Q^T: lane (g, c) holds head g's dims 16ks + 2c, +1 and 16ks + 8 + 2c, +1
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) qb[ks][0] = qb[ks][1] = 0u;
  if (g < p.G) {
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      asm volatile("ld.global.b32 %0, [%1];" : "=r"(qb[ks][0]) : "l"(q_lane + 16 * ks));
      asm volatile("ld.global.b32 %0, [%1];" : "=r"(qb[ks][1]) : "l"(q_lane + 16 * ks + 8));
    }
  }
  const uint16_t *kn = append ? p.k_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  const uint16_t *vn = append ? p.v_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  uint4 new_row = make_uint4(0u, 0u, 0u, 0u);            // lanes 0-15: 16 bytes of k_new, lanes 16-31: of v_new
  int step = 0, my_ticket = -1;
  if (append) {
    new_row = ld_v4((lane < 16 ? kn : vn) + (lane & 15) * 8);
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(step) : "l"(p.d_step));
    // One ticket per CTA, taken once the counter has been read, by a thread of the warp with the fewest tiles.
    // The increment is computed from the value read (its sign bit, never set, plus one), so the atomic cannot
    // be issued before the load has returned; a release fence in its place held the warp for 0.5 us, and the
    // block barrier after the first product with it.  The answer is looked at only when the CTA is done.
    if (tid == kConsumerThreads - 1)
      asm volatile("{ .reg .b32 inc; shr.u32 inc, %2, 31; add.u32 inc, inc, 1; atom.add.relaxed.gpu.global.s32 %0, [%1], inc; }"
                   : "=r"(my_ticket) : "l"(p.tickets + p.B * p.H_kv), "r"(step) : "memory");
  }

  bool timed_out = false;                 // a copy never arrived: reported through the status word; the CTA runs on (its output is then meaningless)
  if (n > 0 && !mbar_wait(kbar, 0u)) timed_out = true;
  SAGEKV_STAMP(3);

  // the staged copy of the replaced row is stale: the warp that works on its tile patches K now, and V as soon as
  // the tile's V copy is here (now, for an early tile; after the first product, for a late one)
  int slot = -1, st = -1;                 // the replaced window row and its CTA-local tile (if 0 <= st < n)
  if (append) {
    uint32_t r = (uint32_t)step - __umulhi((uint32_t)step, ring_magic) * (uint32_t)p.ring_len;   // the quotient may be one short
    while (r >= (uint32_t)p.ring_len) r -= (uint32_t)p.ring_len;
    slot = p.S + p.n_sel + (int)r;
    st = (slot >> 4) - first_tile;
  }
  const bool patcher = append && st >= 0 && st < n && (st & (kDecodeWarps - 1)) == warp;
  auto patch = [&](bool is_v) {           // lanes 0-15 hold the new K row, lanes 16-31 the new V row
    if ((lane >= 16) == is_v) {
      const int row = slot & 15, piece = lane & 15;
      const uint32_t dst = stage + (uint32_t)((is_v ? v_slot(st) : st) * kSlotBytes) + tile_offset(row, piece);
      asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(new_row.x), "r"(new_row.y), "r"(new_row.z), "r"(new_row.w) : "memory");
    }
  };
  if (patcher) {
    patch(false);
    if (st < n_early) {
      if (!mbar_wait(vbar_e, 0u)) timed_out = true;
      patch(true);
    }
    if (SAGEKV_OK_INDEX(p.status, slot >= 0 && slot < p.L)) {
      uint16_t *gdst = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                       (int64_t)slot * p.cs.token_stride + (lane & 15) * 8;
      st_v4(gdst, new_row);
    }
    __syncwarp();
  }

  // ---- S = K Q^T: this warp's tiles are warp, warp + 8, ...; three at a time ----
  // An mma takes far longer than its issue slot, so the work is laid out as short independent chains: per
  // tile four accumulators (k-steps j and j + 4), the fragments requested ahead of the mmas.
  float sv[kQk][4];
  float wm0 = -INFINITY, wm1 = -INFINITY;
#pragma unroll
  constexpr int kGrp = kLong ? 2 : kQkGroup;                // tiles at once: two where the scores of six tiles stay in registers
  for (int grp = 0; grp < kQk / kGrp; ++grp) {
    if (warp + kDecodeWarps * kGrp * grp < n) {
      float ch[kGrp][4][4];
      uint32_t fa[kGrp][4][4];
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {                   // k-steps 0..3, then 4..7
#pragma unroll
        for (int i = 0; i < kGrp; ++i) {
          const int t = warp + kDecodeWarps * (kGrp * grp + i);
          if (t < n) {
            const uint32_t tb = stage + (uint32_t)(t * kSlotBytes);
#pragma unroll
            for (int j = 0; j < 4; ++j) ldmatrix_x4(tb + k_off[4 * hf + j], fa[i][j][0], fa[i][j][1], fa[i][j][2], fa[i][j][3]);
          }
        }
#pragma unroll
        for (int i = 0; i < kGrp; ++i) {
          if (warp + kDecodeWarps * (kGrp * grp + i) < n) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (hf == 0)
                mma_first(ch[i][j][0], ch[i][j][1], ch[i][j][2], ch[i][j][3], fa[i][j][0], fa[i][j][1], fa[i][j][2], fa[i][j][3],
                          qb[j][0], qb[j][1]);
              else
                mma_bf16_16816(ch[i][j][0], ch[i][j][1], ch[i][j][2], ch[i][j][3], fa[i][j][0], fa[i][j][1], fa[i][j][2], fa[i][j][3],
                               qb[4 + j][0], qb[4 + j][1]);
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kGrp; ++i) {
        const int ti = kGrp * grp + i;
        const bool have = warp + kDecodeWarps * ti < n;
        const uint32_t vb4 = have ? (vis >> (4 * ti)) & 15u : 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float x = have ? (ch[i][0][e] + ch[i][1][e]) + (ch[i][2][e] + ch[i][3][e]) : 0.f;
          sv[ti][e] = ((vb4 >> e) & 1u) ? x * p.scale_log2 : -INFINITY;
        }
        wm0 = fmaxf(wm0, fmaxf(sv[ti][0], sv[ti][2]));
        wm1 = fmaxf(wm1, fmaxf(sv[ti][1], sv[ti][3]));
      }
    } else {
#pragma unroll
      for (int i = 0; i < kGrp; ++i)
        sv[kGrp * grp + i][0] = sv[kGrp * grp + i][1] = sv[kGrp * grp + i][2] = sv[kGrp * grp + i][3] = -INFINITY;
    }
  }
  // over the eight lanes that hold the same heads (equal c)
  // (three exchange steps: measured, redux.sync.max.f32 over such a partial lane mask took 0.2 us apiece)
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    wm0 = fmaxf(wm0, __shfl_xor_sync(0xffffffffu, wm0, o));
    wm1 = fmaxf(wm1, __shfl_xor_sync(0xffffffffu, wm1, o));
  }
  if (g == 0) { sh.warp_m[warp][h0] = wm0; sh.warp_m[warp][h1] = wm1; }
  bar_sync(1, kDecodeThreads);   // A: the maxima are complete, and nobody reads a K slot any more (the copy warp refills them)

  float M0, M1;                  // maxima of heads 2c, 2c+1 over the CTA's rows (log2 units)
  {
    float a0[kDecodeWarps], a1[kDecodeWarps];
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) { a0[w] = sh.warp_m[w][h0]; a1[w] = sh.warp_m[w][h1]; }
#pragma unroll
    for (int s2 = kDecodeWarps / 2; s2 > 0; s2 >>= 1)   // a tree, not a chain
#pragma unroll
      for (int w = 0; w < s2; ++w) { a0[w] = fmaxf(a0[w], a0[w + s2]); a1[w] = fmaxf(a1[w], a1[w + s2]); }
    M0 = a0[0]; M1 = a1[0];
  }
  SAGEKV_STAMP_AFTER(4, M0 + M1);
  const float s0 = M0 == -INFINITY ? 0.f : M0, s1 = M1 == -INFINITY ? 0.f : M1;
  // the weights enter the second product as bf16: one word per (tile, head, row pair g: rows 2g and 2g + 1);
  // their sums per head are taken from the rounded values, so that numerator and denominator agree
  float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
  for (int i = 0; i < kQk; ++i) {
    const int t = warp + kDecodeWarps * i;
    if (t < n) {
      const float x0 = fast_exp2(sv[i][0] - s0), x2 = fast_exp2(sv[i][2] - s0);              // head h0: elements 0 and 2
      const float x1 = fast_exp2(sv[i][1] - s1), x3 = fast_exp2(sv[i][3] - s1);              // head h1: elements 1 and 3
      const uint32_t p0 = g < 4 ? pack_bf16x2(x0, x2) : pack_bf16x2(x2, x0);                 // (row 2g in the low half)
      const uint32_t p1 = g < 4 ? pack_bf16x2(x1, x3) : pack_bf16x2(x3, x1);
      ls0 += __uint_as_float(p0 << 16) + __uint_as_float(p0 & 0xffff0000u);                  // the weights as rounded
      ls1 += __uint_as_float(p1 << 16) + __uint_as_float(p1 & 0xffff0000u);
      const uint32_t wa = pw_addr + (uint32_t)(t * kPTileWords * 4);
      asm volatile("st.shared.u32 [%0], %1;" ::"r"(wa), "r"(p0) : "memory");
      asm volatile("st.shared.u32 [%0], %1;" ::"r"(wa + kPHeadWords * 4), "r"(p1) : "memory");
    }
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    ls0 += __shfl_xor_sync(0xffffffffu, ls0, o);
    ls1 += __shfl_xor_sync(0xffffffffu, ls1, o);
  }
  if (g == 0) { sh.warp_l[warp][h0] = ls0; sh.warp_l[warp][h1] = ls1; }
  bar_sync(2, kConsumerThreads);   // B: the weights are in shared memory (and a patched early V row is visible)
  SAGEKV_STAMP(5);
  // The (max, sum) pairs of the CTA go to every CTA of the cluster now, ahead of the second product, with
  // asynchronous stores that count their bytes on a barrier of their own at the receiver: the finishing stage
  // has its weights ready before the columns arrive.
  cluster.barrier_wait();                                // pairs with the arrive at kernel entry: every peer runs, its barriers are set up
  auto send2 = [&](uint32_t addr, uint32_t rbar, float x, float y) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(addr), "f"(x), "f"(y), "r"(rbar) : "memory");
  };
  if (warp == 0 && g < cs) {
    float L0 = 0.f, L1 = 0.f;            // sums of the (bf16-rounded) weights of heads 2c, 2c+1 over the CTA's rows
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) { L0 += sh.warp_l[w][h0]; L1 += sh.warp_l[w][h1]; }
    send2(dst_ml, bar_ml, M0, L0);
    send2(dst_ml + 8u, bar_ml, M1, L1);
  }

  // ---- O^T = V^T P: columns 16*warp .. +15 over all rows, the early V tiles first ----
  // A B fragment is two of the weight words (rows 2c, 2c+1 and 2c+8, 2c+9 of head g).  Six tiles per step, each on an
  // accumulator chain of its own, all fragments requested before the mmas.  (An mma's result takes about 130
  // cycles: the sums of the weights used to come from a second mma per tile against a fragment of ones, on two
  // chains eleven links long, and those chains alone took 0.75 us; they are summed in registers now.)
  float acc[4] = {0.f, 0.f, 0.f, 0.f};    // O^T: (col_a, h0) (col_a, h1) (col_b, h0) (col_b, h1)
  float xc[5][4];
#pragma unroll
  for (int u = 0; u < 5; ++u) xc[u][0] = xc[u][1] = xc[u][2] = xc[u][3] = 0.f;
  auto second_product = [&](int t_lo, int t_hi) {
    for (int t6 = t_lo; t6 < t_hi; t6 += 6) {
      uint32_t va[6][4], pb[6][2];
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        if (t6 + u < t_hi) {
          ldmatrix_x4_trans(stage + (uint32_t)(v_slot(t6 + u) * kSlotBytes) + v_off, va[u][0], va[u][1], va[u][2], va[u][3]);
          const uint32_t ra = pr_addr + (uint32_t)((t6 + u) * kPTileWords * 4);
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(pb[u][0]) : "r"(ra));
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(pb[u][1]) : "r"(ra + 16));
        }
      }
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        if (t6 + u < t_hi) {
          if (u == 0) mma_bf16_16816(acc[0], acc[1], acc[2], acc[3], va[u][0], va[u][1], va[u][2], va[u][3], pb[u][0], pb[u][1]);
          else mma_bf16_16816(xc[u - 1][0], xc[u - 1][1], xc[u - 1][2], xc[u - 1][3], va[u][0], va[u][1], va[u][2], va[u][3], pb[u][0], pb[u][1]);
        }
      }
    }
  };
  if (n_early > 0 && !mbar_wait(vbar_e, 0u)) timed_out = true;
  second_product(0, n_early);
  if (kLong && n_late > 0) {                             // (the same for every thread of the CTA)
    if (!mbar_wait(vbar_l, 0u)) timed_out = true;
    if (patcher && st >= n_early) patch(true);
    bar_sync(2, kConsumerThreads);                       // a patched late V row is visible
    second_product(n_early, n);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) acc[e] += ((xc[0][e] + xc[1][e]) + (xc[2][e] + xc[3][e])) + xc[4][e];
  if (timed_out) atomicOr(p.status, kStatusWaitTimeout);
  SAGEKV_STAMP_AFTER(6, acc[0] + acc[1] + acc[2] + acc[3]);

  // ---- merge the CTAs of the cluster: the owner of a column slice receives it from every CTA ----
  // Every warp sends its 16 columns straight from registers into the owners' inboxes with asynchronous stores
  // that count their bytes on the owner's barrier: data and signal travel together and nobody waits for an
  // acknowledgement or for a cluster-wide barrier; a CTA only waits for its own inbox to fill.
  if (h0 < p.G) {
    send2(dst_a, bar_a, acc[0], acc[1]);
    send2(dst_b, bar_b, acc[2], acc[3]);
  }
  SAGEKV_STAMP(7);
  // the weights of the sources for this thread's first output: worked out while the columns are still on their way
  float fin_w[kDecodeMaxCluster], fin_M = -INFINITY, fin_inv = 0.f, fin_l = 0.f;
  auto source_weights = [&](int h) {
    float mx[kDecodeMaxCluster], lsum[kDecodeMaxCluster];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) {
      const float2 ml = sI < n_src ? sh.inbox_ml[sI][h] : make_float2(-INFINITY, 0.f);
      mx[sI] = ml.x; lsum[sI] = ml.y;
    }
    float tm[kDecodeMaxCluster];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) tm[sI] = mx[sI];
#pragma unroll
    for (int w2 = kDecodeMaxCluster / 2; w2 > 0; w2 >>= 1)
#pragma unroll
      for (int sI = 0; sI < w2; ++sI) tm[sI] = fmaxf(tm[sI], tm[sI + w2]);
    fin_M = tm[0];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) {
      fin_w[sI] = fin_M == -INFINITY ? 0.f : fast_exp2(mx[sI] - fin_M);
      lsum[sI] *= fin_w[sI];
    }
#pragma unroll
    for (int w2 = kDecodeMaxCluster / 2; w2 > 0; w2 >>= 1)
#pragma unroll
      for (int sI = 0; sI < w2; ++sI) lsum[sI] += lsum[sI + w2];
    fin_l = lsum[0];
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(fin_inv) : "f"(fin_l));   // the output is rounded to bf16: an approximate reciprocal is ample
  };
  if (!mbar_wait(ml_bar, 0u) && tid == 0) atomicOr(p.status, kStatusWaitTimeout);
  if (tid < fin_items) source_weights(fin_h);
  if (!mbar_wait(inbox_bar, 0u) && tid == 0) atomicOr(p.status, kStatusWaitTimeout);
  SAGEKV_STAMP(8);

  // ---- finish columns [rank*cols, rank*cols + my_cols) of every head from the inbox ----
  const int bk = b * p.H_kv + kvh;
  float *part = p.partials + ((int64_t)bk * n_clusters + cl) * kPartialStride;
  for (int item = tid; item < fin_items; item += kConsumerThreads) {
    if (item != tid) {
      fin_lc = item / p.G;
      fin_h = item - fin_lc * p.G;
      fin_out = p.out + ((int64_t)b * p.H_q + kvh * p.G + fin_h) * kHeadDim + rank * cols + fin_lc;
    }
    if (item != tid) source_weights(fin_h);
    const int lc = fin_lc, h = fin_h, col = rank * cols + lc;
    float ov[kDecodeMaxCluster];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI)       // the loads of all sources are in flight together
      ov[sI] = sI < n_src ? sh.inbox_o[(sI * cols + lc) * kMaxGroup + h] * fin_w[sI] : 0.f;
#pragma unroll
    for (int w2 = kDecodeMaxCluster / 2; w2 > 0; w2 >>= 1)
#pragma unroll
      for (int sI = 0; sI < w2; ++sI) ov[sI] += ov[sI + w2];
    const float o = ov[0], l = fin_l, M = fin_M;
    if (n_clusters == 1) {
      const float outv = l > 0.f ? o * fin_inv : 0.f;
      *fin_out = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
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

  if (n_clusters > 1) {
    // ---- several clusters per head: the last CTA to arrive merges the cluster results ----
    __threadfence();
    bar_sync(2, kConsumerThreads);
    if (tid == 0) sh.last = atomicAdd(&p.tickets[bk], 1) == (int)gridDim.x - 1;
    bar_sync(2, kConsumerThreads);
    if (sh.last != 0) {
      __threadfence();
      const float *all = p.partials + (int64_t)bk * n_clusters * kPartialStride;
      for (int item = tid; item < p.G * kHeadDim; item += kConsumerThreads) {
        const int h = item >> 7, col = item & 127;
        float M = -INFINITY;
        for (int i = 0; i < n_clusters; ++i) M = fmaxf(M, __ldcg(all + i * kPartialStride + kMaxGroup * kHeadDim + h));
        float o = 0.f, l = 0.f;
        for (int i = 0; i < n_clusters; ++i) {
          const float *pi = all + i * kPartialStride;
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
  // ---- the step counter: whoever took the last ticket of the launch knows that every CTA has read it ----
  if (append && tid == kConsumerThreads - 1 && my_ticket == (int)(gridDim.x * gridDim.y * gridDim.z) - 1) {
    p.tickets[p.B * p.H_kv] = 0;
    *p.d_step = step + 1;
  }
  SAGEKV_STAMP(9);
  SAGEKV_TRACE_END(p.out);
}

}  // namespace sagekv

#include "decode_attn_tc.cuh"

namespace sagekv {

static size_t decode_tc_smem_bytes(int per_cta) {
  return 1024 + (size_t)((per_cta + 7) / 8) * kTcBlockBytes + (size_t)per_cta * kSlotBytes + sizeof(DecShared);
}

static_assert(1024 + (size_t)kDecodeSlots * kSlotBytes + sizeof(DecShared) <= 232448, "the staging area and the rest fit into 227 KB");
static int decode_slots(int per_cta) { return 2 * per_cta < kDecodeSlots ? 2 * per_cta : kDecodeSlots; }
static size_t decode_smem_bytes(int per_cta) {
  return 1024 + (size_t)decode_slots(per_cta) * kSlotBytes + sizeof(DecShared);
}

// How many clusters of `c` CTAs that take `tiles` tiles each can be on the device at once (a cluster must fit
// into one GPC, so this is not n_sm / c: on this part 15 clusters of 8 whole-SM CTAs but 22 of 6).  Asked of the
// runtime once per (device, size, tiles) and remembered.  0: unknown.
static int g_cluster_cap[64][kDecodeMaxCluster + 1][kDecodeMaxTiles + 1];   // answer + 1; 0 = not asked yet
static std::mutex g_cap_mutex;

static int cluster_capacity(int device, int c, int tiles) {
  if (device < 0 || device >= 64 || c < 1 || c > kDecodeMaxCluster || tiles < 0 || tiles > kDecodeMaxTiles) return 0;
  std::lock_guard<std::mutex> lock(g_cap_mutex);
  int &slot = g_cluster_cap[device][c][tiles];
  if (slot == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(c * 64), 1, 1);
    cfg.blockDim = dim3(kDecodeThreads, 1, 1);
    cfg.dynamicSmemBytes = decode_smem_bytes(tiles);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int nn = 0;
    if (cudaOccupancyMaxActiveClusters(&nn, decode_attn_kernel<true>, &cfg) != cudaSuccess) {
      (void)cudaGetLastError();
      nn = 0;
    }
    slot = nn + 1;
  }
  return slot - 1;
}

cudaError_t decode_setup(DeviceInfo *dev) {
  (void)dev;
  const cudaError_t e = cudaFuncSetAttribute(decode_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)decode_smem_bytes(kDecodeMaxTiles));
  if (e != cudaSuccess) return e;
  const cudaError_t e2 = cudaFuncSetAttribute(decode_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)decode_smem_bytes(kDecodeMaxTiles));
  if (e2 != cudaSuccess) return e2;
  return cudaFuncSetAttribute(decode_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)decode_tc_smem_bytes(kTcMaxTiles));
}

// Launch geometry for a reduced cache of L rows: nc clusters of c CTAs per KV head, a CTA taking at most
// kDecodeMaxTiles tiles (its K tiles must all be resident); nc > 1 only beyond that, the clusters' results then
// merged through scratch by the last CTA to arrive.  heads = batch x KV heads of the launch (0, or dev null: not
// known; then clusters of 8).  Back-to-back launches overlap (the next one fetches its rows while this one
// computes), which only works if the clusters of two launches fit on the device together, so the cluster sizes
// are compared by a cost fitted to measurements (below).
// (15 clusters of 8 whole-SM CTAs fit at once, 22 of 6, 26 of 5, 33 of 4.)
void decode_geometry(int L, int heads, const DeviceInfo *dev, int *n_clusters, int *cs, int *per_cta_tiles, int *smem_bytes) {
  const int n_tiles = (L + 15) / 16;
  int c = 1;
  while (c < kDecodeBaseCluster && c * 2 <= n_tiles) c <<= 1;                   // cluster size 1, 2, 4 or 8
  int nc = (n_tiles + c * kDecodeMaxTiles - 1) / (c * kDecodeMaxTiles);          // the fewest clusters per head
  if (dev != nullptr && heads > 0 && c == kDecodeBaseCluster) {
    float best = 0.f;
    int best_c = c, best_nc = nc;
    // up to kDecodeExtraClusters more clusters per head than needed: beyond one cluster the results are merged
    // through scratch anyway, and more, smaller clusters leave fewer V tiles waiting for a K slot
    for (int n_try = nc; n_try <= (nc > 1 ? nc + kDecodeExtraClusters : nc); ++n_try) {
      for (int cand = kDecodeBaseCluster; cand >= 4; --cand) {
        const int per = (n_tiles + cand * n_try - 1) / (cand * n_try);
        if (per > kDecodeMaxTiles) continue;
        const int cap = cluster_capacity(dev->device, cand, per);
        if (cap <= 0) continue;
        // measured on this part (us per launch, batch 1 x 8 heads, L = 1025 / 2049 / 4097, clusters of 5 to 8):
        // 2.97 + 0.0445 per tile of a CTA; the same again per tile when the clusters of two launches do not fit
        // together (the copies are then issued on the critical path); 0.084 per V tile that has to wait for a K
        // slot; 2.6 for the merge through scratch (L = 8193)
        const int late = 2 * per > kDecodeSlots ? 2 * per - kDecodeSlots : 0;
        const int waves = (heads * n_try + cap - 1) / cap;                      // of one launch
        const float one = 2.97f + 0.0445f * (float)per * (2 * heads * n_try <= cap ? 1.f : 2.f) + 0.084f * (float)late +
                          (n_try > 1 ? 2.6f : 0.f);
        const float cost = (float)waves * one;
        if (best == 0.f || cost < best) { best = cost; best_c = cand; best_nc = n_try; }
      }
    }
    c = best_c;
    nc = best_nc;
  } else if (nc > 1) {
    nc += kDecodeExtraClusters;                          // (context set-up: the most clusters per head a launch may choose)
  }
  const int per_cta = (n_tiles + c * nc - 1) / (c * nc);                         // most tiles a CTA gets
  *n_clusters = nc;
  *cs = c;
  *per_cta_tiles = per_cta;
  *smem_bytes = (int)decode_smem_bytes(per_cta);
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link against the driver)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
    else
      (void)cudaGetLastError();
  });
  return fn;
}

// [B, H_kv, L, 128] bf16 through the cache strides, boxes of 16 rows x 64 columns with the 128-byte swizzle;
// rows at and beyond L read as zeros
static bool make_cache_map(CUtensorMap *map, const uint16_t *base, const DecodeParams &p) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (enc == nullptr) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)p.L, (cuuint64_t)p.H_kv, (cuuint64_t)p.B};
  const cuuint64_t strides[3] = {(cuuint64_t)p.cs.token_stride * 2, (cuuint64_t)p.cs.head_stride * 2,
                                 (cuuint64_t)p.cs.batch_stride * 2};
  const cuuint32_t box[4] = {64, 16, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<uint16_t *>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_decode(const DecodeParams &p, const DeviceInfo &dev, cudaStream_t stream) {
  int n_clusters, cs, per_cta, smem;
  decode_geometry(p.L, p.B * p.H_kv, &dev, &n_clusters, &cs, &per_cta, &smem);
  CUtensorMap map_k, map_v;
  if (!make_cache_map(&map_k, p.Kc, p) || !make_cache_map(&map_v, p.Vc, p)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_clusters * cs), (unsigned)p.H_kv, (unsigned)p.B);
  cfg.blockDim = dim3(kDecodeThreads, 1, 1);
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
  // the tensor-memory variant where it applies: one cluster per head, every tile resident twice over
  if (p.variant == 2 && n_clusters == 1 && per_cta <= kTcMaxTiles) {
    cfg.dynamicSmemBytes = decode_tc_smem_bytes(per_cta);
    return cudaLaunchKernelEx(&cfg, decode_attn_tc_kernel, p, map_k, map_v, per_cta);
  }
  // the short instance keeps three tiles' scores per warp and has every V tile resident from the start
  const bool is_long = 2 * per_cta > kDecodeSlots || per_cta > kQkGroup * kDecodeWarps;
  return is_long ? cudaLaunchKernelEx(&cfg, decode_attn_kernel<true>, p, map_k, map_v, decode_slots(per_cta))
                                    : cudaLaunchKernelEx(&cfg, decode_attn_kernel<false>, p, map_k, map_v, decode_slots(per_cta));
}

}  // namespace sagekv

SAGEKV_TRACE_READER(sagekv_trace_read)
