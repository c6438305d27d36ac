// Step 4 on the fifth-generation tensor cores: the variant of decode_attn_kernel for caches whose tiles all fit
// into the staging area twice over (the common case).  Included by decode_attn.cu, whose helpers it uses.
//
// What differs from decode_attn_kernel: both products are issued by ONE thread as tcgen05.mma instructions that
// read their operands from shared memory themselves and accumulate in tensor memory, instead of eight warps
// pulling every K and V tile through ldmatrix into mma.sync (that path is bound by the shared-memory port: 88 KB
// per product through 128 bytes per clock, and P once per warp on top).
//   S = K Q^T     M = 128 tokens (a block of eight tiles), N = 16 (the KV head's query heads, padded), K = 128
//                 dims in eight instructions.  K tiles land in blocks of eight: [block][column half][128 rows x
//                 128 bytes], the K-major operand layout with the 128-byte swizzle the tensor copy already applies.
//                 The query is written by the threads into the same layout (2 x 16 rows x 128 bytes).
//   softmax       every thread reads the scores of one token (a tensor-memory lane) per block and all heads; one
//                 maximum per head over the CTA; the weights go to shared memory as the K-major B operand of the
//                 second product (16 heads x 64 tokens per 2 KB chunk), their sums are taken from the rounded values.
//   O^T = V^T P   M = 128 dims, N = 16 heads, K = 16 tokens per instruction, one per tile.  A V tile as the tensor
//                 copy leaves it ([16 tokens][64 dims] twice) IS the MN-major operand layout: nothing is moved.
// Measured on B200 (C3-2048, 22 tiles per CTA): every tcgen05.mma of M = 128 takes about 110 clocks whatever N is
// (one operand row per clock), so the 24 + 22 instructions of a CTA take 1.3 + 1.2 us, against 0.55 + 0.83 us on
// the mma.sync path, and a launch 5.65 us against 4.14 us.  With so few useful columns the contraction is too
// narrow for this unit; the variant is kept as a checked alternative (sagekv_set_decode_variant), not the default.
// The rest (tensor copies by a ninth warp, dependent launch, patch of the replaced row, one-way merge through the
// owners' inboxes, finishing stage, step-counter ticket) is the same as in decode_attn_kernel.
//
// Every wait (copy barriers, the two barriers the tensor core arrives on) is bounded; tensor memory is freed on
// every path, by the warp that allocated it.
#pragma once

namespace sagekv {

constexpr int kTcBlockBytes = 8 * kSlotBytes;        // eight K tiles: 128 rows x 256 bytes, as two column halves
constexpr int kTcHalfBytes = 8 * kHalfBytes;         // 128 rows x 128 bytes
constexpr int kTcMaxTiles = 22;                      // tiles per CTA: three blocks (their K blocks and V tiles fit the staging area)
constexpr int kTcMaxBlocks = (kTcMaxTiles + 7) / 8;
constexpr int kTcColumns = 64;                       // tensor-memory columns: 16 per score block, 16 for the output
constexpr int kTcOutColumn = 16 * kTcMaxBlocks;
constexpr int kTcQBytes = 4096;                      // the query operand: 2 column halves x 16 rows x 128 bytes
constexpr uint32_t kTcWaitLimit = 1u << 14;        // polls of a barrier the tensor core arrives on (each poll blocks for a while)
constexpr int kTcPBytes = 12288;                     // the weight operand: 6 chunks of 64 tokens x 16 heads
static_assert(kTcPBytes + kTcQBytes <= (int)sizeof(uint32_t) * kDecodeMaxTiles * kPTileWords, "operands fit the weight buffer");
static_assert(kTcMaxTiles * 16 <= 6 * 64, "weight chunks cover the tokens");

// shared-memory operand descriptor (Blackwell format): start address, leading and stride byte offsets in
// 16-byte units, version 1, 128-byte swizzle
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor of kind::f16: fp32 accumulators, bf16 A and B, N = 16, M = 128; a_mn: A is MN-major
__device__ __forceinline__ uint32_t tc_idesc(bool a_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn ? (1u << 15) : 0u) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u) : "memory");
}
// the barrier gets one arrival when every tcgen05.mma this thread has issued so far is complete
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// lane i of the warp gets columns col .. col + 7 of tensor-memory lane 32 * (warp % 4) + i
__device__ __forceinline__ void tc_load8(uint32_t taddr, float (&x)[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
  // (the registers are operands of the wait, so that no use of them can be scheduled ahead of it)
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]) :: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ bool tc_wait(uint32_t bar) {
  for (uint32_t i = 0; i < kTcWaitLimit; ++i)
    if (mbar_try_wait(bar, 0u)) return true;
  return false;
}

// per_cta: the most tiles a CTA of this launch gets (the staging area holds ceil(per_cta / 8) K blocks and per_cta
// V tiles); at most kTcMaxTiles.
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_attn_tc_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const int per_cta) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t stage = (raw + 1023u) & ~1023u;                 // K blocks, then V tiles: everything on 1024-byte boundaries
  const int n_blocks_room = (per_cta + 7) >> 3;
  const uint32_t v_base = stage + (uint32_t)(n_blocks_room * kTcBlockBytes);
  DecShared &sh = *reinterpret_cast<DecShared *>(smem_raw + (stage - raw) + (size_t)n_blocks_room * kTcBlockBytes +
                                                 (size_t)per_cta * kSlotBytes);
  const uint32_t p_base = smem_u32(sh.P), q_base = p_base + kTcPBytes;

  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int ci = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool producer = warp == kDecodeWarps;
  const bool append = p.k_new != nullptr;
  SAGEKV_TRACE_BEGIN
  SAGEKV_STAMP(0);

  // tiles of this CTA: an even deal of the head's n_tiles over the gridDim.x CTAs, contiguous ranges
  const int n_tiles = (p.L + 15) >> 4;
  const int base_n = n_tiles / (int)gridDim.x, rem = n_tiles % (int)gridDim.x;
  const int first_tile = ci * base_n + min(ci, rem);
  const int n = base_n + (ci < rem ? 1 : 0);                      // my tiles (<= per_cta)
  const int n_blocks = (n + 7) >> 3;                              // blocks of 128 tokens in use

  const int cols = ((kHeadDim + cs - 1) / cs + 3) & ~3;           // columns each CTA of the cluster finishes
  const int my_cols = max(0, min(cols, kHeadDim - rank * cols));
  const int n_pairs = (p.G + 1) >> 1;

  const uint32_t kbar = smem_u32(&sh.bar[0]), vbar = smem_u32(&sh.bar[1]);
  const uint32_t sbar = smem_u32(&sh.bar[3]), obar = smem_u32(&sh.bar[4]);
  const uint32_t inbox_bar = smem_u32(&sh.inbox_bar);
  if (warp == 0) {
    if (lane == 0) {
      mbar_init(kbar, 1);
      mbar_init(vbar, 1);
      mbar_init(sbar, 1);
      mbar_init(obar, 1);
      mbar_init(inbox_bar, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
      mbar_expect_tx(inbox_bar, (uint32_t)(cs * (my_cols * n_pairs * 8 + 64)));
    }
    __syncwarp();
    // 64 columns of tensor memory for the CTA (one CTA per SM: nobody competes for them)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(kTcColumns) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the two small operands start as zeros: rows of heads that do not exist must be finite
  if (!producer) {
#pragma unroll
    for (int i = 0; i < (kTcPBytes + kTcQBytes) / (16 * kConsumerThreads); ++i)
      asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(p_base + (uint32_t)((i * kConsumerThreads + tid) * 16)), "r"(0u) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  cluster.barrier_arrive();                              // waited for just before the first store into a peer

  if (p.pdl_mode < 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }

  // ---- the ninth warp: requests the copies, then issues the two products ----
  if (producer) {
    uint64_t stream_policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
    if (lane == 0 && n > 0) {
      mbar_expect_tx(kbar, (uint32_t)n * kSlotBytes);
      mbar_expect_tx(vbar, (uint32_t)n * kSlotBytes);
    }
    __syncwarp();
    for (int op = lane; op < n * 2; op += 32) {            // K: tile t, column half hf -> its place in block t / 8
      const int t = op >> 1, hf = op & 1;
      const uint32_t dst = stage + (uint32_t)((t >> 3) * kTcBlockBytes + hf * kTcHalfBytes + (t & 7) * kHalfBytes);
      tensor_copy_4d(dst, &map_k, hf * 64, (first_tile + t) << 4, kvh, b, kbar, stream_policy);
    }
    for (int op = lane; op < n * 2; op += 32) {            // V: tile t as two boxes, one behind the other
      const int t = op >> 1, hf = op & 1;
      tensor_copy_4d(v_base + (uint32_t)(t * kSlotBytes + hf * kHalfBytes), &map_v, hf * 64, (first_tile + t) << 4, kvh, b, vbar,
                     stream_policy);
    }
    // The descriptors are worked out here, ahead of the barriers: between them only additions remain.
    const uint64_t k_desc = tc_desc(stage, 16, 1024), q_desc = tc_desc(q_base, 16, 1024);
    const uint64_t v_desc = tc_desc(v_base, kHalfBytes, 1024), p_desc = tc_desc(p_base, 16, 1024);
    const uint32_t idesc_s = tc_idesc(false), idesc_o = tc_idesc(true);
    bool late = false;
    bar_sync(1, kDecodeThreads);                           // A: the query is in shared memory, the replaced K row patched
    if (lane == 0 && n > 0) {
      if (!mbar_wait(kbar, 0u)) late = true;
      tc_fence_after();
#pragma unroll
      for (int blk = 0; blk < kTcMaxBlocks; ++blk) {
        if (blk < n_blocks) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {                 // 16 dims per instruction: 32 bytes along a swizzled row
            const uint64_t off = (uint64_t)((((ks >> 2) * kTcHalfBytes + (ks & 3) * 32) >> 4));
            const uint64_t qoff = (uint64_t)(((ks >> 2) * 2048 + (ks & 3) * 32) >> 4);
            tc_mma(tmem + (uint32_t)(blk * 16), k_desc + (uint64_t)(blk * (kTcBlockBytes >> 4)) + off, q_desc + qoff, idesc_s, ks > 0);
          }
        }
      }
      tc_commit(sbar);
    } else if (lane == 0) {
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sbar) : "memory");   // no tiles: nothing to wait for
    }
    __syncwarp();
    bar_sync(3, kDecodeThreads);                           // C: the weights are in shared memory, the replaced V row patched
    if (lane == 0 && n > 0) {
      if (!mbar_wait(vbar, 0u)) late = true;
      tc_fence_after();
      uint64_t a = v_desc, bp = p_desc;
      for (int t = 0; t < n; t += 4) {                     // 16 tokens per instruction: one V tile, 32 bytes of a weight row
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (t + u < n) tc_mma(tmem + (uint32_t)kTcOutColumn, a + (uint64_t)(u * (kSlotBytes >> 4)), bp + (uint64_t)(u * 2), idesc_o, t + u > 0);
        a += 4 * (kSlotBytes >> 4);
        bp += 2048 >> 4;
      }
      tc_commit(obar);
      if (!tc_wait(obar)) late = true;               // the warp stays until the tensor core is done with shared memory
      if (late) atomicOr(p.status, kStatusWaitTimeout);
    } else if (lane == 0) {
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(obar) : "memory");
    }
    __syncwarp();
    return;                                                // (its cluster arrival at entry stands)
  }

  // ---- consumer warps: everything that does not depend on the predecessor is worked out before the wait ----
  // Warp w reads tensor-memory lanes 32 (w % 4) .. + 31: in a score block lane = token, in the output lane = dim.
  // Warps 0-3 take score blocks 0 and 2, warps 4-7 block 1; warps 0-3 read the output.
  const int q4 = warp & 3, wg = warp >> 2;
  const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
  const int win_lo = p.S + p.n_sel;
  uint32_t vis = 0;                                       // bit 8 j + h: head h sees this thread's token of its j-th block
  int lt[2];                                              // the tokens, counted from the CTA's first row
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int blk = wg + 2 * j;
    lt[j] = blk * 128 + q4 * 32 + lane;
    const int r = (first_tile << 4) + lt[j];
    const bool ok = blk < n_blocks && lt[j] < (n << 4) && r < p.L;
    const bool shared_row = r < p.S || r >= win_lo;
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
      const int seg_lo = p.S + (p.pooled ? 0 : h * p.k_q);
      if (ok && h < p.G && (shared_row || (r >= seg_lo && r < seg_lo + p.k_q))) vis |= 1u << (8 * j + h);
    }
  }
  // where this thread's weights go: chunk of 64 tokens, row = head, 16-byte piece (token / 8) ^ head, 2 bytes per token
  uint32_t pw[2];
#pragma unroll
  for (int j = 0; j < 2; ++j) pw[j] = p_base + (uint32_t)((lt[j] >> 6) * 2048 + (lt[j] & 7) * 2);
  const int piece = (lt[0] & 63) >> 3;                    // the same for both blocks (they are 256 tokens apart)
  // where the results go: the owner of output column d, as an address in its shared memory
  const int d = q4 * 32 + lane;
  const int own = d / cols;
  uint32_t dst_o, bar_o, dst_ml = 0, bar_ml = 0;
  {
    const uint32_t lo = smem_u32(sh.inbox_o) + (uint32_t)(((rank * cols + (d - own * cols)) * kMaxGroup) * 4);
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst_o) : "r"(lo), "r"(own));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar_o) : "r"(inbox_bar), "r"(own));
    if (warp == 0 && (lane >> 2) < cs) {                   // lane (g, c) of warp 0 tells CTA g the (max, sum) of heads 2c, 2c+1
      const uint32_t lm = smem_u32(&sh.inbox_ml[rank][2 * (lane & 3)]);
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst_ml) : "r"(lm), "r"(lane >> 2));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar_ml) : "r"(inbox_bar), "r"(lane >> 2));
    }
  }
  // the finishing stage: one thread per output value (own column lc, head fh)
  const int fin_items = my_cols * p.G, n_src = cs;
  int fin_lc = tid / p.G, fin_h = tid - fin_lc * p.G;
  uint16_t *fin_out = p.out + ((int64_t)b * p.H_q + kvh * p.G + fin_h) * kHeadDim + rank * cols + fin_lc;
  // the query: thread (head, piece) moves 16 bytes into the operand layout
  const bool q_mover = tid < p.G * 16;
  const uint16_t *q_src = p.q + ((int64_t)b * p.H_q + kvh * p.G + min(tid >> 4, p.G - 1)) * kHeadDim + (tid & 15) * 8;
  const uint32_t q_dst = q_base + (uint32_t)(((tid & 15) >> 3) * 2048 + (tid >> 4) * 128 + ((((tid & 15) & 7) ^ ((tid >> 4) & 7)) << 4));
  pin(vis); pin(pw[0]); pin(pw[1]); pin(dst_o); pin(bar_o); pin(dst_ml); pin(bar_ml); pin(fin_lc); pin(fin_h);
  asm volatile("" : "+l"(fin_out));
  asm volatile("" : "+l"(q_src));

  SAGEKV_STAMP(1);
  if (p.pdl_mode >= 2) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  SAGEKV_STAMP(2);

  // What the predecessor may have written is read now, all requests issued back to back (the query first).
  uint4 qv = make_uint4(0u, 0u, 0u, 0u);
  if (q_mover) qv = ld_v4(q_src);
  const uint16_t *kn = append ? p.k_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  const uint16_t *vn = append ? p.v_new + ((int64_t)b * p.H_kv + kvh) * kHeadDim : nullptr;
  uint4 new_row = make_uint4(0u, 0u, 0u, 0u);            // lanes 0-15: 16 bytes of k_new, lanes 16-31: of v_new
  int step = 0, my_ticket = -1;
  if (append) {
    new_row = ld_v4((lane < 16 ? kn : vn) + (lane & 15) * 8);
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(step) : "l"(p.d_step));
    // one ticket per CTA, ordered after the read of the counter by a data dependency (see decode_attn_kernel)
    if (tid == kConsumerThreads - 1)
      asm volatile("{ .reg .b32 inc; shr.u32 inc, %2, 31; add.u32 inc, inc, 1; atom.add.relaxed.gpu.global.s32 %0, [%1], inc; }"
                   : "=r"(my_ticket) : "l"(p.tickets + p.B * p.H_kv), "r"(step) : "memory");
  }
  if (q_mover) asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(q_dst), "r"(qv.x), "r"(qv.y), "r"(qv.z), "r"(qv.w) : "memory");

  // the staged copy of the replaced window row is stale: one warp patches K now, V after the first barrier
  bool timed_out = false;
  int slot = -1, st = -1;
  if (append) {
    slot = p.S + p.n_sel + step % p.ring_len;
    st = (slot >> 4) - first_tile;
  }
  const bool patcher = append && st >= 0 && st < n && (st & (kDecodeWarps - 1)) == warp;
  if (patcher) {
    if (!mbar_wait(kbar, 0u)) timed_out = true;
    if (lane < 16) {
      const int row = slot & 15;
      const uint32_t dst = stage + (uint32_t)((st >> 3) * kTcBlockBytes + (lane >> 3) * kTcHalfBytes + (st & 7) * kHalfBytes + row * 128 +
                                              (((lane & 7) ^ (row & 7)) << 4));
      asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(new_row.x), "r"(new_row.y), "r"(new_row.z), "r"(new_row.w) : "memory");
    }
    if (SAGEKV_OK_INDEX(p.status, slot >= 0 && slot < p.L)) {
      uint16_t *gdst = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                       (int64_t)slot * p.cs.token_stride + (lane & 15) * 8;
      st_v4(gdst, new_row);
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads what the threads have just written
  bar_sync(1, kDecodeThreads);                           // A

  // ---- scores: one token per thread and block, all heads ----
  if (!tc_wait(sbar)) timed_out = true;
  tc_fence_after();
  SAGEKV_STAMP(3);
  float x[2][kMaxGroup];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    if (wg + 2 * j < n_blocks) {                          // (the same for the whole warp)
      tc_load8(tmem + lane_base + (uint32_t)((wg + 2 * j) * 16), x[j]);
    } else {
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h) x[j][h] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) x[j][h] = ((vis >> (8 * j + h)) & 1u) ? x[j][h] * p.scale_log2 : -INFINITY;
  }
  // one maximum per head over the CTA: over the warp as order-preserving integers, then through shared memory
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    if (h < p.G) {
      const uint32_t key = __reduce_max_sync(0xffffffffu, score_key(fmaxf(x[0][h], x[1][h])));
      if (lane == 0) sh.warp_m[warp][h] = __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
    }
  }
  bar_sync(2, kConsumerThreads);
  SAGEKV_STAMP(4);
  float ls[kMaxGroup];                                    // sums of this thread's weights, as rounded
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    ls[h] = 0.f;
    if (h < p.G) {
      float M = sh.warp_m[0][h];
#pragma unroll
      for (int w = 1; w < kDecodeWarps; ++w) M = fmaxf(M, sh.warp_m[w][h]);
      const float s0 = M == -INFINITY ? 0.f : M;
      const uint32_t off = (uint32_t)(h * 128 + ((piece ^ h) << 4));
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (wg + 2 * j < n_blocks && lt[j] < (n << 4)) {
          const uint32_t wb = pack_bf16x2(fast_exp2(x[j][h] - s0), 0.f) & 0xffffu;
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(pw[j] + off), "h"((unsigned short)wb) : "memory");
          ls[h] += __uint_as_float(wb << 16);
        }
      }
    }
  }
  if (patcher) {                                           // the replaced V row, in the tile as the tensor copy left it
    if (!mbar_wait(vbar, 0u)) timed_out = true;
    if (lane >= 16) {
      const uint32_t dst = v_base + (uint32_t)(st * kSlotBytes) + tile_offset(slot & 15, lane & 15);
      asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(new_row.x), "r"(new_row.y), "r"(new_row.z), "r"(new_row.w) : "memory");
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  bar_sync(3, kDecodeThreads);                           // C: the second product may start
  SAGEKV_STAMP(5);

  // ---- while the tensor core works: the sums of the weights, and the (max, sum) pairs to every CTA ----
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) {
    if (h < p.G) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ls[h] += __shfl_xor_sync(0xffffffffu, ls[h], o);
      if (lane == 0) sh.warp_l[warp][h] = ls[h];
    }
  }
  bar_sync(2, kConsumerThreads);
  cluster.barrier_wait();                                // pairs with the arrive at kernel entry: every peer runs, its barrier is set up
  auto send2 = [&](uint32_t addr, uint32_t rbar, float a, float c2) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(addr), "f"(a), "f"(c2), "r"(rbar) : "memory");
  };
  if (warp == 0 && (lane >> 2) < cs) {
    const int h0 = 2 * (lane & 3), h1 = h0 + 1;
    float M0 = -INFINITY, M1 = -INFINITY, L0 = 0.f, L1 = 0.f;
#pragma unroll
    for (int w = 0; w < kDecodeWarps; ++w) {
      M0 = fmaxf(M0, sh.warp_m[w][h0]); M1 = fmaxf(M1, sh.warp_m[w][h1]);
      L0 += sh.warp_l[w][h0]; L1 += sh.warp_l[w][h1];
    }
    if (h0 >= p.G) { M0 = -INFINITY; L0 = 0.f; }
    if (h1 >= p.G) { M1 = -INFINITY; L1 = 0.f; }
    send2(dst_ml, bar_ml, M0, L0);
    send2(dst_ml + 8u, bar_ml, M1, L1);
  }

  // ---- outputs: warps 0-3 read one dim per thread, all heads, and send them to the owners of the columns ----
  if (!tc_wait(obar)) timed_out = true;
  tc_fence_after();
  SAGEKV_STAMP(6);
  if (wg == 0) {
    float o[kMaxGroup];
    tc_load8(tmem + lane_base + (uint32_t)kTcOutColumn, o);
#pragma unroll
    for (int pr = 0; pr < kMaxGroup / 2; ++pr)
      if (pr < n_pairs) send2(dst_o + (uint32_t)(8 * pr), bar_o, n > 0 ? o[2 * pr] : 0.f, n > 0 ? o[2 * pr + 1] : 0.f);
  }
  if (timed_out) atomicOr(p.status, kStatusWaitTimeout);
  // tensor memory goes back once every warp has read what it needs
  tc_fence_before();
  bar_sync(2, kConsumerThreads);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcColumns) : "memory");
  }
  SAGEKV_STAMP(7);
  if (!mbar_wait(inbox_bar, 0u) && tid == 0) atomicOr(p.status, kStatusWaitTimeout);
  SAGEKV_STAMP(8);

  // ---- finish columns [rank*cols, rank*cols + my_cols) of every head from the inbox ----
  for (int item = tid; item < fin_items; item += kConsumerThreads) {
    if (item != tid) {
      fin_lc = item / p.G;
      fin_h = item - fin_lc * p.G;
      fin_out = p.out + ((int64_t)b * p.H_q + kvh * p.G + fin_h) * kHeadDim + rank * cols + fin_lc;
    }
    const int lc = fin_lc, h = fin_h, col = rank * cols + lc;
    float mx[kDecodeMaxCluster], lsum[kDecodeMaxCluster], ov[kDecodeMaxCluster];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) {   // the loads of all sources are in flight together
      const float2 ml = sI < n_src ? sh.inbox_ml[sI][h] : make_float2(-INFINITY, 0.f);
      mx[sI] = ml.x; lsum[sI] = ml.y;
      ov[sI] = sI < n_src ? sh.inbox_o[(sI * cols + lc) * kMaxGroup + h] : 0.f;
    }
    float tm[kDecodeMaxCluster];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) tm[sI] = mx[sI];
#pragma unroll
    for (int w2 = kDecodeMaxCluster / 2; w2 > 0; w2 >>= 1)
#pragma unroll
      for (int sI = 0; sI < w2; ++sI) tm[sI] = fmaxf(tm[sI], tm[sI + w2]);
    const float M = tm[0];
#pragma unroll
    for (int sI = 0; sI < kDecodeMaxCluster; ++sI) {
      const float wgt = M == -INFINITY ? 0.f : fast_exp2(mx[sI] - M);
      ov[sI] *= wgt; lsum[sI] *= wgt;
    }
#pragma unroll
    for (int w2 = kDecodeMaxCluster / 2; w2 > 0; w2 >>= 1)
#pragma unroll
      for (int sI = 0; sI < w2; ++sI) { ov[sI] += ov[sI + w2]; lsum[sI] += lsum[sI + w2]; }
    const float o = ov[0], l = lsum[0];
    float inv;                                             // the output is rounded to bf16: an approximate reciprocal is ample
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(l));
    const float outv = l > 0.f ? o * inv : 0.f;
    *fin_out = (uint16_t)(pack_bf16x2(outv, 0.f) & 0xffffu);
    if (p.lse != nullptr && col == 0)
      p.lse[(int64_t)b * p.H_q + kvh * p.G + h] = l > 0.f ? (M + log2f(l)) * kLn2 : -INFINITY;
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
