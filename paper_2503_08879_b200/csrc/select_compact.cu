// Step 2 (second half) and Step 3: per-query-head top-k over the score rows, then the gather that
// builds the reduced cache  C = Concat(sink, selected, recent, last).
//
// One thread-block cluster (up to 8 CTAs) owns one score row.  Each CTA stages its contiguous slice of
// the row in shared memory once (cp.async, 16 bytes per request); every later step works on that copy, so
// the scores cross the memory system a single time.  When the row carries the group maxima of the score
// step (see common.cuh) the slice is needed only once: it is not staged but requested into L2 with one bulk
// prefetch and read from there, and the cluster shrinks when there are more rows than cluster slots.
//
// Fast path (k_q small against the row, the normal case): a prefilter instead of a full radix select.
//   1. every thread takes the maximum of its elements; the cluster's thread maxima are exchanged over
//      distributed shared memory (or all of the row's group maxima are read from behind the row: a hint that
//      is checked by its outcome, see fast_select).  The k_q-th largest of these maxima is a lower bound T0 of the k_q-th
//      largest score (k_q distinct elements are >= it), and it is tight: about k_q * (1 + few %) scores
//      are >= T0.  T0 is taken as the lower edge of the histogram bin (512 bins laid over the actual
//      range of the maxima) in which that maximum falls.
//   2. scores >= T0 become candidates (order-preserving key, position), written in position order; every
//      CTA takes a copy of all lists, CTA by CTA, so each holds the same position-sorted candidate list.
//   3. every CTA decides for all candidates: a histogram of the candidate keys finds the bin of the k_q-th
//      largest; candidates above it are kept, the few inside it are ranked exactly, with the position as
//      tie-break (lowest positions win).
//   4. a kept candidate's output slot is the number of kept candidates before it in the list (one prefix sum):
//      ascending positions.  Each CTA writes and gathers an even share of the slots.
// General path (k_q large, tiny rows, or more candidates than the buffers hold, e.g. a row of equal
// scores): three-digit radix select (11 + 11 + 10 bits) with histograms merged in CTA 0's shared memory by
// distributed-shared-memory atomics, then a ballot/popcount ranking in row order.
// The rows on a CTA's list are then copied into the head's segment of the reduced cache (general path: the
// CTA that owns a kept element copies it), together with a share of the KV head's sink, recent and last rows.
#include <cooperative_groups.h>

#include "common.cuh"
#include "trace.cuh"

namespace cg = cooperative_groups;

namespace sagekv {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxCluster = 8;
constexpr int kMaxBins = 2048;
constexpr int kSelSmemLimit = 227 * 1024;             // the most a CTA can have on this part
constexpr int kGeneralScratch = 4 * kMaxBins * 4;   // general path: three merged histograms and the local one

struct SelShared {
  uint32_t hist_fast[kSelThreads];     // fast path: histogram of the thread maxima
  uint32_t gmax[kSelThreads];          // thread maxima of this CTA, read by the peers
  uint32_t red[3][kSelWarps];
  uint32_t gstat[kMaxCluster][4];      // (min, max, count) of every CTA's non-empty thread maxima, pushed by the peers
  int totals[kMaxCluster][2];          // general path: (kept-larger, equal-to-threshold) per CTA; rank 0's copy
  int cand_cnt[kMaxCluster];           // fast path: candidates per CTA, pushed by each CTA to every peer
  int wsum[kSelWarps + 1];             // fast path: candidates per warp, then those among the slice's tail elements
  int warp_cnt[kSelWarps][2];
  int scan_tmp[kSelWarps];
  int found[2];
  int list_count;
  int n_border;
  int pad_[3];
};
static_assert(sizeof(SelShared) % 16 == 0, "staged scores must stay 16-byte aligned");

__device__ __forceinline__ float key_to_score(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// exclusive prefix of v over the CTA in thread order
__device__ __forceinline__ int block_exclusive_scan(int v, int *tmp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += n;
  }
  __syncthreads();                     // tmp may still be read from an earlier call
  if (lane == 31) tmp[warp] = inc;
  __syncthreads();
  // the totals of the warps before this one: one load per lane and one warp-wide sum (not a chain of loads)
  const int base = __reduce_add_sync(0xffffffffu, lane < warp ? tmp[lane] : 0);
  return base + inc - v;
}

// In a histogram of nb bins (nb = 1024 or 2048), find the bin in which the k-th largest key falls, counting
// from the top bin down.  found[0] = bin, found[1] = rank of the key inside that bin.  Ends with a barrier.
__device__ __forceinline__ void find_bin_from_top(const uint32_t *hist, int nb, int k, SelShared &sh) {
  const int tid = threadIdx.x;
  const int per = nb / kSelThreads;    // thread t looks at bins nb-1-t*per ... downwards
  uint32_t cnt[4];
  int mine = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    cnt[e] = 0;
    if (e < per) {
      cnt[e] = hist[nb - 1 - (tid * per + e)];
      mine += (int)cnt[e];
    }
  }
  int above = block_exclusive_scan(mine, sh.scan_tmp);   // keys in higher bins
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (e < per) {
      if (above < k && above + (int)cnt[e] >= k) {
        sh.found[0] = nb - 1 - (tid * per + e);
        sh.found[1] = k - above;
      }
      above += (int)cnt[e];
    }
  }
  __syncthreads();
}

// one warp copies one K row (lanes 0-15) and one V row (lanes 16-31), 16 bytes per lane
__device__ __forceinline__ void copy_kv_row(const SelectParams &p, int b, int kvh, int64_t src_tok, int64_t dst_row,
                                            int lane) {
  const uint16_t *src = (lane < 16 ? p.K : p.V) + (int64_t)b * p.ks.batch_stride + (int64_t)kvh * p.ks.head_stride +
                        src_tok * p.ks.token_stride;
  uint16_t *dst = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                  dst_row * p.cs.token_stride;
  const int piece = (lane & 15) * 8;
  if (SAGEKV_OK_INDEX(p.status, src_tok >= 0 && src_tok < p.N && dst_row >= 0 &&
                                    dst_row < (int64_t)p.S + (int64_t)p.G * p.k_q + p.R + 1))
    st_v4(dst + piece, ld_stream_v4(src + piece));
}

// sink rows, recent rows and the last token: positions known without the scores
__device__ void copy_static_rows(const SelectParams &p, int cta, int n_ctas) {
  const int lane = threadIdx.x & 31;
  const int per_head = p.S + p.R + 1;
  const int items = p.B * p.H_kv * per_head;
  const int n_warps = n_ctas * kSelWarps;
  for (int it = cta * kSelWarps + (threadIdx.x >> 5); it < items; it += n_warps) {
    const int bk = it / per_head, r = it - bk * per_head;
    const int b = bk / p.H_kv, kvh = bk - b * p.H_kv;
    const int64_t src_tok = r < p.S ? r : (int64_t)p.E + r;                 // S + E + (r - S)
    const int64_t dst_row = r < p.S ? r : (int64_t)p.G * p.k_q + r;         // S + G*k_q + (r - S)
    copy_kv_row(p, b, kvh, src_tok, dst_row, lane);
  }
  if (cta == 0 && threadIdx.x == 0) *p.d_step = 0;
}

// Geometry shared by the two paths
struct SelCtx {
  int cs, rank, row, lo, n_local, chunk;
  const float *data;       // this CTA's slice (shared memory when staged, else global)
  int2 *list;              // (slot, position) of the rows this CTA has to gather
  int list_cap;
  unsigned char *scratch;  // union: general-path histograms / fast-path candidate buffers
  int cand_cap;            // candidates per CTA and in total that the fast path can hold
};

// Which 16-byte vectors of the CTA's slice a thread works on: vector (it*8 + u)*512 + tid for iteration it and
// u = 0..7, so that a run of neighbouring scores is spread over as many threads as it has vectors (the bound of
// step 1 is only tight when large scores do not share a thread).  (it, u, tid, element) order is position order.
__device__ __forceinline__ int n_iterations(int n_vec) { return (n_vec + 8 * kSelThreads - 1) / (8 * kSelThreads); }

// The eight vectors of iteration `it` of this thread, all loads issued before any use.  Missing ones read as
// -inf, which is below every threshold and never a maximum.
// kCoherent: the slice was written earlier in this kernel (by this thread), so the read-only path must not be used.
template <bool kStaged, bool kCoherent = false>
__device__ __forceinline__ void load8(const float *data, int n_vec, int it, float4 (&x)[8]) {
  const float ninf = -INFINITY;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int v = (it * 8 + u) * kSelThreads + (int)threadIdx.x;
    x[u] = make_float4(ninf, ninf, ninf, ninf);
    if (v < n_vec) {
      if (kStaged) {
        const uint32_t a = (uint32_t)__cvta_generic_to_shared(data + 4 * v);
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w) : "r"(a));
      } else if (kCoherent) {
        asm volatile("ld.global.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w) : "l"(data + 4 * v) : "memory");
      } else {
        asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w) : "l"(data + 4 * v));
      }
    }
  }
}

template <int kPending>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory");
}

// ---- fast path ----------------------------------------------------------------------------------
// Returns false (for every CTA of the cluster alike) when the prefilter cannot be used for this row;
// nothing has been written to global memory in that case.
// With kStaged the slice arrives through the four cp.async groups the kernel body has issued; every thread
// reads only the vectors it copied itself, so it waits for its own groups and needs no barrier.
// kSketch: the bound comes from the histogram of the row's group maxima that the score step left behind the
// row (hint, loaded by the caller ahead of everything else): steps 1 and 2 are a scan of 512 counts, with no
// pass over the data and no exchange.  It is only a hint (the scores may have changed since): too few or too
// many candidates send the row back here without it.  entered: the cluster's entry barrier has been waited
// for already.
// Returns kFastDone, kFastRetry / kFastRetryEntered (sketch variant: run the other variant; the entry barrier
// has / has not been waited for yet) or kFastGeneral (take the general path).
constexpr int kFastDone = 1, kFastRetry = 0, kFastRetryEntered = -1, kFastGeneral = -2;

struct SketchHint {
  uint32_t cnt;    // count of bin kSketchBins - 1 - threadIdx.x of the row's histogram
  uint32_t bin0;   // key >> kSketchShift of bin 0's lower edge
  uint32_t kmax;   // key of the row maximum
};

// The path is cut in two: fast_candidates (steps 1 to 3: every CTA ends with the same position-sorted candidate
// list, the bound T0 and the row maximum) and fast_decide (steps 4 and 5).  The score step can run the first
// half itself while it normalises a row (kOwnMax: the caller hands in the maximum of the thread's own elements,
// which it has just written to `c.data`) and leave the list behind the row for the select step to start from.
#if defined(SAGEKV_TRACE)
#define SAGEKV_STAMP_AT(tr_, i_) do { if ((tr_) != nullptr && threadIdx.x == 0) (tr_)[i_] = trace_now(); } while (0)
#else
#define SAGEKV_STAMP_AT(tr_, i_) do { } while (0)
#endif
template <bool kStaged, bool kSketch, bool kOwnMax = false>
__device__ int fast_candidates(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c,
                               const SketchHint &hint, bool entered, float own_max, uint32_t &T0_out, uint32_t &kmax_out,
                               int &M_out, int &my_start, unsigned long long *tr = nullptr) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned long long *cand_local = reinterpret_cast<unsigned long long *>(c.scratch);
  unsigned long long *cand_all = cand_local + c.cand_cap;            // 16-byte aligned: cand_cap is even
  unsigned char *flag = reinterpret_cast<unsigned char *>(cand_all + c.cand_cap + 2);
  const int n_vec = c.n_local >> 2;
  const int n_it = n_iterations(n_vec);
  const int tail_i = (n_vec << 2) + tid;                 // the slice's last (n_local % 4) elements: threads 0..2
  const bool has_tail = tail_i < c.n_local;

  uint32_t T0 = 0u, kmax = 0u;      // key of the threshold bound, key of the row maximum
  if (kSketch) {
    // 1', 2'. the bin of the k_q-th largest group maximum, counted from the top of the row's histogram
    const int cnt = (int)hint.cnt;
    int inc = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, off);
      if (lane >= off) inc += n;
    }
    if (lane == 31) sh.scan_tmp[warp] = inc;
    if (tid == 0) { sh.n_border = 0; sh.found[0] = 0; }
    __syncthreads();
    int above = inc - cnt, total = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
      const int t = sh.scan_tmp[w];
      if (w < warp) above += t;
      total += t;
    }
    if (total < 2 * p.k_q || total > kSketchFloats) return kFastRetry;   // (the same answer in every CTA, here and below)
    if (above < p.k_q && above + cnt >= p.k_q) sh.found[0] = kSketchBins - 1 - tid;
    __syncthreads();
    const uint32_t b = (uint32_t)sh.found[0];
    if (b == 0u) return kFastRetry;                      // bin 0 also holds everything below the histogram's range
    T0 = (hint.bin0 + b) << kSketchShift;
    kmax = hint.kmax;
    if (kmax < T0) return kFastRetry;
  } else {
  // 1. thread maxima (float order equals key order, so one fmaxf per element and one key per thread)
  uint32_t tmax = 0;   // 0 is below the key of every number: "no element"
  {
    float fm = -INFINITY;
    if (kOwnMax) {
      fm = own_max;
    } else if (kStaged) {
      const int q = n_it * 2;                            // items (it, u) per copy group
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (g == 0) cp_async_wait<3>();
        if (g == 1) cp_async_wait<2>();
        if (g == 2) cp_async_wait<1>();
        if (g == 3) cp_async_wait<0>();
        for (int k = g * q; k < (g + 1) * q; ++k) {
          const int v = k * kSelThreads + tid;
          if (v < n_vec) {
            const float4 x = *reinterpret_cast<const float4 *>(c.data + 4 * v);
            fm = fmaxf(fmaxf(fm, x.x), fmaxf(x.y, fmaxf(x.z, x.w)));
          }
        }
      }
    } else {
      for (int it = 0; it < n_it; ++it) {
        float4 x[8];
        load8<false>(c.data, n_vec, it, x);
#pragma unroll
        for (int u = 0; u < 8; ++u) fm = fmaxf(fmaxf(fm, x[u].x), fmaxf(x[u].y, fmaxf(x[u].z, x[u].w)));
      }
    }
    if (has_tail && !kOwnMax) fm = fmaxf(fm, c.data[tail_i]);
    if (tid < n_vec || has_tail) tmax = score_key(fm);
  }
  sh.gmax[tid] = tmax;
  {
    const uint32_t wmin = __reduce_min_sync(0xffffffffu, tmax ? tmax : 0xffffffffu);
    const uint32_t wmax = __reduce_max_sync(0xffffffffu, tmax);
    const uint32_t wcnt = __popc(__ballot_sync(0xffffffffu, tmax != 0u));
    if (lane == 0) { sh.red[0][warp] = wmin; sh.red[1][warp] = wmax; sh.red[2][warp] = wcnt; }
  }
  if (tid == 0) sh.n_border = 0;
  __syncthreads();
  if (!entered) cluster.barrier_wait();                  // pairs with the arrive at kernel entry: every peer runs
  if (warp == 0) {   // (min, max, count) of this CTA's maxima, pushed into every peer's gstat table
    uint32_t mn = lane < kSelWarps ? sh.red[0][lane] : 0xffffffffu;
    uint32_t mx = lane < kSelWarps ? sh.red[1][lane] : 0u;
    uint32_t cnt = lane < kSelWarps ? sh.red[2][lane] : 0u;
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (lane < c.cs) {
      uint32_t *gs = cluster.map_shared_rank(&sh.gstat[0][0], lane) + 4 * c.rank;
      gs[0] = mn; gs[1] = mx; gs[2] = cnt;
    }
  }
  cluster.sync();
  SAGEKV_STAMP_AT(tr, 5);

  // 2. all maxima of the cluster -> T0 (512 bins laid over [kmin, kmax])
  uint32_t gm[kMaxCluster];
  uint32_t kmin = 0xffffffffu, n_ne = 0u;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) {
    gm[r] = 0u;
    if (r < c.cs) {
      gm[r] = cluster.map_shared_rank(sh.gmax, r)[tid];
      kmin = min(kmin, sh.gstat[r][0]); kmax = max(kmax, sh.gstat[r][1]); n_ne += sh.gstat[r][2];
    }
  }
  if ((int)n_ne < 2 * p.k_q) return kFastGeneral;       // too few groups for a tight bound (same answer in every CTA)
  const uint32_t diff = kmax ^ kmin;
  const int hi = diff ? 31 - __clz(diff) : -1;           // highest bit in which the maxima differ
  const int shift = hi > 8 ? hi - 8 : 0;                 // (kmax >> shift) - (kmin >> shift) < 512
  const uint32_t base = kmin >> shift;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r)
    if (gm[r] != 0u) atomicAdd(&sh.hist_fast[(gm[r] >> shift) - base], 1u);
  __syncthreads();
  find_bin_from_top(sh.hist_fast, kSelThreads, p.k_q, sh);
  T0 = (base + (uint32_t)sh.found[0]) << shift;
  sh.hist_fast[tid] = 0;                                 // reused in step 4 (barriers in between)
  }
  const float T0f = key_to_score(T0);
  SAGEKV_STAMP_AT(tr, 6);

  // 3. candidates: scores >= T0 as (key, position), packed so that a larger value precedes in
  //    (score desc, position asc), written in position order.  A thread's hits of one iteration are a 32-bit
  //    mask (bit 4u + e: element e of its vector u); a row is the 512 vectors of one (it, u).  Pass A leaves the
  //    hits of every (row, warp) in a byte table, pass B turns the table into offsets and writes.
  if (kSketch && kStaged) cp_async_wait<0>();            // no pass over the slice so far: this thread's copies must have landed
  auto hit_mask = [&](int it) {
    float4 x[8];
    load8<kStaged, kOwnMax>(c.data, n_vec, it, x);
    uint32_t m = 0;
#pragma unroll
    for (int u = 0; u < 8; ++u)
      m |= ((x[u].x >= T0f ? 1u : 0u) | (x[u].y >= T0f ? 2u : 0u) | (x[u].z >= T0f ? 4u : 0u) | (x[u].w >= T0f ? 8u : 0u)) << (4 * u);
    return m;
  };
  // hits per vector u (0..4) as bytes: u = 0..3 in lo, 4..7 in hi
  auto nibble_counts = [](uint32_t m, uint32_t &lo, uint32_t &hi) {
    uint32_t v = m - ((m >> 1) & 0x55555555u);
    v = (v & 0x33333333u) + ((v >> 2) & 0x33333333u);                  // every nibble holds its bit count
    lo = v & 0xffffu; hi = v >> 16;
    lo = (lo | (lo << 8)) & 0x00ff00ffu; lo = (lo | (lo << 4)) & 0x0f0f0f0fu;
    hi = (hi | (hi << 8)) & 0x00ff00ffu; hi = (hi | (hi << 4)) & 0x0f0f0f0fu;
  };
  unsigned char *table = reinterpret_cast<unsigned char *>(cand_all);   // [it][u][warp], free until the lists are exchanged
  uint32_t mask = 0;                                     // of the last iteration (the only one when the slice is short)
  for (int it = 0; it < n_it; ++it) {
    mask = hit_mask(it);
    uint32_t c_lo, c_hi;
    nibble_counts(mask, c_lo, c_hi);
    const uint32_t t_lo = __reduce_add_sync(0xffffffffu, c_lo), t_hi = __reduce_add_sync(0xffffffffu, c_hi);   // <= 128 per byte
    if (lane < 8) table[(it * 8 + lane) * kSelWarps + warp] = (unsigned char)(((lane < 4 ? t_lo : t_hi) >> (8 * (lane & 3))) & 0xffu);
  }
  if (warp == 0) {                                       // the tail elements come last in position order
    const uint32_t hits = __ballot_sync(0xffffffffu, has_tail && c.data[tail_i] >= T0f);
    if (lane == 0) sh.wsum[0] = __popc(hits);
  }
  __syncthreads();
  auto byte_sum = [](uint32_t w) { return (w & 0xffu) + ((w >> 8) & 0xffu) + ((w >> 16) & 0xffu) + (w >> 24); };
  SAGEKV_STAMP_AT(tr, 7);
  int n_loc = sh.wsum[0];
  for (int it = 0; it < n_it; ++it)                      // lane l holds row l/4, warps 4*(l%4) .. +3 of the iteration's table
    n_loc += (int)__reduce_add_sync(0xffffffffu, byte_sum(reinterpret_cast<const uint32_t *>(table)[it * 32 + lane]));
  if (kSketch) cluster.barrier_wait();                   // pairs with the arrive at kernel entry: every peer runs
  if (tid < c.cs) cluster.map_shared_rank(sh.cand_cnt, tid)[c.rank] = n_loc;
  // The score step needs only the peers' counts, not their candidates: it arrives here (release: the count is
  // written) and waits after its own second pass, so that nobody waits for a peer's second pass.
  if (kOwnMax) cluster.barrier_arrive();
  if (n_loc <= c.cand_cap) {
    int run_base = 0;                                    // hits of the iterations before this one
    for (int it = 0; it < n_it; ++it) {
      if (n_it > 1) mask = hit_mask(it);
      const uint32_t word = reinterpret_cast<const uint32_t *>(table)[it * 32 + lane];
      const uint32_t mine = byte_sum(word);
      uint32_t inc = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += n;
      }
      const int it_total = (int)__shfl_sync(0xffffffffu, inc, 31);
      if (__any_sync(0xffffffffu, mask != 0u)) {
        // hits before this warp's part of row u: in the rows before, and in the lower warps of the row
        const uint32_t slot = inc - mine + byte_sum(word & ((1u << (8 * (warp & 3))) - 1u));
        uint32_t rb[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) rb[u] = (uint32_t)run_base + __shfl_sync(0xffffffffu, slot, u * 4 + (warp >> 2));
        // hits in the lower lanes of the warp, all eight rows at once (a row has at most 128 per warp: bytes suffice)
        uint32_t c_lo, c_hi;
        nibble_counts(mask, c_lo, c_hi);
        uint32_t s_lo = c_lo, s_hi = c_hi;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t t_lo = __shfl_up_sync(0xffffffffu, s_lo, off), t_hi = __shfl_up_sync(0xffffffffu, s_hi, off);
          if (lane >= off) { s_lo += t_lo; s_hi += t_hi; }
        }
        const uint32_t x_lo = s_lo - c_lo, x_hi = s_hi - c_hi;          // per byte: no borrow, s >= c
        // as 16-bit pairs (offsets stay below cand_cap < 65536 here)
        const uint32_t b01 = (rb[0] | (rb[1] << 16)) + __byte_perm(x_lo, 0, 0x4140), b23 = (rb[2] | (rb[3] << 16)) + __byte_perm(x_lo, 0, 0x4342);
        const uint32_t b45 = (rb[4] | (rb[5] << 16)) + __byte_perm(x_hi, 0, 0x4140), b67 = (rb[6] | (rb[7] << 16)) + __byte_perm(x_hi, 0, 0x4342);
        const int elem0 = 4 * (it * 8 * kSelThreads + tid);             // slice index of element 0 of vector u = 0
        uint32_t m = mask;
        while (m) {
          const int bit = __ffs(m) - 1;
          m &= m - 1;
          const int u = bit >> 2;
          const uint32_t w = (u & 4) ? ((u & 2) ? b67 : b45) : ((u & 2) ? b23 : b01);
          const int before = (int)((w >> ((u & 1) * 16)) & 0xffffu);
          const int within = __popc(mask & ((1u << bit) - 1u) & (0xfu << (4 * u)));
          const int i = elem0 + u * (4 * kSelThreads) + (bit & 3);
          cand_local[before + within] =
              ((unsigned long long)score_key(c.data[i]) << 32) | (0xffffffffu - (uint32_t)(c.lo + i));
        }
      }
      run_base += it_total;
    }
    if (warp == 0) {
      const bool hit = has_tail && c.data[tail_i] >= T0f;
      const uint32_t hits = __ballot_sync(0xffffffffu, hit);
      if (hit)
        cand_local[n_loc - __popc(hits) + __popc(hits & ((1u << lane) - 1u))] =
            ((unsigned long long)score_key(c.data[tail_i]) << 32) | (0xffffffffu - (uint32_t)(c.lo + tail_i));
    }
  }
  SAGEKV_STAMP_AT(tr, 8);
  if (kOwnMax) {
    __syncthreads();                                     // the CTA's candidates are complete: other threads copy them out
    cluster.barrier_wait();
  } else {
    cluster.sync();
  }
  int start[kMaxCluster + 1];
  bool overflow = false;
  start[0] = 0;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) {
    const int n = r < c.cs ? sh.cand_cnt[r] : 0;
    overflow |= n > c.cand_cap;
    start[r + 1] = start[r] + n;
  }
  const int M = start[kMaxCluster];
  // same counts in every CTA: the whole cluster takes the same way out
  if (overflow || M > c.cand_cap) return kSketch ? kFastRetryEntered : kFastGeneral;
  if (kSketch && M < p.k_q) return kFastRetryEntered;    // the sketch did not describe these scores
  my_start = start[0];
#pragma unroll
  for (int r = 1; r < kMaxCluster; ++r) my_start = r == c.rank ? start[r] : my_start;
  if (kOwnMax) {   // the score step: each CTA writes its own part of the row's list to global memory; no peer's memory is read
    T0_out = T0; kmax_out = kmax; M_out = M;
    return kFastDone;
  }
  // every CTA takes a copy of all candidates, in CTA order: the list is sorted by position
  for (int i = tid; i < M; i += kSelThreads) {
    int r = 0;
#pragma unroll
    for (int q = 1; q < kMaxCluster; ++q) r += i >= start[q] ? 1 : 0;
    cand_all[i] = cluster.map_shared_rank(cand_local, r)[i - start[r]];
  }
  __syncthreads();
  // This CTA is done with its peers' shared memory (the values it read are stored and past a barrier); the
  // arrival is waited for before the kernel ends.  It orders no data, so it need not be a release.
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  T0_out = T0; kmax_out = kmax; M_out = M;
  return kFastDone;
}

// Steps 4 and 5 on a position-sorted candidate list that every CTA of the cluster holds in `cand_all` (at least
// k_q entries, each >= T0; sh.hist_fast zero, sh.n_border zero).  arrived: the CTA has a cluster arrival pending
// (from fast_candidates) that has to be waited for before another path may run.  defer_idx: nothing is written to
// global memory here; the CTA's (slot, position) list in shared memory is all that comes out.
__device__ int fast_decide(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c, uint32_t T0,
                           uint32_t kmax, int M, bool arrived, bool defer_idx = false, unsigned long long *tr = nullptr) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned long long *cand_all = reinterpret_cast<unsigned long long *>(c.scratch) + c.cand_cap;
  unsigned char *flag = reinterpret_cast<unsigned char *>(cand_all + c.cand_cap + 2);

  // 4. which candidates are kept (every CTA decides for all of them).  A 512-bin histogram of the candidate
  //    keys over [T0, row maximum] locates the bin b1 holding the k_q-th largest: higher bins are kept, lower
  //    bins dropped, and the few candidates inside b1 are ranked exactly (key, then position).
  const uint32_t d2 = kmax ^ T0;
  const int hb = d2 ? 31 - __clz(d2) : -1;
  const int shift2 = hb > 8 ? hb - 8 : 0;
  const uint32_t base2 = T0 >> shift2;
  // (a stale sketch may have understated the row maximum: keys above it share the top bin)
  for (int i = tid; i < M; i += kSelThreads)
    atomicAdd(&sh.hist_fast[min((uint32_t)(cand_all[i] >> (32 + shift2)) - base2, (uint32_t)kSelThreads - 1u)], 1u);
  __syncthreads();
  find_bin_from_top(sh.hist_fast, kSelThreads, p.k_q, sh);
  const uint32_t b1 = (uint32_t)sh.found[0];
  const int r1 = sh.found[1];                            // the k_q-th largest is the r1-th largest inside b1
  SAGEKV_STAMP_AT(tr, 3);
  uint32_t *border = sh.gmax;                            // free: every peer is past step 2
  for (int i = tid; i < M; i += kSelThreads) {
    const uint32_t bin = min((uint32_t)(cand_all[i] >> (32 + shift2)) - base2, (uint32_t)kSelThreads - 1u);
    flag[i] = bin > b1 ? 1 : 0;
    if (bin == b1) {
      const int n = atomicAdd(&sh.n_border, 1);
      if (n < kSelThreads) border[n] = (uint32_t)i;
    }
  }
  __syncthreads();
  SAGEKV_STAMP_AT(tr, 4);
  const int nb = sh.n_border;
  if (nb > kSelThreads) {                                // a large group of near-equal scores at the cut
    if (arrived) cluster.barrier_wait();
    return kFastGeneral;
  }
  for (int j = warp; j < nb; j += kSelWarps) {           // one warp per candidate of the border bin
    const uint32_t i = border[j];
    const unsigned long long mine = cand_all[i];
    int before = 0;
    for (int jj = lane; jj < nb; jj += 32) before += cand_all[border[jj]] > mine ? 1 : 0;
    before = __reduce_add_sync(0xffffffffu, before);
    if (lane == 0) flag[i] = before < r1 ? 1 : 0;
  }
  __syncthreads();
  SAGEKV_STAMP_AT(tr, 5);

  // 5. output slots: the list is in position order, so a kept candidate's slot is the number of kept ones
  //    before it.  The CTA writes and gathers an even share of the slots, wherever the rows come from.
  {
    const int per_cta = (p.k_q + c.cs - 1) / c.cs;
    const int slot_lo = min(p.k_q, c.rank * per_cta), slot_hi = min(p.k_q, slot_lo + per_cta);
    const int cpt = (M + kSelThreads - 1) / kSelThreads;   // candidates per thread, a contiguous run
    const int i_lo = min(M, tid * cpt), i_hi = min(M, i_lo + cpt);
    int mine_cnt = 0;
    for (int i = i_lo; i < i_hi; ++i) mine_cnt += flag[i];
    int slot = block_exclusive_scan(mine_cnt, sh.scan_tmp);
    int32_t *idx_row = p.idx + (int64_t)c.row * p.k_q;
    for (int i = i_lo; i < i_hi; ++i) {
      if (flag[i]) {
        if (slot >= slot_lo && slot < slot_hi) {
          const int pos = p.S + (int)(0xffffffffu - (uint32_t)(cand_all[i] & 0xffffffffull));
          (void)SAGEKV_OK_INDEX(p.status, pos >= p.S && pos < p.S + p.E && slot - slot_lo < c.list_cap);
          if (!defer_idx) idx_row[slot] = pos;            // deferred: the caller writes them from the list, later
          c.list[slot - slot_lo] = make_int2(slot, pos);
        }
        ++slot;
      }
    }
    if (tid == 0) sh.list_count = slot_hi - slot_lo;
  }
  __syncthreads();
  return kFastDone;
}

template <bool kStaged, bool kSketch>
__device__ int fast_select(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c,
                           const SketchHint &hint, bool entered) {
  uint32_t T0 = 0u, kmax = 0u;
  int M = 0, my_start = 0;
  const int code = fast_candidates<kStaged, kSketch>(cluster, sh, p, c, hint, entered, 0.f, T0, kmax, M, my_start);
  if (code != kFastDone) return code;
  return fast_decide(cluster, sh, p, c, T0, kmax, M, true);
}

// ---- general path -------------------------------------------------------------------------------
__device__ void general_select(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t(*hist_merged)[kMaxBins] = reinterpret_cast<uint32_t(*)[kMaxBins]>(c.scratch);   // only rank 0's copy is used
  uint32_t *hist_local = reinterpret_cast<uint32_t *>(c.scratch) + 3 * kMaxBins;
  const float *data = c.data;
  const int n_local = c.n_local;
  asm volatile("cp.async.wait_all;" ::: "memory");       // the staged slice: every thread reads all of it here
  __syncthreads();
  for (int i = tid; i < kMaxBins; i += kSelThreads) {
    hist_local[i] = 0;
    hist_merged[0][i] = 0; hist_merged[1][i] = 0; hist_merged[2][i] = 0;
  }
  if (tid == 0) sh.list_count = 0;
  __syncthreads();
  cluster.sync();   // every CTA's merge histograms are zero before any peer adds into them

  // radix select: threshold key and how many keys equal to it are kept
  uint32_t prefix = 0;        // digits found so far, right-aligned
  int k_rem = p.k_q;          // rank of the wanted key among keys matching `prefix`
#pragma unroll
  for (int pass = 0; pass < 3; ++pass) {
    const int bits = pass == 2 ? 10 : 11;               // digits of 11, 11 and 10 bits, most significant first
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nb = 1 << bits;
    const int hi_shift = shift + bits;                  // bits above this digit
    for (int base = 0; base < n_local; base += kSelThreads) {
      const int i = base + tid;
      uint32_t bin = 0xffffffffu;
      if (i < n_local) {
        const uint32_t key = score_key(data[i]);
        if (pass == 0 || (key >> hi_shift) == prefix) bin = (key >> shift) & (nb - 1);
      }
      const uint32_t mn = __reduce_min_sync(0xffffffffu, bin);
      const uint32_t mx = __reduce_max_sync(0xffffffffu, bin);
      if (mn == mx) {                                   // whole warp in one bin (or nothing to count)
        if (lane == 0 && bin != 0xffffffffu) atomicAdd(&hist_local[bin], 32u);
      } else if (bin != 0xffffffffu) {
        atomicAdd(&hist_local[bin], 1u);
      }
    }
    __syncthreads();
    uint32_t *merged0 = cluster.map_shared_rank(&hist_merged[pass][0], 0);
    for (int bin = tid; bin < nb; bin += kSelThreads) {
      const uint32_t v = hist_local[bin];
      if (v) {
        atomicAdd(merged0 + bin, v);
        hist_local[bin] = 0;
      }
    }
    cluster.sync();
    find_bin_from_top(merged0, nb, k_rem, sh);
    prefix = (prefix << bits) | (uint32_t)sh.found[0];
    k_rem = sh.found[1];
    __syncthreads();                                    // found[] is rewritten by the next pass
  }
  const uint32_t tau = prefix;                          // exact key of the k-th largest score
  const int ties_kept = k_rem;                          // >= 1 keys equal to tau are kept, lowest positions first

  // ranks in row order: warp w owns the contiguous range [w*wlen, (w+1)*wlen) of the slice
  const int wlen = (((c.chunk + kSelWarps - 1) / kSelWarps) + 31) & ~31;
  const int wlo = warp * wlen, whi = min(n_local, wlo + wlen);
  int n_gt = 0, n_eq = 0;
  for (int base = wlo; base < whi; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < whi ? score_key(data[i]) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < whi && key > tau));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < whi && key == tau));
  }
  if (lane == 0) { sh.warp_cnt[warp][0] = n_gt; sh.warp_cnt[warp][1] = n_eq; }
  __syncthreads();
  int gt_before = 0, eq_before = 0, cta_gt = 0, cta_eq = 0;
  for (int w = 0; w < kSelWarps; ++w) {
    const int a = sh.warp_cnt[w][0], e = sh.warp_cnt[w][1];
    if (w < warp) { gt_before += a; eq_before += e; }
    cta_gt += a; cta_eq += e;
  }
  if (tid == 0) {
    int *t0 = cluster.map_shared_rank(&sh.totals[0][0], 0);
    t0[2 * c.rank] = cta_gt;
    t0[2 * c.rank + 1] = cta_eq;
  }
  cluster.sync();
  {
    const int *t0 = cluster.map_shared_rank(&sh.totals[0][0], 0);
    for (int r = 0; r < c.rank; ++r) { gt_before += t0[2 * r]; eq_before += t0[2 * r + 1]; }
  }

  int32_t *idx_row = p.idx + (int64_t)c.row * p.k_q;
  for (int base = wlo; base < whi; base += 32) {
    const int i = base + lane;
    const uint32_t key = i < whi ? score_key(data[i]) : 0u;
    const bool gt = i < whi && key > tau, eq = i < whi && key == tau;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const uint32_t below = (1u << lane) - 1u;
    const int g_here = gt_before + __popc(bg & below), e_here = eq_before + __popc(be & below);
    int slot = -1;
    if (gt) slot = g_here + min(e_here, ties_kept);
    else if (eq && e_here < ties_kept) slot = g_here + e_here;
    if (slot >= 0) {
      const int pos = p.S + c.lo + i;
      if (SAGEKV_OK_INDEX(p.status, slot < p.k_q && pos < p.S + p.E)) idx_row[slot] = pos;
      const int n = atomicAdd(&sh.list_count, 1);
      if (n < c.list_cap) c.list[n] = make_int2(slot, pos);
    }
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  __syncthreads();
  cluster.sync();   // no CTA moves on (and may exit) while a peer still reads its shared memory
}

// kAhead: the instance for launches that start from a trusted candidate list with the dependency wait put off
// (eight rows in flight per warp, which the other instance has no registers for).
template <bool kAhead>
__global__ void __launch_bounds__(kSelThreads, 2) select_compact_kernel(const SelectParams p, int n_rows, int chunk,
                                                                      int resident, int list_cap, int cand_cap,
                                                                      int try_fast, int64_t sketch_off, int64_t list_off) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int cid = blockIdx.x / cs;
  SAGEKV_TRACE_BEGIN
  SAGEKV_STAMP(0);
  // Programmatic dependent launch (sagekv_set_select_overlap): the kernel may have been scheduled while its
  // predecessor on the stream was still running.  Mode 1 reads and writes nothing before the predecessor is
  // complete (a request to bring the candidate list into L2 changes nothing a program can observe).  Mode 2 (the
  // caller vouches that the predecessor writes none of this call's inputs) puts the wait off until the first
  // write: selection and the first round of row loads run ahead of it, on the candidate-list path.
  bool waited = p.pdl == 0;
  if (p.pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.pdl == 1 || (p.pdl == 2 && (list_off < 0 || cid >= n_rows))) {
    if (list_off >= 0 && cid < n_rows) {
      const char *lines = reinterpret_cast<const char *>(p.scores + (int64_t)cid * p.row_stride + list_off);
      const int n_lines = (kListTagWords * 4 + cand_cap * 8 + 127) >> 7;
      const int mine = rank + (int)threadIdx.x * cs;
      if (mine < n_lines) asm volatile("prefetch.global.L2 [%0];" ::"l"(lines + (int64_t)mine * 128));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    waited = true;
  }
  SAGEKV_STAMP(1);
  if (cid >= n_rows) {   // whole cluster takes this branch together; it touches no peer's memory
    copy_static_rows(p, (cid - n_rows) * cs + rank, (gridDim.x / cs - n_rows) * cs);
    return;
  }

  cluster.barrier_arrive();   // completed below: every CTA of the cluster runs before anyone writes into a peer
  SelShared &sh = *reinterpret_cast<SelShared *>(smem_raw);
  float *staged = reinterpret_cast<float *>(smem_raw + sizeof(SelShared));
  unsigned char *after = smem_raw + sizeof(SelShared) + (resident ? (size_t)chunk * sizeof(float) : 0);
  SelCtx c;
  c.cs = cs; c.rank = rank; c.row = cid; c.chunk = chunk;
  c.lo = rank * chunk;
  c.n_local = max(0, min(p.E - c.lo, chunk));
  c.list = nullptr;           // placed by the path that runs
  c.list_cap = list_cap;
  c.scratch = after;          // 16-byte aligned
  c.cand_cap = cand_cap;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = c.row / p.H_q, h = c.row - b * p.H_q;
  const int kvh = h / p.G, j = h - kvh * p.G;
  const float *grow = p.scores + (int64_t)c.row * p.row_stride + c.lo;   // 16-byte aligned: chunk % 4 == 0
  (void)SAGEKV_OK_INDEX(p.status, c.row < p.B * p.H_q && (int64_t)c.lo + c.n_local <= p.row_stride && c.lo + c.n_local <= p.E &&
                                      (sketch_off < 0 || sketch_off + kSketchBins + 4 <= p.row_stride));

  sh.hist_fast[tid] = 0;
  c.data = grow;
  // the histogram of the row's group maxima, if the score step left it behind the row: requested first
  SketchHint hint = {0u, 0u, 0u};
  uint32_t tag0 = 0u, tag1 = 0u;
  if (sketch_off >= 0) {
    const uint32_t *sk = reinterpret_cast<const uint32_t *>(p.scores + (int64_t)c.row * p.row_stride + sketch_off);
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(hint.cnt) : "l"(sk + kSketchBins - 1 - tid));
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(tag0) : "l"(sk + kSketchBins));
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(tag1) : "l"(sk + kSketchBins + 1));
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(hint.bin0) : "l"(sk + kSketchBins + 2));
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(hint.kmax) : "l"(sk + kSketchBins + 3));
  }
  // the candidate list of the score step, if the caller vouches for it: its tag words and this thread's share of
  // the entries (as many as the list can have; which of them count is known once the tag is here)
  constexpr int kListRegs = 7;                            // 7 x 512 entries: the longest list there can be (k_q = 2048)
  uint32_t lt[6] = {0u, 0u, 0u, 0u, 0u, 0u};
  unsigned long long le[kListRegs] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
  if (list_off >= 0) {
    const uint32_t *tg = reinterpret_cast<const uint32_t *>(p.scores + (int64_t)c.row * p.row_stride + list_off);
#pragma unroll
    for (int i = 0; i < 6; ++i) asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(lt[i]) : "l"(tg + i));
    const unsigned long long *le_src = reinterpret_cast<const unsigned long long *>(tg + kListTagWords);
#pragma unroll
    for (int i = 0; i < kListRegs; ++i)
      if (tid + i * kSelThreads < cand_cap) asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(le[i]) : "l"(le_src + tid + i * kSelThreads));
  }
  if (!resident && sketch_off >= 0 && tid == 0 && c.n_local >= 4) {
    // not staged: ask for the slice to be brought into L2 while the threshold bound is worked out from the hint
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(grow), "r"((uint32_t)(c.n_local >> 2) * 16u) : "memory");
  }
  if (resident) {
    // four copy groups per thread, over exactly the vectors the thread works on later (see n_iterations)
    const int n_vec = c.n_local >> 2;
    const int q = n_iterations(n_vec) * 2;
    for (int g = 0; g < 4; ++g) {
      for (int k = g * q; k < (g + 1) * q; ++k) {
        const int v = k * kSelThreads + tid;
        if (v < n_vec) {
          const uint32_t dst = (uint32_t)__cvta_generic_to_shared(staged + 4 * v);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(grow + 4 * v) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const int tail_i = (n_vec << 2) + tid;
    if (tail_i < c.n_local) staged[tail_i] = grow[tail_i];
    c.data = staged;
  }

  // The gather list follows the buffers of the path that runs (see select_smem_bytes).
  bool done = false, exit_wait = false;   // exit_wait: a cluster arrival of the prefilter is still to be waited for
  bool idx_deferred = false;              // the selection wrote no indices: they follow from the gather lists
  if (try_fast) {
    c.list = reinterpret_cast<int2 *>(c.scratch + (size_t)cand_cap * 16 + 16 + (((size_t)cand_cap + 15) & ~(size_t)15));
    int code = kFastRetry;
    if (list_off >= 0 && lt[0] == kListMagic && lt[1] == (uint32_t)p.E && lt[2] == (uint32_t)p.k_q && (int)lt[3] >= p.k_q &&
        (int)lt[3] <= cand_cap && cand_cap <= kListRegs * kSelThreads) {   // the same words in every CTA of the row
      // start from the score step's list: no pass over the row, no exchange between the CTAs
      const int M = (int)lt[3];
      unsigned long long *cand_all = reinterpret_cast<unsigned long long *>(c.scratch) + cand_cap;
#pragma unroll
      for (int i = 0; i < kListRegs; ++i)
        if (tid + i * kSelThreads < M) cand_all[tid + i * kSelThreads] = le[i];
      if (tid == 0) sh.n_border = 0;
      cluster.barrier_wait();                              // the arrive at kernel entry; no peer's memory is touched on this path
      __syncthreads();
      SAGEKV_STAMP(2);
#if defined(SAGEKV_TRACE)
      code = fast_decide(cluster, sh, p, c, lt[4], lt[5], M, false, !waited, trace_t);
#else
      code = fast_decide(cluster, sh, p, c, lt[4], lt[5], M, false, !waited);
#endif
      SAGEKV_STAMP(6);
      idx_deferred = !waited && code == kFastDone;
      if (code == kFastGeneral) {                          // (a large group of equal scores at the cut)
        if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
        c.list = reinterpret_cast<int2 *>(c.scratch + kGeneralScratch);
        general_select(cluster, sh, p, c);
        code = kFastDone;
      }
      done = true;
    }
    if (!done && !waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }   // the other paths write as they go
    if (!done && sketch_off >= 0 && tag0 == kSketchMagic && tag1 == (uint32_t)p.E)   // the same words in every CTA of the row
      code = resident ? fast_select<true, true>(cluster, sh, p, c, hint, false)
                      : fast_select<false, true>(cluster, sh, p, c, hint, false);
    if (!done) {
      if (code == kFastRetry || code == kFastRetryEntered)
        code = resident ? fast_select<true, false>(cluster, sh, p, c, hint, code == kFastRetryEntered)
                        : fast_select<false, false>(cluster, sh, p, c, hint, code == kFastRetryEntered);
      done = code == kFastDone;
      exit_wait = done;
    }
  } else {
    cluster.barrier_wait();
  }
  if (!done) {
    if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
    c.list = reinterpret_cast<int2 *>(c.scratch + kGeneralScratch);
    general_select(cluster, sh, p, c);
  }

  // gather the rows on this CTA's list into head j's segment of the reduced cache: a warp moves eight rows at a
  // time (K in lanes 0-15, V in lanes 16-31), all loads issued before the stores
  const bool gather = p.Kc != nullptr;                   // null: the caller wants the indices only
  int32_t *idx_row = p.idx + (int64_t)c.row * p.k_q;
  const int n_list_all = min(sh.list_count, list_cap);
  const int n_list = gather ? n_list_all : 0;
  const uint16_t *src_base = (lane < 16 ? p.K : p.V) + (int64_t)b * p.ks.batch_stride + (int64_t)kvh * p.ks.head_stride +
                             (lane & 15) * 8;
  uint16_t *dst_base = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                       ((int64_t)p.S + (int64_t)j * p.k_q) * p.cs.token_stride + (lane & 15) * 8;
  // The sink, recent and last rows of the KV head (positions known without the scores) are shared out over the
  // warps of the head's G clusters, at most one row per warp per round, loaded together with the first batch.
  const int n_static = gather ? p.S + p.R + 1 : 0;
  const int static_stride = p.G * cs * kSelWarps;
  int sr = (j * cs + rank) * kSelWarps + warp;           // this warp's first static row
  constexpr int kRows = kAhead ? 8 : 4;                    // rows a warp has in flight: all loads issued before the stores
  const int per_warp = n_list > kSelWarps * 4 ? kRows : 4;   // a short list is spread over all the warps
  for (int e0 = warp * per_warp; e0 < n_list || sr < n_static; e0 += kSelWarps * per_warp) {
    uint4 v[kRows], vs = make_uint4(0u, 0u, 0u, 0u);
    const bool has_static = sr < n_static;
    if (has_static) {
      const int64_t src_tok = sr < p.S ? sr : (int64_t)p.E + sr;                 // S + E + (sr - S)
      (void)SAGEKV_OK_INDEX(p.status, src_tok >= 0 && src_tok < p.N);
      vs = ld_stream_v4(src_base + src_tok * p.ks.token_stride);
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      if (u < per_warp && e0 + u < n_list) {
        int pos = c.list[e0 + u].y;
        if (!SAGEKV_OK_INDEX(p.status, pos >= p.S && pos < p.S + p.E)) pos = p.S;
        v[u] = ld_stream_v4(src_base + (int64_t)pos * p.ks.token_stride);
      }
    }
    if (!waited) {                                         // the first write of this warp
      asm volatile("griddepcontrol.wait;" ::: "memory");
      waited = true;
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      if (u < per_warp && e0 + u < n_list) {
        int slot = c.list[e0 + u].x;
        if (!SAGEKV_OK_INDEX(p.status, slot >= 0 && slot < p.k_q)) slot = 0;
        st_v4(dst_base + (int64_t)slot * p.cs.token_stride, v[u]);
      }
    }
    if (has_static) {
      // dst_base points at the head's segment S + j*k_q; static rows are addressed from row 0 of the KV head
      const int64_t dst_row = sr < p.S ? sr : (int64_t)p.G * p.k_q + sr;         // S + G*k_q + (sr - S)
      st_v4(dst_base + (dst_row - ((int64_t)p.S + (int64_t)j * p.k_q)) * p.cs.token_stride, vs);
      sr += static_stride;
    }
  }
  if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");   // a warp without a round of the loop
  if (idx_deferred)                                        // every thread is here, and past the wait
    for (int i = tid; i < n_list_all; i += kSelThreads) {
      const int2 sp = c.list[i];
      if (SAGEKV_OK_INDEX(p.status, sp.x >= 0 && sp.x < p.k_q)) idx_row[sp.x] = sp.y;
    }
  SAGEKV_STAMP(7);
  if (cid == 0 && rank == 0 && tid == 0 && p.d_step != nullptr) *p.d_step = 0;
  SAGEKV_STAMP(8);
  SAGEKV_STAMP(9);
  SAGEKV_TRACE_END(p.idx);
  if (exit_wait) cluster.barrier_wait();   // prefilter path: a peer may still have been copying this CTA's candidates
}

// ---- second pass of the score step in hint mode 2 -----------------------------------------------------------
// One cluster of 8 CTAs per score row.  Each CTA normalises its slice of the row in place (logits in log2 units
// -> probabilities, exactly as score_finalize_kernel does), keeps the slice in shared memory when it fits, and
// then the cluster runs the first half of the select step's prefilter on it (fast_candidates, the thread maxima
// coming from the normalisation loop).  Every CTA writes its part of the position-sorted candidate list behind
// the row, CTA 0 the tag (layout: common.cuh); M = 0 when the prefilter did not apply.
__global__ void __launch_bounds__(kSelThreads, 2) score_finalize_candidates_kernel(const ScoreParams sp, const SelectParams p,
                                                                                 int chunk, int resident, int cand_cap,
                                                                                 int64_t list_off) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int row = blockIdx.x / cs;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  cluster.barrier_arrive();   // completed in fast_candidates: every CTA of the cluster runs before anyone writes into a peer
  SAGEKV_TRACE_BEGIN
  SAGEKV_STAMP(0);
  SelShared &sh = *reinterpret_cast<SelShared *>(smem_raw);
  float *staged = reinterpret_cast<float *>(smem_raw + sizeof(SelShared));
  SelCtx c;
  c.cs = cs; c.rank = rank; c.row = row; c.chunk = chunk;
  c.lo = rank * chunk;
  c.n_local = max(0, min(p.E - c.lo, chunk));
  c.list = nullptr;
  c.list_cap = 0;
  c.scratch = smem_raw + sizeof(SelShared) + (resident ? (size_t)chunk * sizeof(float) : 0);
  c.cand_cap = cand_cap;
  sh.hist_fast[tid] = 0;

  // (max, sum) of the row from the first pass's partials
  float *sm_m = reinterpret_cast<float *>(&sh.red[0][0]), *sm_l = reinterpret_cast<float *>(&sh.red[1][0]);   // free until the prefilter
  float m = -INFINITY, l = 0.f;
  const float2 *part = sp.partials + (int64_t)row * sp.n_chunks;
  for (int i = tid; i < sp.n_chunks; i += kSelThreads) {
    const float2 v = part[i];
    merge_ml(m, l, v.x, v.y);
  }
  {   // the maximum first, then the sums rescaled to it: independent exponentials instead of a chain of merges
    float wm = m;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
    l = wm == -INFINITY ? 0.f : l * fast_exp2(m - wm);
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if (lane == 0) { sm_m[warp] = wm; sm_l[warp] = l; }
    __syncthreads();
    float mm[kSelWarps], ll[kSelWarps];
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) { mm[w] = sm_m[w]; ll[w] = sm_l[w]; }
    m = mm[0];
#pragma unroll
    for (int w = 1; w < kSelWarps; ++w) m = fmaxf(m, mm[w]);
    l = 0.f;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) l += mm[w] == -INFINITY ? 0.f : ll[w] * fast_exp2(mm[w] - m);
  }
  const float inv = 1.f / l;
  __syncthreads();   // the prefilter reuses the words the pairs were exchanged in
  SAGEKV_STAMP(1);

  // normalise this thread's vectors (the ones it works on in the prefilter: see n_iterations)
  float *grow = sp.scores + (int64_t)row * sp.row_stride + c.lo;
  const int n_vec = c.n_local >> 2, n_it = n_iterations(n_vec);
  float fm = -INFINITY;
  for (int it = 0; it < n_it; ++it) {
    float4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v = (it * 8 + u) * kSelThreads + tid;
      if (v < n_vec) x[u] = *reinterpret_cast<const float4 *>(grow + 4 * v);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v = (it * 8 + u) * kSelThreads + tid;
      if (v < n_vec) {
        x[u].x = fast_exp2(x[u].x - m) * inv; x[u].y = fast_exp2(x[u].y - m) * inv;
        x[u].z = fast_exp2(x[u].z - m) * inv; x[u].w = fast_exp2(x[u].w - m) * inv;
        *reinterpret_cast<float4 *>(grow + 4 * v) = x[u];
        if (resident) *reinterpret_cast<float4 *>(staged + 4 * v) = x[u];
        fm = fmaxf(fmaxf(fm, x[u].x), fmaxf(x[u].y, fmaxf(x[u].z, x[u].w)));
      }
    }
  }
  const int tail_i = (n_vec << 2) + tid;
  if (tail_i < c.n_local) {
    const float y = fast_exp2(grow[tail_i] - m) * inv;
    grow[tail_i] = y;
    if (resident) staged[tail_i] = y;
    fm = fmaxf(fm, y);
  }
  c.data = resident ? staged : grow;
  SAGEKV_STAMP_AFTER(2, fm);

  SketchHint none = {0u, 0u, 0u};
  uint32_t T0 = 0u, kmax = 0u;
  int M = 0, my_start = 0;
#if defined(SAGEKV_TRACE)
  unsigned long long *tr = trace_t;
#else
  unsigned long long *tr = nullptr;
#endif
  const int code = resident ? fast_candidates<true, false, true>(cluster, sh, p, c, none, false, fm, T0, kmax, M, my_start, tr)
                            : fast_candidates<false, false, true>(cluster, sh, p, c, none, false, fm, T0, kmax, M, my_start, tr);
  SAGEKV_STAMP(3);
  uint32_t *tag = reinterpret_cast<uint32_t *>(sp.scores + (int64_t)row * sp.row_stride + list_off);
  if (code == kFastDone) {   // the CTAs' lists, one behind the other, are the row's list in position order
    const unsigned long long *cand_local = reinterpret_cast<const unsigned long long *>(c.scratch);
    unsigned long long *dst = reinterpret_cast<unsigned long long *>(tag + kListTagWords) + my_start;
    const int n_mine = sh.cand_cnt[rank];
    for (int i = tid; i < n_mine; i += kSelThreads) dst[i] = cand_local[i];
  } else {
    M = 0;
  }
  if (rank == 0 && tid == 0) {
    tag[0] = kListMagic; tag[1] = (uint32_t)p.E; tag[2] = (uint32_t)p.k_q; tag[3] = (uint32_t)M;
    tag[4] = T0; tag[5] = kmax; tag[6] = 0u; tag[7] = 0u;
  }
  SAGEKV_STAMP(4);
  SAGEKV_STAMP(9);
  SAGEKV_TRACE_END(sp.scores);
}

static size_t select_smem_bytes(int chunk, int list_cap, int cand_cap, int share, bool resident) {
  // fast path: candidates (own, all), one keep flag per candidate, the gather list of the CTA's share of the slots;
  // general path: the histograms, then the gather list (as long as the slice, or k_q)
  size_t scratch = (size_t)cand_cap * (8 + 8) + 16 + (((size_t)cand_cap + 15) & ~(size_t)15) + (size_t)share * sizeof(int2);
  const size_t general = (size_t)kGeneralScratch + (size_t)list_cap * sizeof(int2);
  if (scratch < general) scratch = general;
  scratch = (scratch + 15) & ~(size_t)15;
  return sizeof(SelShared) + scratch + (resident ? (size_t)chunk * sizeof(float) : 0);
}

cudaError_t select_compact_setup() {
  cudaError_t e = cudaFuncSetAttribute(select_compact_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelSmemLimit);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(select_compact_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelSmemLimit);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_finalize_candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelSmemLimit);
}

cudaError_t launch_score_finalize_candidates(const ScoreParams &sp, cudaStream_t stream) {
  const int rows = sp.B * sp.H_q, cs = kMaxCluster;
  int chunk = (sp.E + cs - 1) / cs;
  chunk = (chunk + 3) & ~3;
  const int cand_cap = list_cand_cap(sp.list_k_q);
  // two CTAs per SM keep every row's cluster resident at once: stage the slice only while two such CTAs fit
  const bool resident = select_smem_bytes(chunk, 1, cand_cap, 0, true) <= (size_t)kSelSmemLimit / 2;
  const size_t smem = select_smem_bytes(chunk, 1, cand_cap, 0, resident);
  SelectParams p = {};
  p.E = sp.E;
  p.k_q = sp.list_k_q;
  p.status = sp.status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(rows * cs), 1, 1);
  cfg.blockDim = dim3(kSelThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, score_finalize_candidates_kernel, sp, p, chunk, (int)resident, cand_cap, sketch_offset(sp.E));
}

cudaError_t launch_select_compact(const SelectParams &p, int n_sm, cudaStream_t stream) {
  const bool select = p.k_q > 0 && p.E > 0;
  const int n_rows = select ? p.B * p.H_q : 0;
  // The rows may carry the group maxima of the score step (see common.cuh): then the threshold bound costs no
  // pass over the data, the slice is read straight from global memory (no staging: it is needed once), and with
  // many rows smaller clusters pay, because two CTAs per SM times the SM count is all that runs at once.
  const bool list = select && p.list && list_applies(p.E, p.k_q, p.row_stride);
  const bool sketch = list || (select && p.sketch && sketch_fits(p.E, p.row_stride));   // both read the row unstaged, if at all
  // cluster size: slices of at least 2048 scores, at most 8 CTAs (the portable limit)
  int cs = 1;
  // From a candidate list nothing but the gather scales with the cluster: a CTA takes up to 128 rows (one round of
  // its 16 warps), and small launches leave room for the next launch's CTAs to run ahead (sagekv_set_select_overlap).
  const bool ahead = list && p.pdl == 2;
  while (cs < kMaxCluster && (int64_t)cs * 2048 < p.E &&
         (ahead ? (p.k_q + cs - 1) / cs > 128 : (!sketch || (int64_t)n_rows * cs * 2 <= 2 * (int64_t)n_sm))) cs <<= 1;
  int chunk = (p.E + cs - 1) / cs;
  chunk = (chunk + 3) & ~3;
  if (chunk < 4) chunk = 4;
  const int list_cap = chunk < p.k_q ? chunk : (p.k_q > 0 ? p.k_q : 1);
  // the prefilter needs at least 2*k_q thread maxima; its buffers hold 1.5*k_q + 256 candidates
  // (and its per-row hit table, kept where the candidate copies go later, holds 16 iterations of 4096 vectors)
  const int try_fast = select && chunk <= 16 * 8 * kSelThreads * 4 &&
                       (2 * (int64_t)p.k_q <= (int64_t)cs * kSelThreads || (sketch && 2 * p.k_q <= kSketchFloats));
  const int cand_cap = try_fast ? (p.k_q + p.k_q / 2 + 256) & ~1 : 0;
  const int share = (p.k_q + cs - 1) / cs;              // slots a CTA writes and gathers on the fast path
  const bool resident = !sketch && select_smem_bytes(chunk, list_cap, cand_cap, share, true) <= (size_t)kSelSmemLimit;
  const size_t smem = select_smem_bytes(chunk, list_cap, cand_cap, share, resident);

  // Without a selection (k_q = 0 or an empty eviction region) there are no row clusters: plain copy clusters
  // move the sink, recent and last rows.  Otherwise the row clusters copy them along with the kept rows.
  int copy_clusters = 0;
  if (!select) {
    const int static_items = p.B * p.H_kv * (p.S + p.R + 1);
    copy_clusters = (static_items + cs * kSelWarps * 2 - 1) / (cs * kSelWarps * 2);
    if (copy_clusters < 1) copy_clusters = 1;
    const int cap = (n_sm + cs - 1) / cs;
    if (copy_clusters > cap) copy_clusters = cap;
  }

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_rows + copy_clusters) * cs), 1, 1);
  cfg.blockDim = dim3(kSelThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  // Only launches that start from a candidate list are short enough to gain from early scheduling: the others
  // pass over the row, and successors scheduled early take bandwidth and SM room from that.
  SelectParams pl = p;
  if (!list) pl.pdl = 0;
  cfg.numAttrs = pl.pdl ? 2 : 1;
  const int64_t sketch_off = try_fast && sketch && !list ? sketch_offset(p.E) : (int64_t)-1;
  const int64_t list_off = try_fast && list ? sketch_offset(p.E) : (int64_t)-1;
  return ahead ? cudaLaunchKernelEx(&cfg, select_compact_kernel<true>, pl, n_rows, chunk, (int)resident, list_cap, cand_cap,
                                    try_fast, sketch_off, list_off)
               : cudaLaunchKernelEx(&cfg, select_compact_kernel<false>, pl, n_rows, chunk, (int)resident, list_cap, cand_cap,
                                    try_fast, sketch_off, list_off);
}

}  // namespace sagekv

SAGEKV_TRACE_READER(sagekv_trace_read_select)
