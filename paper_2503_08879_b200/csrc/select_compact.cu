// Step 2 (second half) and Step 3: per-query-head top-k over the score rows, then the gather that
// builds the reduced cache  C = Concat(sink, selected, recent, last).
//
// One thread-block cluster (up to 8 CTAs) owns one score row.  Each CTA stages its contiguous slice of
// the row in shared memory once (cp.async, 16 bytes per request); every later step works on that copy, so
// the scores cross the memory system a single time.
//
// Fast path (k_q small against the row, the normal case): a prefilter instead of a full radix select.
//   1. every thread takes the maximum of its elements; the cluster's thread maxima are exchanged over
//      distributed shared memory.  The k_q-th largest of these maxima is a lower bound T0 of the k_q-th
//      largest score (k_q distinct elements are >= it), and it is tight: about k_q * (1 + few %) scores
//      are >= T0.  T0 is taken as the lower edge of the histogram bin (2048 bins laid over the actual
//      range of the maxima) in which that maximum falls.
//   2. scores >= T0 become candidates (order-preserving key, position); the lists are exchanged.
//   3. a histogram of all candidate keys finds the bin of the k_q-th largest; own candidates above it are
//      kept, the few inside it are ranked exactly, with the position as tie-break (lowest positions win).
//   4. kept counts are exchanged; slot = kept in lower CTAs + kept before it in this CTA: ascending order.
// General path (k_q large, tiny rows, or more candidates than the buffers hold, e.g. a row of equal
// scores): three-digit radix select (11 + 11 + 10 bits) with histograms merged in CTA 0's shared memory by
// distributed-shared-memory atomics, then a ballot/popcount ranking in row order.
// Either way the CTA that owns a kept element copies its K and V rows into the head's segment of the
// reduced cache, and a few extra clusters copy the sink, recent and last rows.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace sagekv {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxCluster = 8;
constexpr int kMaxBins = 2048;
constexpr int kSelSmemLimit = 200 * 1024;
constexpr int kGeneralScratch = 4 * kMaxBins * 4;   // general path: three merged histograms and the local one

struct SelShared {
  uint32_t hist_fast[kSelThreads];     // fast path: histogram of the thread maxima
  uint32_t gmax[kSelThreads];          // thread maxima of this CTA, read by the peers
  uint32_t red[3][kSelWarps];
  uint32_t gstat[kMaxCluster][4];      // (min, max, count) of every CTA's non-empty thread maxima, pushed by the peers
  int totals[kMaxCluster][2];          // general path: (kept-larger, equal-to-threshold) per CTA; rank 0's copy
  int cand_cnt[kMaxCluster];           // fast path: candidates per CTA, pushed by each CTA to every peer
  int sel_cnt[kMaxCluster];            // fast path: kept per CTA
  int warp_cnt[kSelWarps][2];
  int scan_tmp[kSelWarps];
  int found[2];
  int list_count;
  int n_cand_local;
  int n_sel_local;
  int pad_[3];
};
static_assert(sizeof(SelShared) % 16 == 0, "staged scores must stay 16-byte aligned");

__device__ __forceinline__ uint32_t score_key(float x) {
  const uint32_t u = __float_as_uint(x + 0.0f);         // -0 becomes +0: the two compare equal as numbers
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);   // larger float <=> larger unsigned key
}

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
  int base = 0;
  for (int w = 0; w < warp; ++w) base += tmp[w];
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

// Eight float4 of this thread's elements (vector indices v0 + tid + u*512), all loads issued before any use.
// Missing ones (index >= n_vec) read as -inf, which is below every threshold and never a maximum.
template <bool kStaged>
__device__ __forceinline__ void load8(const float *data, int v0, int n_vec, float4 (&x)[8]) {
  const float ninf = -INFINITY;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int v = v0 + (int)threadIdx.x + u * kSelThreads;
    x[u] = make_float4(ninf, ninf, ninf, ninf);
    if (v < n_vec) {
      if (kStaged) {
        const uint32_t a = (uint32_t)__cvta_generic_to_shared(data + 4 * v);
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w) : "r"(a));
      } else {
        asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(x[u].x), "=f"(x[u].y), "=f"(x[u].z), "=f"(x[u].w) : "l"(data + 4 * v));
      }
    }
  }
}

// ---- fast path ----------------------------------------------------------------------------------
// Returns false (for every CTA of the cluster alike) when the prefilter cannot be used for this row;
// nothing has been written to global memory in that case.
template <bool kStaged>
__device__ bool fast_select(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned long long *cand_local = reinterpret_cast<unsigned long long *>(c.scratch);
  unsigned long long *cand_all = cand_local + c.cand_cap;            // 16-byte aligned: cand_cap is even
  int *sel_pos = reinterpret_cast<int *>(cand_all + c.cand_cap + 2);
  const int n_vec = c.n_local >> 2;

  // 1. thread maxima (float order equals key order, so one fmaxf per element and one key per thread)
  uint32_t tmax = 0;   // 0 is below the key of every number: "no element"
  {
    float fm = -INFINITY;
    for (int v0 = 0; v0 < n_vec; v0 += 8 * kSelThreads) {
      float4 x[8];
      load8<kStaged>(c.data, v0, n_vec, x);
#pragma unroll
      for (int u = 0; u < 8; ++u) fm = fmaxf(fmaxf(fm, x[u].x), fmaxf(x[u].y, fmaxf(x[u].z, x[u].w)));
    }
    bool any = tid < n_vec;
    for (int i = (n_vec << 2) + tid; i < c.n_local; i += kSelThreads) { fm = fmaxf(fm, c.data[i]); any = true; }
    if (any) tmax = score_key(fm);
  }
  sh.gmax[tid] = tmax;
  {
    const uint32_t wmin = __reduce_min_sync(0xffffffffu, tmax ? tmax : 0xffffffffu);
    const uint32_t wmax = __reduce_max_sync(0xffffffffu, tmax);
    const uint32_t wcnt = __popc(__ballot_sync(0xffffffffu, tmax != 0u));
    if (lane == 0) { sh.red[0][warp] = wmin; sh.red[1][warp] = wmax; sh.red[2][warp] = wcnt; }
  }
  if (tid == 0) { sh.n_cand_local = 0; sh.n_sel_local = 0; }
  __syncthreads();
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

  // 2. all maxima of the cluster -> T0 (512 bins laid over [kmin, kmax])
  uint32_t gm[kMaxCluster];
  uint32_t kmin = 0xffffffffu, kmax = 0u, n_ne = 0u;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) {
    gm[r] = 0u;
    if (r < c.cs) {
      gm[r] = cluster.map_shared_rank(sh.gmax, r)[tid];
      kmin = min(kmin, sh.gstat[r][0]); kmax = max(kmax, sh.gstat[r][1]); n_ne += sh.gstat[r][2];
    }
  }
  if ((int)n_ne < 2 * p.k_q) return false;              // too few groups for a tight bound (same answer in every CTA)
  const uint32_t diff = kmax ^ kmin;
  const int hi = diff ? 31 - __clz(diff) : -1;           // highest bit in which the maxima differ
  const int shift = hi > 8 ? hi - 8 : 0;                 // (kmax >> shift) - (kmin >> shift) < 512
  const uint32_t base = kmin >> shift;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r)
    if (gm[r] != 0u) atomicAdd(&sh.hist_fast[(gm[r] >> shift) - base], 1u);
  __syncthreads();
  find_bin_from_top(sh.hist_fast, kSelThreads, p.k_q, sh);
  const uint32_t T0 = (base + (uint32_t)sh.found[0]) << shift;
  const float T0f = key_to_score(T0);
  sh.hist_fast[tid] = 0;                                 // reused in step 4 (barriers in between)

  // 3. candidates: (key, position) packed so that a larger value precedes in (score desc, position asc)
  for (int v0 = 0; v0 < n_vec; v0 += 8 * kSelThreads) {
    float4 x[8];
    load8<kStaged>(c.data, v0, n_vec, x);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (x[u].x >= T0f || x[u].y >= T0f || x[u].z >= T0f || x[u].w >= T0f) {
        const float xs[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
        const int v = v0 + tid + u * kSelThreads;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (xs[e] >= T0f) {
            const int n = atomicAdd(&sh.n_cand_local, 1);
            if (n < c.cand_cap)
              cand_local[n] = ((unsigned long long)score_key(xs[e]) << 32) | (0xffffffffu - (uint32_t)(c.lo + 4 * v + e));
          }
        }
      }
    }
  }
  for (int i = (n_vec << 2) + tid; i < c.n_local; i += kSelThreads) {
    const float x = c.data[i];
    if (x >= T0f) {
      const int n = atomicAdd(&sh.n_cand_local, 1);
      if (n < c.cand_cap)
        cand_local[n] = ((unsigned long long)score_key(x) << 32) | (0xffffffffu - (uint32_t)(c.lo + i));
    }
  }
  __syncthreads();
  const int n_loc = sh.n_cand_local;
  if (tid < c.cs) cluster.map_shared_rank(sh.cand_cnt, tid)[c.rank] = n_loc;
  cluster.sync();
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
  if (overflow || M > c.cand_cap) return false;         // same counts in every CTA: the whole cluster falls back
  for (int i = tid; i < M; i += kSelThreads) {
    int r = 0;
#pragma unroll
    for (int q = 1; q < kMaxCluster; ++q) r += i >= start[q] ? 1 : 0;
    cand_all[i] = cluster.map_shared_rank(cand_local, r)[i - start[r]];
  }
  __syncthreads();

  // 4. which own candidates are kept.  A 512-bin histogram of ALL candidate keys over [T0, row maximum]
  //    locates the bin b1 holding the k_q-th largest candidate: higher bins are kept, lower bins dropped,
  //    and only the few candidates inside b1 are ranked exactly (key, then position) against their bin.
  {
    const uint32_t d2 = kmax ^ T0;
    const int hb = d2 ? 31 - __clz(d2) : -1;
    const int shift2 = hb > 8 ? hb - 8 : 0;
    const uint32_t base2 = T0 >> shift2;
    for (int i = tid; i < M; i += kSelThreads)
      atomicAdd(&sh.hist_fast[(uint32_t)(cand_all[i] >> (32 + shift2)) - base2], 1u);
    __syncthreads();
    find_bin_from_top(sh.hist_fast, kSelThreads, p.k_q, sh);
    const uint32_t b1 = (uint32_t)sh.found[0];
    const int r1 = sh.found[1];                          // the k_q-th largest is the r1-th largest inside b1
    for (int ci = tid; ci < n_loc; ci += kSelThreads) {  // the clear cases, one thread each
      const unsigned long long mine = cand_local[ci];
      if ((uint32_t)(mine >> (32 + shift2)) - base2 > b1) {
        const int n = atomicAdd(&sh.n_sel_local, 1);
        sel_pos[n] = (int)(0xffffffffu - (uint32_t)(mine & 0xffffffffull));
      }
    }
    for (int ci = warp; ci < n_loc; ci += kSelWarps) {   // the border cases, one warp each
      const unsigned long long mine = cand_local[ci];
      if ((uint32_t)(mine >> (32 + shift2)) - base2 == b1) {
        int before = 0;
        for (int i = lane; i < M; i += 32) {
          const unsigned long long o = cand_all[i];
          before += ((uint32_t)(o >> (32 + shift2)) - base2 == b1 && o > mine) ? 1 : 0;
        }
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) before += __shfl_xor_sync(0xffffffffu, before, off);
        if (lane == 0 && before < r1) {
          const int n = atomicAdd(&sh.n_sel_local, 1);
          sel_pos[n] = (int)(0xffffffffu - (uint32_t)(mine & 0xffffffffull));
        }
      }
    }
  }
  __syncthreads();
  const int n_sel = sh.n_sel_local;
  if (tid < c.cs) cluster.map_shared_rank(sh.sel_cnt, tid)[c.rank] = n_sel;
  cluster.sync();   // last access to a peer's shared memory
  int offset = 0;
  for (int r = 0; r < c.rank; ++r) offset += sh.sel_cnt[r];

  // 5. output slots in ascending position: offset + number of kept positions of this CTA below one's own.
  int32_t *idx_row = p.idx + (int64_t)c.row * p.k_q;
  const int n_words = (c.n_local + 31) >> 5;
  if (n_sel > 128 && (size_t)n_words * 4 <= (size_t)c.cand_cap * 8) {
    // many kept rows in this CTA (clustered scores): a bitmap of the slice and a popcount prefix, O(n) instead
    // of the pairwise count.  The candidate list is no longer needed (every CTA is past its ranking).
    uint32_t *bm = reinterpret_cast<uint32_t *>(cand_all);
    uint32_t *thread_base = sh.gmax;                     // free since step 2
    for (int w = tid; w < n_words; w += kSelThreads) bm[w] = 0u;
    __syncthreads();
    for (int ci = tid; ci < n_sel; ci += kSelThreads) {
      const int lp = sel_pos[ci] - c.lo;
      atomicOr(&bm[lp >> 5], 1u << (lp & 31));
    }
    __syncthreads();
    const int wpt = (n_words + kSelThreads - 1) / kSelThreads;   // words per thread
    int mine_cnt = 0;
    for (int w = tid * wpt; w < min(n_words, (tid + 1) * wpt); ++w) mine_cnt += __popc(bm[w]);
    thread_base[tid] = (uint32_t)block_exclusive_scan(mine_cnt, sh.scan_tmp);
    __syncthreads();
    for (int ci = tid; ci < n_sel; ci += kSelThreads) {
      const int pos = sel_pos[ci], lp = pos - c.lo, w0 = lp >> 5, t = w0 / wpt;
      int before = (int)thread_base[t];
      for (int w = t * wpt; w < w0; ++w) before += __popc(bm[w]);
      before += __popc(bm[w0] & ((1u << (lp & 31)) - 1u));
      const int slot = offset + before;
      idx_row[slot] = p.S + pos;
      if (ci < c.list_cap) c.list[ci] = make_int2(slot, p.S + pos);
    }
  } else {
    int tps = 32;
    while (tps > 1 && n_sel * tps > kSelThreads) tps >>= 1;
    const int sub2 = tid & (tps - 1);
    for (int c0 = 0; c0 < n_sel; c0 += kSelThreads / tps) {
      const int ci = c0 + tid / tps;
      const bool valid = ci < n_sel;
      const int mine = valid ? sel_pos[ci] : 0;
      int before = 0;
      if (valid)
        for (int i = sub2; i < n_sel; i += tps) before += sel_pos[i] < mine ? 1 : 0;
      for (int off = 1; off < tps; off <<= 1) before += __shfl_xor_sync(0xffffffffu, before, off);
      if (valid && sub2 == 0) {
        const int slot = offset + before;
        idx_row[slot] = p.S + mine;
        if (ci < c.list_cap) c.list[ci] = make_int2(slot, p.S + mine);
      }
    }
  }
  // When the kept rows sit in few CTAs (clustered scores) the gather is re-dealt evenly: the positions are
  // in idx by now, so after one more cluster barrier every CTA copies an equal range of slots.
  int most = 0;
  for (int r = 0; r < c.cs; ++r) most = max(most, sh.sel_cnt[r]);
  const bool redeal = c.cs > 1 && most > 2 * (p.k_q / c.cs) + 64;   // same answer in every CTA
  if (tid == 0) sh.list_count = redeal ? -1 : n_sel;
  __syncthreads();
  if (redeal) cluster.sync();                            // every CTA's idx entries are written (and visible in the cluster)
  return true;
}

// ---- general path -------------------------------------------------------------------------------
__device__ void general_select(cg::cluster_group &cluster, SelShared &sh, const SelectParams &p, const SelCtx &c) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t(*hist_merged)[kMaxBins] = reinterpret_cast<uint32_t(*)[kMaxBins]>(c.scratch);   // only rank 0's copy is used
  uint32_t *hist_local = reinterpret_cast<uint32_t *>(c.scratch) + 3 * kMaxBins;
  const float *data = c.data;
  const int n_local = c.n_local;
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
      idx_row[slot] = pos;
      const int n = atomicAdd(&sh.list_count, 1);
      if (n < c.list_cap) c.list[n] = make_int2(slot, pos);
    }
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  __syncthreads();
  cluster.sync();   // no CTA moves on (and may exit) while a peer still reads its shared memory
}

__global__ void __launch_bounds__(kSelThreads) select_compact_kernel(const SelectParams p, int n_rows, int chunk,
                                                                      int resident, int list_cap, int cand_cap,
                                                                      int try_fast) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int cid = blockIdx.x / cs;
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
  c.list = reinterpret_cast<int2 *>(after);
  c.list_cap = list_cap;
  c.scratch = after + (((size_t)list_cap * sizeof(int2) + 15) & ~(size_t)15);   // 16-byte aligned
  c.cand_cap = cand_cap;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = c.row / p.H_q, h = c.row - b * p.H_q;
  const int kvh = h / p.G, j = h - kvh * p.G;
  const float *grow = p.scores + (int64_t)c.row * p.row_stride + c.lo;   // 16-byte aligned: chunk % 4 == 0

  sh.hist_fast[tid] = 0;
  c.data = grow;
  if (resident) {
    const int n_vec = c.n_local >> 2;
    for (int v = tid; v < n_vec; v += kSelThreads) {
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(staged + 4 * v);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(grow + 4 * v) : "memory");
    }
    for (int i = (n_vec << 2) + tid; i < c.n_local; i += kSelThreads) staged[i] = grow[i];
    asm volatile("cp.async.wait_all;" ::: "memory");
    c.data = staged;
  }
  __syncthreads();
  cluster.barrier_wait();

  bool done = false;
  if (try_fast) done = resident ? fast_select<true>(cluster, sh, p, c) : fast_select<false>(cluster, sh, p, c);
  if (!done) general_select(cluster, sh, p, c);

  // gather this CTA's kept rows into head j's segment of the reduced cache: a warp moves four rows at a
  // time (K in lanes 0-15, V in lanes 16-31), all loads issued before the stores
  const bool redeal = sh.list_count < 0;                 // take slots [rank, rank+1) * k_q / cs, positions from idx
  const int per_cta = (p.k_q + cs - 1) / cs;
  const int slot_lo = redeal ? min(p.k_q, rank * per_cta) : 0;
  const int n_list = redeal ? min(p.k_q, slot_lo + per_cta) - slot_lo : min(sh.list_count, list_cap);
  const int32_t *idx_row = p.idx + (int64_t)c.row * p.k_q;
  const uint16_t *src_base = (lane < 16 ? p.K : p.V) + (int64_t)b * p.ks.batch_stride + (int64_t)kvh * p.ks.head_stride +
                             (lane & 15) * 8;
  uint16_t *dst_base = (lane < 16 ? p.Kc : p.Vc) + (int64_t)b * p.cs.batch_stride + (int64_t)kvh * p.cs.head_stride +
                       ((int64_t)p.S + (int64_t)j * p.k_q) * p.cs.token_stride + (lane & 15) * 8;
  for (int e0 = warp * 4; e0 < n_list; e0 += kSelWarps * 4) {
    uint4 v[4];
    int slot[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = min(e0 + u, n_list - 1);
      const int2 sp = redeal ? make_int2(slot_lo + e, __ldcg(idx_row + slot_lo + e)) : c.list[e];
      slot[u] = sp.x;
      v[u] = ld_stream_v4(src_base + (int64_t)sp.y * p.ks.token_stride);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (e0 + u < n_list) st_v4(dst_base + (int64_t)slot[u] * p.cs.token_stride, v[u]);
  }
}

static size_t select_smem_bytes(int chunk, int list_cap, int cand_cap, bool resident) {
  size_t scratch = (size_t)cand_cap * (8 + 8) + 16 + (size_t)list_cap * 4;   // candidates (own, all) and kept positions
  if (scratch < (size_t)kGeneralScratch) scratch = kGeneralScratch;
  return sizeof(SelShared) + (((size_t)list_cap * sizeof(int2) + 15) & ~(size_t)15) + scratch +
         (resident ? (size_t)chunk * sizeof(float) : 0);
}

cudaError_t select_compact_setup() {
  return cudaFuncSetAttribute(select_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelSmemLimit);
}

cudaError_t launch_select_compact(const SelectParams &p, int n_sm, cudaStream_t stream) {
  const bool select = p.k_q > 0 && p.E > 0;
  const int n_rows = select ? p.B * p.H_q : 0;
  // cluster size: slices of at least 2048 scores, at most 8 CTAs (the portable limit)
  int cs = 1;
  while (cs < kMaxCluster && (int64_t)cs * 2048 < p.E) cs <<= 1;
  int chunk = (p.E + cs - 1) / cs;
  chunk = (chunk + 3) & ~3;
  if (chunk < 4) chunk = 4;
  const int list_cap = chunk < p.k_q ? chunk : (p.k_q > 0 ? p.k_q : 1);
  // the prefilter needs at least 2*k_q thread maxima; its buffers hold 1.5*k_q + 256 candidates
  const int try_fast = select && 2 * (int64_t)p.k_q <= (int64_t)cs * kSelThreads;
  const int cand_cap = try_fast ? (p.k_q + p.k_q / 2 + 256) & ~1 : 0;
  const bool resident = select_smem_bytes(chunk, list_cap, cand_cap, true) <= (size_t)kSelSmemLimit;
  const size_t smem = select_smem_bytes(chunk, list_cap, cand_cap, resident);

  const int static_items = p.B * p.H_kv * (p.S + p.R + 1);
  int copy_clusters = (static_items + cs * kSelWarps * 2 - 1) / (cs * kSelWarps * 2);
  if (copy_clusters < 1) copy_clusters = 1;
  const int cap = (n_sm + cs - 1) / cs;
  if (copy_clusters > cap) copy_clusters = cap;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_rows + copy_clusters) * cs), 1, 1);
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
  return cudaLaunchKernelEx(&cfg, select_compact_kernel, p, n_rows, chunk, (int)resident, list_cap, cand_cap,
                            try_fast);
}

}  // namespace sagekv
