// Step 2 (second half) and Step 3: per-query-head top-k over the score rows, then the gather that
// builds the reduced cache  C = Concat(sink, selected, recent, last).
//
// One thread-block cluster owns one score row.  Each CTA of the cluster stages its contiguous slice of
// the row in shared memory once (cp.async, 16 bytes per request) and every later pass works on that
// copy, so the scores cross the memory system a single time.  The k-th largest key is found by a
// three-digit radix select (11 + 11 + 10 bits of the order-preserving integer image of the fp32
// score): per digit every CTA histograms its slice in shared memory, the histograms are added into
// CTA 0's shared memory through distributed-shared-memory atomics, and after a cluster barrier every
// CTA locates the digit in which the k-th key falls.  With the exact threshold known, a ballot/popcount
// ranking in row order (warp -> CTA -> cluster prefix) gives every kept element its output slot
// directly: strictly larger keys are kept, of the keys equal to the threshold the lowest positions are
// kept, and the slots are ascending in position.  The CTA that owns an element also copies its K and V
// rows into the head's segment of the reduced cache.  A few extra clusters copy the sink, recent and
// last rows, which do not depend on the scores.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace sagekv {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxCluster = 8;
constexpr int kMaxBins = 2048;
constexpr int kSelSmemLimit = 200 * 1024;

struct SelShared {
  uint32_t hist_local[kMaxBins];
  uint32_t hist_merged[3][kMaxBins];   // merge target: only cluster rank 0's copy is written
  int totals[kMaxCluster][2];          // (kept-larger, equal-to-threshold) per CTA; rank 0's copy
  int warp_cnt[kSelWarps][2];
  int scan_tmp[kSelWarps];
  int found[2];
  int list_count;
  int pad_[1];
};
static_assert(sizeof(SelShared) % 16 == 0, "staged scores must stay 16-byte aligned");

__device__ __forceinline__ uint32_t score_key(float x) {
  const uint32_t u = __float_as_uint(x + 0.0f);         // -0 becomes +0: the two compare equal as numbers
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);   // larger float <=> larger unsigned key
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

__global__ void __launch_bounds__(kSelThreads) select_compact_kernel(const SelectParams p, int n_rows, int chunk,
                                                                      int resident, int list_cap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int cid = blockIdx.x / cs;
  if (cid >= n_rows) {   // whole cluster takes this branch together; it touches no peer's memory
    copy_static_rows(p, (cid - n_rows) * cs + rank, (gridDim.x / cs - n_rows) * cs);
    return;
  }

  SelShared &sh = *reinterpret_cast<SelShared *>(smem_raw);
  float *staged = reinterpret_cast<float *>(smem_raw + sizeof(SelShared));
  int2 *list = reinterpret_cast<int2 *>(smem_raw + sizeof(SelShared) + (resident ? (size_t)chunk * sizeof(float) : 0));

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = cid;
  const int b = row / p.H_q, h = row - b * p.H_q;
  const int kvh = h / p.G, j = h - kvh * p.G;
  const int lo = rank * chunk;
  const int n_local = max(0, min(p.E - lo, chunk));
  const float *grow = p.scores + (int64_t)row * p.row_stride + lo;   // 16-byte aligned: chunk % 4 == 0

  for (int i = tid; i < kMaxBins; i += kSelThreads) {
    sh.hist_local[i] = 0;
    sh.hist_merged[0][i] = 0; sh.hist_merged[1][i] = 0; sh.hist_merged[2][i] = 0;
  }
  if (tid == 0) sh.list_count = 0;

  const float *data = grow;
  if (resident) {
    const int n_vec = n_local >> 2;
    for (int v = tid; v < n_vec; v += kSelThreads) {
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(staged + 4 * v);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(grow + 4 * v) : "memory");
    }
    for (int i = (n_vec << 2) + tid; i < n_local; i += kSelThreads) staged[i] = grow[i];
    asm volatile("cp.async.wait_all;" ::: "memory");
    data = staged;
  }
  __syncthreads();
  cluster.sync();   // every CTA's merge histograms are zero before any peer adds into them

  // ---- radix select: threshold key and how many keys equal to it are kept ----
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
        if (lane == 0 && bin != 0xffffffffu) atomicAdd(&sh.hist_local[bin], 32u);
      } else if (bin != 0xffffffffu) {
        atomicAdd(&sh.hist_local[bin], 1u);
      }
    }
    __syncthreads();
    uint32_t *merged0 = cluster.map_shared_rank(&sh.hist_merged[pass][0], 0);
    for (int bin = tid; bin < nb; bin += kSelThreads) {
      const uint32_t v = sh.hist_local[bin];
      if (v) {
        atomicAdd(merged0 + bin, v);
        sh.hist_local[bin] = 0;
      }
    }
    cluster.sync();
    // thread t looks at bins nb-1-t*per ... downwards; `above` = keys in higher bins
    const int per = nb / kSelThreads;
    uint32_t cnt[4];
    int mine = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      cnt[e] = 0;
      if (e < per) {
        cnt[e] = merged0[nb - 1 - (tid * per + e)];
        mine += (int)cnt[e];
      }
    }
    int above = block_exclusive_scan(mine, sh.scan_tmp);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (e < per) {
        if (above < k_rem && above + (int)cnt[e] >= k_rem) {
          sh.found[0] = nb - 1 - (tid * per + e);
          sh.found[1] = k_rem - above;
        }
        above += (int)cnt[e];
      }
    }
    __syncthreads();
    prefix = (prefix << bits) | (uint32_t)sh.found[0];
    k_rem = sh.found[1];
    __syncthreads();                                    // found[] is rewritten by the next pass
  }
  const uint32_t tau = prefix;                          // exact key of the k-th largest score
  const int ties_kept = k_rem;                          // >= 1 keys equal to tau are kept, lowest positions first

  // ---- ranks in row order: warp w owns the contiguous range [w*wlen, (w+1)*wlen) of the slice ----
  const int wlen = (((chunk + kSelWarps - 1) / kSelWarps) + 31) & ~31;
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
    t0[2 * rank] = cta_gt;
    t0[2 * rank + 1] = cta_eq;
  }
  cluster.sync();
  {
    const int *t0 = cluster.map_shared_rank(&sh.totals[0][0], 0);
    for (int r = 0; r < rank; ++r) { gt_before += t0[2 * r]; eq_before += t0[2 * r + 1]; }
  }

  int32_t *idx_row = p.idx + (int64_t)row * p.k_q;
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
      const int pos = p.S + lo + i;
      idx_row[slot] = pos;
      const int n = atomicAdd(&sh.list_count, 1);
      if (n < list_cap) list[n] = make_int2(slot, pos);
    }
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  __syncthreads();

  // ---- gather this CTA's kept rows into head j's segment of the reduced cache ----
  const int n_list = min(sh.list_count, list_cap);
  for (int e = warp; e < n_list; e += kSelWarps) {
    const int2 sp = list[e];
    copy_kv_row(p, b, kvh, sp.y, (int64_t)p.S + (int64_t)j * p.k_q + sp.x, lane);
  }
  cluster.sync();   // no CTA leaves while a peer may still read its shared memory
}

static size_t select_smem_bytes(int chunk, int list_cap, bool resident) {
  return sizeof(SelShared) + (size_t)list_cap * sizeof(int2) + (resident ? (size_t)chunk * sizeof(float) : 0);
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
  const bool resident = select_smem_bytes(chunk, list_cap, true) <= (size_t)kSelSmemLimit;
  const size_t smem = select_smem_bytes(chunk, list_cap, resident);

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
  return cudaLaunchKernelEx(&cfg, select_compact_kernel, p, n_rows, chunk, (int)resident, list_cap);
}

}  // namespace sagekv
