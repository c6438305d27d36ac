// Step 2 (first half): softmax attention of the last token's query over the eviction region.
//
// Pass 1 (score_logits_kernel) streams the K rows of the eviction region once.  A warp takes 16 tokens
// per tensor-core tile: token rows are the M dimension, the KV head's G query heads (padded to 8) the
// N dimension, head_dim the contraction.  Every lane loads 16-byte pieces of "its" two token rows
// straight from global memory into the A fragment; because a dot product does not care in which order
// the 128 products are summed, the fragment's k slots are filled with whatever columns those 16 bytes
// hold and the query (B fragment) is loaded with the same permutation.  The kernel writes the scaled
// logits (log2 units) and one (max, sum-of-exp2) pair per CTA and head.
// Pass 2 (score_finalize_kernel) merges those pairs per row and normalises the row in place; the
// logits were written a few microseconds earlier and are still in L2.
#include "common.cuh"

namespace sagekv {

__global__ void __launch_bounds__(kScoreWarps * 32) score_logits_kernel(const ScoreParams p) {
  const int chunk = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  if (chunk == 0 && p.sketch_off >= 0) {   // the rows' histograms are filled by atomic adds in the second pass
    for (int i = threadIdx.x; i < p.G * (kSketchBins + 4); i += kScoreWarps * 32) {
      const int h = i / (kSketchBins + 4);
      reinterpret_cast<uint32_t *>(p.scores + ((int64_t)b * p.H_q + kvh * p.G + h) * p.row_stride + p.sketch_off)[i - h * (kSketchBins + 4)] = 0u;
    }
  }

  // B fragments: query head (kvh*G + g) for n = g, zero padding for n >= G
  uint4 qf[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) qf[j] = make_uint4(0u, 0u, 0u, 0u);
  if (g < p.G) {
    const uint16_t *qrow = p.q + ((int64_t)b * p.H_q + kvh * p.G + g) * kHeadDim;
#pragma unroll
    for (int j = 0; j < 4; ++j) qf[j] = *reinterpret_cast<const uint4 *>(qrow + j * 32 + c * 8);
  }

  const uint16_t *Kbase = p.K + (int64_t)b * p.ks.batch_stride + (int64_t)kvh * p.ks.head_stride +
                          (int64_t)p.S * p.ks.token_stride;
  const int tok_base = chunk * kScoreChunk + warp * kScoreTokPerWarp;
  const int last = p.E - 1;

  // lane (g, c) holds, of token rows g and g+8 of each tile, the 16-byte pieces at columns j*32 + c*8
  uint4 ka[2][4], kb[2][4];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r0 = min(tok_base + t * 16 + g, last);
    const int r1 = min(tok_base + t * 16 + g + 8, last);
    const char *pa = reinterpret_cast<const char *>(Kbase + (int64_t)r0 * p.ks.token_stride) + c * 16;
    const char *pb = reinterpret_cast<const char *>(Kbase + (int64_t)r1 * p.ks.token_stride) + c * 16;
    const bool ok = SAGEKV_OK_INDEX(p.status, r0 >= 0 && r0 < p.E && r1 >= 0 && r1 < p.E && kvh < p.H_kv && b < p.B);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      ka[t][j] = ok ? ld_stream_v4(pa + j * 64) : make_uint4(0u, 0u, 0u, 0u);
      kb[t][j] = ok ? ld_stream_v4(pb + j * 64) : make_uint4(0u, 0u, 0u, 0u);
    }
  }

  // running softmax statistics of heads 2c and 2c+1 over the rows this lane sees
  float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;
  const int h0 = 2 * c, h1 = 2 * c + 1;
  float *row0 = p.scores + ((int64_t)b * p.H_q + kvh * p.G + h0) * p.row_stride;
  float *row1 = row0 + p.row_stride;

#pragma unroll
  for (int t = 0; t < 2; ++t) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      mma_bf16_16816(a0, a1, a2, a3, ka[t][j].x, kb[t][j].x, ka[t][j].y, kb[t][j].y, qf[j].x, qf[j].y);
      mma_bf16_16816(a0, a1, a2, a3, ka[t][j].z, kb[t][j].z, ka[t][j].w, kb[t][j].w, qf[j].z, qf[j].w);
    }
    const int r0 = tok_base + t * 16 + g, r1 = r0 + 8;
    const float s00 = a0 * p.scale_log2, s01 = a1 * p.scale_log2;   // (r0,h0) (r0,h1)
    const float s10 = a2 * p.scale_log2, s11 = a3 * p.scale_log2;   // (r1,h0) (r1,h1)
    const bool v0 = r0 < p.E && SAGEKV_OK_INDEX(p.status, r0 >= 0 && (int64_t)r0 < p.row_stride);
    const bool v1 = r1 < p.E && SAGEKV_OK_INDEX(p.status, r1 >= 0 && (int64_t)r1 < p.row_stride);
    if (h0 < p.G) {
      if (v0) row0[r0] = s00;
      if (v1) row0[r1] = s10;
      const float x0 = v0 ? s00 : -INFINITY, x1 = v1 ? s10 : -INFINITY;
      const float M = fmaxf(m0, fmaxf(x0, x1));
      if (M != -INFINITY) l0 = l0 * fast_exp2(m0 - M) + fast_exp2(x0 - M) + fast_exp2(x1 - M);
      m0 = M;
    }
    if (h1 < p.G) {
      if (v0) row1[r0] = s01;
      if (v1) row1[r1] = s11;
      const float x0 = v0 ? s01 : -INFINITY, x1 = v1 ? s11 : -INFINITY;
      const float M = fmaxf(m1, fmaxf(x0, x1));
      if (M != -INFINITY) l1 = l1 * fast_exp2(m1 - M) + fast_exp2(x0 - M) + fast_exp2(x1 - M);
      m1 = M;
    }
  }

  // over the 8 row groups of the warp (lanes with equal c)
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    merge_ml(m0, l0, __shfl_xor_sync(0xffffffffu, m0, off), __shfl_xor_sync(0xffffffffu, l0, off));
    merge_ml(m1, l1, __shfl_xor_sync(0xffffffffu, m1, off), __shfl_xor_sync(0xffffffffu, l1, off));
  }
  __shared__ float sm_m[kScoreWarps][kMaxGroup], sm_l[kScoreWarps][kMaxGroup];
  if (g == 0) {
    sm_m[warp][h0] = m0; sm_l[warp][h0] = l0;
    sm_m[warp][h1] = m1; sm_l[warp][h1] = l1;
  }
  __syncthreads();
  if (threadIdx.x < p.G) {
    const int h = threadIdx.x;
    float m = sm_m[0][h], l = sm_l[0][h];
#pragma unroll
    for (int w = 1; w < kScoreWarps; ++w) merge_ml(m, l, sm_m[w][h], sm_l[w][h]);
    if (SAGEKV_OK_INDEX(p.status, chunk < p.n_chunks && kvh * p.G + h < p.H_q))
      p.partials[((int64_t)b * p.H_q + kvh * p.G + h) * p.n_chunks + chunk] = make_float2(m, l);
  }
}

constexpr int kFinalizeThreads = 256;

__global__ void __launch_bounds__(kFinalizeThreads) score_finalize_kernel(const ScoreParams p, int per_slice) {
  const int row = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float m = -INFINITY, l = 0.f;
  const float2 *part = p.partials + (int64_t)row * p.n_chunks;
  for (int i = threadIdx.x; i < p.n_chunks; i += kFinalizeThreads) {
    const float2 v = part[i];
    merge_ml(m, l, v.x, v.y);
  }
#pragma unroll
  for (int off = 1; off < 32; off <<= 1)
    merge_ml(m, l, __shfl_xor_sync(0xffffffffu, m, off), __shfl_xor_sync(0xffffffffu, l, off));
  __shared__ float sm_m[kFinalizeThreads / 32], sm_l[kFinalizeThreads / 32];
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
  __syncthreads();
  m = sm_m[0]; l = sm_l[0];
#pragma unroll
  for (int w = 1; w < kFinalizeThreads / 32; ++w) merge_ml(m, l, sm_m[w], sm_l[w]);
  const float inv = 1.f / l;

  float *rowp = p.scores + (int64_t)row * p.row_stride;
  const int lo = blockIdx.x * per_slice;            // per_slice is a multiple of 4
  const int hi = min(p.E, lo + per_slice);
  if (!SAGEKV_OK_INDEX(p.status, row < p.B * p.H_q && lo >= 0 && (int64_t)hi <= p.row_stride)) return;
  // eight 16-byte loads in flight per thread before the first store (the row is read and written in place,
  // so the compiler would otherwise keep every load behind the previous store)
  for (int i0 = lo + threadIdx.x * 4; i0 < hi; i0 += kFinalizeThreads * 4 * 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kFinalizeThreads * 4;
      if (i + 3 < hi) v[u] = *reinterpret_cast<const float4 *>(rowp + i);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kFinalizeThreads * 4;
      if (i + 3 < hi) {
        v[u].x = fast_exp2(v[u].x - m) * inv; v[u].y = fast_exp2(v[u].y - m) * inv;
        v[u].z = fast_exp2(v[u].z - m) * inv; v[u].w = fast_exp2(v[u].w - m) * inv;
        *reinterpret_cast<float4 *>(rowp + i) = v[u];
      } else if (i < hi) {
        for (int e = i; e < hi; ++e) rowp[e] = fast_exp2(rowp[e] - m) * inv;
      }
    }
  }
}

// The normalisation pass for rows that have room for the histogram of the group maxima (see common.cuh): one
// CTA per slice of a row, a thread per group, so a thread's running maximum of what it stores is the group's
// maximum.  The row maximum is exp2(0) / l exactly, so every CTA of the row lays the same bins.
constexpr int kSketchThreads = kSketchGroups;

__global__ void __launch_bounds__(kSketchThreads) score_finalize_sketch_kernel(const ScoreParams p, int chunk) {
  const int row = blockIdx.y, slice = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = -INFINITY, l = 0.f;
  const float2 *part = p.partials + (int64_t)row * p.n_chunks;
  for (int i = tid; i < p.n_chunks; i += kSketchThreads) {
    const float2 v = part[i];
    merge_ml(m, l, v.x, v.y);
  }
#pragma unroll
  for (int off = 1; off < 32; off <<= 1)
    merge_ml(m, l, __shfl_xor_sync(0xffffffffu, m, off), __shfl_xor_sync(0xffffffffu, l, off));
  __shared__ float sm_m[kSketchThreads / 32], sm_l[kSketchThreads / 32];
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
  __syncthreads();
  m = sm_m[0]; l = sm_l[0];
#pragma unroll
  for (int w = 1; w < kSketchThreads / 32; ++w) merge_ml(m, l, sm_m[w], sm_l[w]);
  const float inv = 1.f / l;

  float *rowp = p.scores + (int64_t)row * p.row_stride;
  const int lo = slice * chunk;
  const int n_local = max(0, min(p.E - lo, chunk));
  if (!SAGEKV_OK_INDEX(p.status, row < p.B * p.H_q && p.sketch_off >= p.E && p.sketch_off + kSketchBins + 4 <= p.row_stride))
    return;
  const int n_vec = n_local >> 2;
  float *base = rowp + lo;
  float fm = -INFINITY;
  for (int v0 = 0; v0 < n_vec; v0 += 8 * kSketchThreads) {
    float4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v = v0 + u * kSketchThreads + tid;
      if (v < n_vec) x[u] = *reinterpret_cast<const float4 *>(base + 4 * v);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v = v0 + u * kSketchThreads + tid;
      if (v < n_vec) {
        x[u].x = fast_exp2(x[u].x - m) * inv; x[u].y = fast_exp2(x[u].y - m) * inv;
        x[u].z = fast_exp2(x[u].z - m) * inv; x[u].w = fast_exp2(x[u].w - m) * inv;
        *reinterpret_cast<float4 *>(base + 4 * v) = x[u];
        fm = fmaxf(fmaxf(fm, x[u].x), fmaxf(x[u].y, fmaxf(x[u].z, x[u].w)));
      }
    }
  }
  const int tail_i = (n_vec << 2) + tid;
  if (tail_i < n_local) {
    const float y = fast_exp2(base[tail_i] - m) * inv;
    base[tail_i] = y;
    fm = fmaxf(fm, y);
  }
  __shared__ uint32_t sm_hist[kSketchBins];
  sm_hist[tid] = 0u;
  __syncthreads();
  const uint32_t kmax = score_key(inv);
  const uint32_t bin0 = (kmax >> kSketchShift) - (uint32_t)(kSketchBins - 1);
  if (tid < n_vec || tail_i < n_local) {                  // the group is not empty
    const uint32_t q = score_key(fm) >> kSketchShift;
    atomicAdd(&sm_hist[q > bin0 ? min(q - bin0, (uint32_t)kSketchBins - 1u) : 0u], 1u);
  }
  __syncthreads();
  uint32_t *sketch = reinterpret_cast<uint32_t *>(rowp + p.sketch_off);
  if (sm_hist[tid] != 0u) atomicAdd(&sketch[tid], sm_hist[tid]);
  if (slice == 0 && tid == 0) {
    sketch[kSketchBins] = kSketchMagic;
    sketch[kSketchBins + 1] = (uint32_t)p.E;
    sketch[kSketchBins + 2] = bin0;
    sketch[kSketchBins + 3] = kmax;
  }
}

cudaError_t launch_score(const ScoreParams &p_in, int n_sm, cudaStream_t stream) {
  if (p_in.E <= 0) return cudaSuccess;
  ScoreParams p = p_in;
  const bool list = p.list_k_q > 0 && list_applies(p.E, p.list_k_q, p.row_stride);
  p.sketch_off = !list && p.sketch && sketch_fits(p.E, p.row_stride) ? sketch_offset(p.E) : (int64_t)-1;
  dim3 grid(p.n_chunks, p.H_kv, p.B);
  score_logits_kernel<<<grid, kScoreWarps * 32, 0, stream>>>(p);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  if (list) return launch_score_finalize_candidates(p, stream);
  const int rows = p.B * p.H_q;
  if (p.sketch_off >= 0) {
    score_finalize_sketch_kernel<<<dim3(kSketchSlices, rows), kSketchThreads, 0, stream>>>(p, sketch_chunk(p.E));
    return cudaGetLastError();
  }
  int slices = (n_sm * 4 + rows - 1) / rows;
  const int max_slices = (p.E + 1023) / 1024;
  if (slices > max_slices) slices = max_slices;
  if (slices < 1) slices = 1;
  int per_slice = (p.E + slices - 1) / slices;
  per_slice = (per_slice + 3) & ~3;
  slices = (p.E + per_slice - 1) / per_slice;
  score_finalize_kernel<<<dim3(slices, rows), kFinalizeThreads, 0, stream>>>(p, per_slice);
  return cudaGetLastError();
}

}  // namespace sagekv
