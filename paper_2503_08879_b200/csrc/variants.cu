// Kernels of the comparison paths that sit beside the four steps of the method:
//   - StreamLLM_R (Section 3.1 "Baselines", Appendix A.1): the sink + recent + last rows of a PRE-RoPE key cache,
//     each key rotated by its index inside the kept window while it is copied; values copied verbatim.
//   - the pooled reading of Step 2: the score rows of a KV head's G query heads summed into one row.
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

}  // namespace sagekv
