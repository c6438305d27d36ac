// sagekv_score_static: the score step for callers that must not allocate device memory.
//
// sagekv_score keeps its per-CTA softmax partials in scratch that sagekv_create obtained with
// cudaMalloc.  This variant keeps them in a fixed array that is part of the library image instead, so
// using it needs neither a context nor any allocation.  The array is shared by every call on a device.
#include <math.h>
#include <mutex>

#include "common.cuh"

using namespace sagekv;

namespace {

// (max, sum) pairs: one per score row and 256-token chunk of the eviction region.  256 KiB per GPU
// that loads the library, held until the process exits.
constexpr int kStaticPartials = 32768;
static __device__ __align__(256) float2 g_score_partials[kStaticPartials];

constexpr int kMaxDevices = 64;
struct PerDevice {
  float2 *partials;   // device address of g_score_partials on this device (the symbol itself is only a host-side handle)
  int n_sm;
  bool ready;
};
PerDevice g_dev[kMaxDevices];
std::mutex g_mutex;

// One-time set-up for the current device: resolve the array's device address and read the SM count.
cudaError_t setup_current_device(PerDevice **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  PerDevice &d = g_dev[dev];
  if (!d.ready) {
    float2 *ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_score_partials);
    if (e != cudaSuccess) return e;
    int n_sm = 0;
    e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    d.partials = ptr;
    d.n_sm = n_sm;
    d.ready = true;
  }
  *out = &d;
  return cudaSuccess;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int sagekv_score_static(const sagekv_shape *shape, const void *q_last, const void *K, sagekv_strides ks,
                                   int64_t n_ctx, int32_t n_init, int32_t n_recent, float *scores,
                                   int64_t scores_row_stride, void *stream) {
  if (shape == nullptr || q_last == nullptr || K == nullptr || scores == nullptr) return SAGEKV_ERR_INVALID;
  if (shape->n_q_heads < 1 || shape->n_kv_heads < 1 || shape->batch < 1 ||
      shape->n_q_heads % shape->n_kv_heads != 0 || !(shape->softmax_scale >= 0.f))
    return SAGEKV_ERR_INVALID;
  if (n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx) return SAGEKV_ERR_INVALID;
  const int G = shape->n_q_heads / shape->n_kv_heads;
  if (shape->head_dim != kHeadDim || G > kMaxGroup || n_ctx > (int64_t)1 << 30 ||
      (int64_t)shape->batch * shape->n_q_heads > 65535)
    return SAGEKV_ERR_UNSUPPORTED;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  if (scores_row_stride < E || ks.token_stride < kHeadDim) return SAGEKV_ERR_INVALID;
  if (!aligned16(q_last) || !aligned16(K) || !aligned16(scores) || ks.batch_stride % 8 || ks.head_stride % 8 ||
      ks.token_stride % 8 || scores_row_stride % 4)
    return SAGEKV_ERR_ALIGN;
  const int64_t n_chunks = (E + kScoreChunk - 1) / kScoreChunk;
  // the fixed array bounds the problem: rows * chunks pairs must fit
  if ((int64_t)shape->batch * shape->n_q_heads * n_chunks > kStaticPartials) return SAGEKV_ERR_TOO_LARGE;
  PerDevice *dev = nullptr;
  if (setup_current_device(&dev) != cudaSuccess) return SAGEKV_ERR_CUDA;
  ScoreParams p;
  p.q = static_cast<const uint16_t *>(q_last);
  p.K = static_cast<const uint16_t *>(K);
  p.ks = ks;
  p.scores = scores;
  p.row_stride = scores_row_stride;
  p.partials = dev->partials;     // every pair is written by pass 1 before pass 2 reads it: nothing to clear
  p.n_chunks = (int)n_chunks;
  p.E = (int)E;
  p.S = n_init;
  p.G = G;
  p.H_q = shape->n_q_heads;
  p.H_kv = shape->n_kv_heads;
  p.B = shape->batch;
  const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.0f / sqrtf((float)shape->head_dim);
  p.scale_log2 = scale * kLog2e;
  return launch_score(p, dev->n_sm, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SAGEKV_OK : SAGEKV_ERR_CUDA;
}
