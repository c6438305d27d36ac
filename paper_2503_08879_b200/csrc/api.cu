// The C interface (include/sagekv.h): argument checks on the host, then the kernel launches.
#include <math.h>
#include <mutex>
#include <new>

#include "common.cuh"

using namespace sagekv;

struct sagekv_ctx {
  sagekv_shape shape;
  int G;
  int64_t max_ctx;
  int32_t max_len;
  int device;               // the device the context was created on; every call must find it current
  const DeviceInfo *dev;    // that device's one-time set-up
  float scale;
  float2 *score_partials;   // [B*H_q, ceil(max_ctx / kScoreChunk)]
  int max_chunks;
  float *decode_partials;   // [B*H_kv, max_splits (clusters per head), kPartialStride]
  int max_splits;
  int32_t *tickets;         // [B*H_kv + 1], zero between launches; the status word follows them
  int32_t *status;          // one int32: kStatus* bits raised by the kernels
  int last_cuda_error;
  int overlap;              // 0, 1 or 2: see sagekv_set_overlap
  int select_overlap;       // 0, 1 or 2: see sagekv_set_select_overlap
  int decode_variant;       // 0, 1 or 2: see sagekv_set_decode_variant
  int hint;                 // 0, 1, 2: see sagekv_set_select_hint
  int32_t hint_k;
  int group_mode;           // 0: a selection per query head (the paper's), 1: one per KV head from pooled scores
};

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool strides_ok(const sagekv_strides &s) {
  return s.batch_stride % 8 == 0 && s.head_stride % 8 == 0 && s.token_stride % 8 == 0;
}
int cuda_fail(sagekv_ctx *ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda_error = (int)e;
  return SAGEKV_ERR_CUDA;
}

// One-time set-up per device (function attributes, SM count, cluster capacities), done with that device current.
constexpr int kMaxDevices = 64;
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;

cudaError_t device_setup(int dev, const DeviceInfo **out) {
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  DeviceInfo &d = g_dev[dev];
  if (!d.ready) {
    d.device = dev;
    cudaError_t e = cudaDeviceGetAttribute(&d.n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = select_compact_setup();
    if (e == cudaSuccess) e = decode_setup(&d);
    if (e != cudaSuccess) return e;
    d.ready = true;
  }
  *out = &d;
  return cudaSuccess;
}

// false: another device is current than the one the context belongs to
bool on_own_device(const sagekv_ctx *ctx) {
  int cur = -1;
  return cudaGetDevice(&cur) == cudaSuccess && cur == ctx->device;
}

}  // namespace

extern "C" {

int sagekv_create(sagekv_ctx **out, const sagekv_shape *shape, int64_t max_ctx, int32_t max_len) {
  if (out == nullptr) return SAGEKV_ERR_INVALID;
  *out = nullptr;
  if (shape == nullptr || shape->n_q_heads < 1 || shape->n_kv_heads < 1 || shape->batch < 1 || max_ctx < 1 ||
      max_len < 1 || shape->n_q_heads % shape->n_kv_heads != 0 || !(shape->softmax_scale >= 0.f))
    return SAGEKV_ERR_INVALID;
  if (shape->head_dim != kHeadDim || shape->n_q_heads / shape->n_kv_heads > kMaxGroup ||
      max_ctx > (int64_t)1 << 30 || (int64_t)shape->batch * shape->n_q_heads > 65535)
    return SAGEKV_ERR_UNSUPPORTED;
  sagekv_ctx *ctx = new (std::nothrow) sagekv_ctx();
  if (ctx == nullptr) return SAGEKV_ERR_NOMEM;
  ctx->shape = *shape;
  ctx->G = shape->n_q_heads / shape->n_kv_heads;
  ctx->max_ctx = max_ctx;
  ctx->max_len = max_len;
  ctx->scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.0f / sqrtf((float)shape->head_dim);
  ctx->last_cuda_error = 0;
  ctx->overlap = 0;
  ctx->select_overlap = 0;
  ctx->decode_variant = 0;
  ctx->hint = 0;
  ctx->hint_k = 0;
  ctx->group_mode = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || device_setup(dev, &ctx->dev) != cudaSuccess) {
    delete ctx;
    (void)cudaGetLastError();
    return SAGEKV_ERR_CUDA;
  }
  ctx->device = dev;
  ctx->max_chunks = (int)((max_ctx + kScoreChunk - 1) / kScoreChunk);
  {
    int cs, resident, smem;
    decode_geometry(max_len, 0, nullptr, &ctx->max_splits, &cs, &resident, &smem);   // clusters per head at the largest L ...
    if (ctx->max_splits < 4) ctx->max_splits = 4;                                    // ... or the most the launch geometry ever chooses
  }
  const size_t n_rows = (size_t)shape->batch * shape->n_q_heads;
  const size_t n_heads = (size_t)shape->batch * shape->n_kv_heads;
  cudaError_t e = cudaMalloc(&ctx->score_partials, n_rows * ctx->max_chunks * sizeof(float2));
  if (e == cudaSuccess)
    e = cudaMalloc(&ctx->decode_partials, n_heads * ctx->max_splits * kPartialStride * sizeof(float));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->tickets, (n_heads + 2) * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->tickets, 0, (n_heads + 2) * sizeof(int32_t));
  if (e == cudaSuccess) ctx->status = ctx->tickets + n_heads + 1;
  if (e != cudaSuccess) {
    cudaFree(ctx->score_partials);
    cudaFree(ctx->decode_partials);
    cudaFree(ctx->tickets);
    delete ctx;
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? SAGEKV_ERR_NOMEM : SAGEKV_ERR_CUDA;
  }
  *out = ctx;
  return SAGEKV_OK;
}

int sagekv_destroy(sagekv_ctx *ctx) {
  if (ctx == nullptr) return SAGEKV_ERR_INVALID;
  cudaFree(ctx->score_partials);
  cudaFree(ctx->decode_partials);
  cudaFree(ctx->tickets);
  delete ctx;
  return SAGEKV_OK;
}

int sagekv_budget_split(int32_t B, int32_t G, int32_t *n_init, int32_t *k_q, int32_t *n_recent) {
  if (B < 4 || G < 1 || n_init == nullptr || k_q == nullptr || n_recent == nullptr) return SAGEKV_ERR_INVALID;
  const int32_t sink = B / 4;
  int32_t k;
  if (B % (2 * G) == 0) {
    k = B / (2 * G);
  } else {
    k = 1;
    while ((int64_t)4 * k * G <= B) k *= 2;   // largest power of two with 2*G*k <= B
  }
  *n_init = sink;
  *k_q = k;
  *n_recent = B - sink - G * k;
  return SAGEKV_OK;
}

int sagekv_score(sagekv_ctx *ctx, const void *q_last, const void *K, sagekv_strides ks, int64_t n_ctx, int32_t n_init,
                 int32_t n_recent, float *scores, int64_t scores_row_stride, void *stream) {
  if (ctx == nullptr || q_last == nullptr || K == nullptr || scores == nullptr) return SAGEKV_ERR_INVALID;
  if (n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx) return SAGEKV_ERR_INVALID;
  if (n_ctx > ctx->max_ctx) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  if (scores_row_stride < E || ks.token_stride < kHeadDim) return SAGEKV_ERR_INVALID;
  if (!aligned16(q_last) || !aligned16(K) || !aligned16(scores) || !strides_ok(ks) || scores_row_stride % 4 != 0)
    return SAGEKV_ERR_ALIGN;
  ScoreParams p;
  p.q = static_cast<const uint16_t *>(q_last);
  p.K = static_cast<const uint16_t *>(K);
  p.ks = ks;
  p.scores = scores;
  p.row_stride = scores_row_stride;
  p.partials = ctx->score_partials;
  p.sketch = ctx->hint == 1;
  if (ctx->hint == 2 && ctx->hint_k > 0) {
    const int64_t kq = ctx->hint_k / ctx->G;
    p.list_k_q = (int)(kq < E ? kq : E);
  }
  p.status = ctx->status;
  p.n_chunks = (int)((E + kScoreChunk - 1) / kScoreChunk);
  p.E = (int)E;
  p.S = n_init;
  p.G = ctx->G;
  p.H_q = ctx->shape.n_q_heads;
  p.H_kv = ctx->shape.n_kv_heads;
  p.B = ctx->shape.batch;
  p.scale_log2 = ctx->scale * kLog2e;
  const cudaError_t e = launch_score(p, ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_select_compact(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride, const void *K,
                          const void *V, sagekv_strides ks, int64_t n_ctx, int32_t n_init, int32_t n_recent,
                          int32_t k, int32_t *idx, void *Kc, void *Vc, sagekv_strides cs, sagekv_cache_state *state,
                          void *stream) {
  if (ctx == nullptr || K == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr || state == nullptr ||
      state->d_step == nullptr)
    return SAGEKV_ERR_INVALID;
  const bool pooled = ctx->group_mode == 1;
  const int G = pooled ? 1 : ctx->G;                    // pooled: one score row and one list per KV head
  if (n_init < 0 || n_recent < 0 || k < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx || k % G != 0)
    return SAGEKV_ERR_INVALID;
  if (n_ctx > ctx->max_ctx) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  int64_t k_q = k / G;
  if (k_q > E) k_q = E;
  if (k_q > 0 && (scores == nullptr || idx == nullptr || scores_row_stride < E)) return SAGEKV_ERR_INVALID;
  if (ks.token_stride < kHeadDim || cs.token_stride < kHeadDim) return SAGEKV_ERR_INVALID;
  const int64_t L = (int64_t)n_init + G * k_q + n_recent + 1;
  if (L > ctx->max_len) return SAGEKV_ERR_UNSUPPORTED;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) || !strides_ok(ks) || !strides_ok(cs) ||
      (k_q > 0 && (!aligned16(scores) || scores_row_stride % 4 != 0)))
    return SAGEKV_ERR_ALIGN;
  SelectParams p;
  p.scores = scores;
  p.row_stride = scores_row_stride;
  p.K = static_cast<const uint16_t *>(K);
  p.V = static_cast<const uint16_t *>(V);
  p.ks = ks;
  p.Kc = static_cast<uint16_t *>(Kc);
  p.Vc = static_cast<uint16_t *>(Vc);
  p.cs = cs;
  p.idx = idx;
  p.d_step = state->d_step;
  p.E = (int)E;
  p.S = n_init;
  p.R = n_recent;
  p.N = (int)n_ctx;
  p.k_q = (int)k_q;
  p.G = G;
  p.H_q = pooled ? ctx->shape.n_kv_heads : ctx->shape.n_q_heads;
  p.H_kv = ctx->shape.n_kv_heads;
  p.B = ctx->shape.batch;
  p.status = ctx->status;
  p.sketch = !pooled && ctx->hint == 1;
  p.list = !pooled && ctx->hint == 2 && k == ctx->hint_k;
  p.pdl = ctx->select_overlap;
  const cudaError_t e = launch_select_compact(p, ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  state->n_init = n_init;
  state->k_q = (int32_t)k_q;
  state->n_sel = (int32_t)(G * k_q);
  state->n_recent = n_recent;
  state->ring_len = n_recent + 1;
  state->len = (int32_t)L;
  return SAGEKV_OK;
}

int sagekv_decode_attn(sagekv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *Kc, void *Vc,
                       sagekv_strides cs, const sagekv_cache_state *state, void *out, float *lse, void *stream) {
  if (ctx == nullptr || q == nullptr || Kc == nullptr || Vc == nullptr || state == nullptr || out == nullptr)
    return SAGEKV_ERR_INVALID;
  if ((k_new == nullptr) != (v_new == nullptr)) return SAGEKV_ERR_INVALID;
  if (k_new != nullptr && state->d_step == nullptr) return SAGEKV_ERR_INVALID;
  const bool pooled = ctx->group_mode == 1;
  if (state->n_init < 0 || state->k_q < 0 || state->n_recent < 0 || state->n_sel != (pooled ? 1 : ctx->G) * state->k_q ||
      state->ring_len != state->n_recent + 1 || state->len != state->n_init + state->n_sel + state->ring_len ||
      cs.token_stride < kHeadDim)
    return SAGEKV_ERR_INVALID;
  if (state->len > ctx->max_len) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  if (!aligned16(q) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(out) || !strides_ok(cs) ||
      (k_new != nullptr && (!aligned16(k_new) || !aligned16(v_new))))
    return SAGEKV_ERR_ALIGN;
  DecodeParams p;
  p.q = static_cast<const uint16_t *>(q);
  p.k_new = static_cast<const uint16_t *>(k_new);
  p.v_new = static_cast<const uint16_t *>(v_new);
  p.Kc = static_cast<uint16_t *>(Kc);
  p.Vc = static_cast<uint16_t *>(Vc);
  p.cs = cs;
  p.out = static_cast<uint16_t *>(out);
  p.lse = lse;
  p.partials = ctx->decode_partials;
  p.tickets = ctx->tickets;
  p.d_step = state->d_step;
  p.status = ctx->status;
  p.S = state->n_init;
  p.k_q = state->k_q;
  p.n_sel = state->n_sel;
  p.ring_len = state->ring_len;
  p.L = state->len;
  p.G = ctx->G;
  p.H_q = ctx->shape.n_q_heads;
  p.H_kv = ctx->shape.n_kv_heads;
  p.B = ctx->shape.batch;
  p.scale_log2 = ctx->scale * kLog2e;
  p.pdl_mode = ctx->overlap;
  p.variant = ctx->decode_variant == 0 ? kDecodeDefaultVariant : ctx->decode_variant;
  p.pooled = pooled ? 1 : 0;
  const cudaError_t e = launch_decode(p, *ctx->dev, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_set_overlap(sagekv_ctx *ctx, int mode) {
  if (ctx == nullptr || mode < 0 || mode > 2) return SAGEKV_ERR_INVALID;
  ctx->overlap = mode;
  return SAGEKV_OK;
}

int sagekv_set_select_overlap(sagekv_ctx *ctx, int mode) {
  if (ctx == nullptr || mode < 0 || mode > 2) return SAGEKV_ERR_INVALID;
  ctx->select_overlap = mode;
  return SAGEKV_OK;
}

int sagekv_set_decode_variant(sagekv_ctx *ctx, int variant) {
  if (ctx == nullptr || variant < 0 || variant > 2) return SAGEKV_ERR_INVALID;
  ctx->decode_variant = variant;
  return SAGEKV_OK;
}

int sagekv_set_group_mode(sagekv_ctx *ctx, int mode) {
  if (ctx == nullptr || mode < 0 || mode > 1) return SAGEKV_ERR_INVALID;
  ctx->group_mode = mode;
  return SAGEKV_OK;
}

int sagekv_pool_scores(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride, int64_t n_ctx, int32_t n_init,
                       int32_t n_recent, float *pooled, int64_t pooled_row_stride, void *stream) {
  if (ctx == nullptr || scores == nullptr || pooled == nullptr) return SAGEKV_ERR_INVALID;
  if (n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx) return SAGEKV_ERR_INVALID;
  if (n_ctx > ctx->max_ctx) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  if (scores_row_stride < E || pooled_row_stride < E) return SAGEKV_ERR_INVALID;
  if (!aligned16(scores) || !aligned16(pooled) || scores_row_stride % 4 != 0 || pooled_row_stride % 4 != 0) return SAGEKV_ERR_ALIGN;
  const cudaError_t e = launch_pool_scores(scores, scores_row_stride, pooled, pooled_row_stride, (int)E, ctx->G,
                                           ctx->shape.batch * ctx->shape.n_kv_heads, ctx->dev->n_sm,
                                           static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_compact_window_rope(sagekv_ctx *ctx, const void *K_pre, const void *V, sagekv_strides ks, int64_t n_ctx,
                               int32_t n_init, int32_t n_recent, float rope_theta, void *Kc, void *Vc, sagekv_strides cs,
                               sagekv_cache_state *state, void *stream) {
  if (ctx == nullptr || K_pre == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr || state == nullptr ||
      state->d_step == nullptr)
    return SAGEKV_ERR_INVALID;
  if (n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx || !(rope_theta > 1.f) ||
      ks.token_stride < kHeadDim || cs.token_stride < kHeadDim)
    return SAGEKV_ERR_INVALID;
  if (n_ctx > ctx->max_ctx || (int64_t)n_init + n_recent + 1 > ctx->max_len) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  if (!aligned16(K_pre) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) || !strides_ok(ks) || !strides_ok(cs))
    return SAGEKV_ERR_ALIGN;
  WindowRopeParams p;
  p.K = static_cast<const uint16_t *>(K_pre);
  p.V = static_cast<const uint16_t *>(V);
  p.ks = ks;
  p.Kc = static_cast<uint16_t *>(Kc);
  p.Vc = static_cast<uint16_t *>(Vc);
  p.cs = cs;
  p.d_step = state->d_step;
  p.status = ctx->status;
  p.S = n_init;
  p.R = n_recent;
  p.N = (int)n_ctx;
  p.H_kv = ctx->shape.n_kv_heads;
  p.B = ctx->shape.batch;
  p.theta = rope_theta;
  const cudaError_t e = launch_compact_window_rope(p, ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  state->n_init = n_init;
  state->k_q = 0;
  state->n_sel = 0;
  state->n_recent = n_recent;
  state->ring_len = n_recent + 1;
  state->len = n_init + n_recent + 1;
  return SAGEKV_OK;
}

int sagekv_quest_build(sagekv_ctx *ctx, const void *K, sagekv_strides ks, int64_t n_ctx, int32_t n_init, int32_t n_recent,
                       void *kmin, void *kmax, void *stream) {
  if (ctx == nullptr || K == nullptr || kmin == nullptr || kmax == nullptr) return SAGEKV_ERR_INVALID;
  if (n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx || ks.token_stride < kHeadDim)
    return SAGEKV_ERR_INVALID;
  if (n_ctx > ctx->max_ctx) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  if (!aligned16(K) || !aligned16(kmin) || !aligned16(kmax) || !strides_ok(ks)) return SAGEKV_ERR_ALIGN;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  const cudaError_t e = launch_quest_build(static_cast<const uint16_t *>(K), ks, static_cast<uint16_t *>(kmin),
                                           static_cast<uint16_t *>(kmax), n_init, (int)E, ctx->shape.n_kv_heads,
                                           ctx->shape.batch, ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_quest_bounds(sagekv_ctx *ctx, const void *q, const void *kmin, const void *kmax, int64_t n_blocks, float *bounds,
                        int64_t bounds_row_stride, void *stream) {
  if (ctx == nullptr || q == nullptr || kmin == nullptr || kmax == nullptr || bounds == nullptr || n_blocks < 0 ||
      bounds_row_stride < n_blocks || n_blocks > (int64_t)1 << 28)
    return SAGEKV_ERR_INVALID;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  if (!aligned16(q) || !aligned16(kmin) || !aligned16(kmax)) return SAGEKV_ERR_ALIGN;
  const cudaError_t e = launch_quest_bounds(static_cast<const uint16_t *>(q), static_cast<const uint16_t *>(kmin),
                                            static_cast<const uint16_t *>(kmax), bounds, bounds_row_stride, (int)n_blocks,
                                            ctx->G, ctx->shape.n_q_heads, ctx->shape.n_kv_heads, ctx->shape.batch, ctx->scale,
                                            ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_select_topk(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride, int64_t n, int32_t k_q, int32_t *idx,
                       void *stream) {
  if (ctx == nullptr || scores == nullptr || idx == nullptr || n < 1 || k_q < 1 || scores_row_stride < n) return SAGEKV_ERR_INVALID;
  if (n > ctx->max_ctx) return SAGEKV_ERR_UNSUPPORTED;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  if (!aligned16(scores) || scores_row_stride % 4 != 0) return SAGEKV_ERR_ALIGN;
  SelectParams p = {};
  p.scores = scores;
  p.row_stride = scores_row_stride;
  p.idx = idx;
  p.E = (int)n;
  p.N = (int)n + 1;
  p.k_q = (int)(k_q < n ? k_q : n);
  p.G = ctx->G;
  p.H_q = ctx->shape.n_q_heads;
  p.H_kv = ctx->shape.n_kv_heads;
  p.B = ctx->shape.batch;
  p.status = ctx->status;
  const cudaError_t e = launch_select_compact(p, ctx->dev->n_sm, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SAGEKV_OK : cuda_fail(ctx, e);
}

int sagekv_set_select_hint(sagekv_ctx *ctx, int mode, int32_t k) {
  if (ctx == nullptr || mode < 0 || mode > 2 || k < 0 || k % ctx->G != 0 || (mode == 2 && k == 0)) return SAGEKV_ERR_INVALID;
  ctx->hint = mode;
  ctx->hint_k = k;
  return SAGEKV_OK;
}

int64_t sagekv_scores_row_stride(const sagekv_ctx *ctx, int64_t n_ctx, int32_t n_init, int32_t n_recent) {
  if (ctx == nullptr || n_init < 0 || n_recent < 0 || n_ctx < 1 || (int64_t)n_init + n_recent + 1 > n_ctx)
    return SAGEKV_ERR_INVALID;
  const int64_t E = n_ctx - 1 - n_init - n_recent;
  int64_t stride = (E + 3) & ~(int64_t)3;
  if (stride < 4) stride = 4;
  if (ctx->hint == 1 && E >= kSketchMinE) stride += kSketchRoom;
  if (ctx->hint == 2) {
    const int64_t kq = ctx->hint_k / ctx->G;
    const int k_q = (int)(kq < E ? kq : E);
    const int64_t with_list = stride + ((list_room(k_q) + 3) & ~(int64_t)3);
    if (list_applies(E, k_q, with_list)) stride = with_list;
  }
  return stride;
}

int sagekv_status_code(int32_t bits) {
  if (bits & kStatusWaitTimeout) return SAGEKV_ERR_TIMEOUT;
  if (bits & kStatusBounds) return SAGEKV_ERR_BOUNDS;
  return SAGEKV_OK;
}

int sagekv_status(sagekv_ctx *ctx, int32_t *device_status) {
  if (ctx == nullptr) return SAGEKV_ERR_INVALID;
  if (!on_own_device(ctx)) return SAGEKV_ERR_DEVICE;
  int32_t bits = 0;
  cudaError_t e = cudaMemcpy(&bits, ctx->status, sizeof(bits), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && bits != 0) e = cudaMemset(ctx->status, 0, sizeof(bits));
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (device_status != nullptr) *device_status = bits;
  return sagekv_status_code(bits);
}

int sagekv_checked_build(void) {
#if defined(SAGEKV_CHECKS)
  return 1;
#else
  return 0;
#endif
}

const char *sagekv_strerror(int code) {
  switch (code) {
    case SAGEKV_OK: return "ok";
    case SAGEKV_ERR_INVALID: return "invalid argument";
    case SAGEKV_ERR_ALIGN: return "pointer or stride not aligned";
    case SAGEKV_ERR_UNSUPPORTED: return "unsupported shape or size";
    case SAGEKV_ERR_CUDA: return "CUDA runtime error";
    case SAGEKV_ERR_NOMEM: return "out of memory";
    case SAGEKV_ERR_TOO_LARGE: return "problem larger than the fixed scratch array";
    case SAGEKV_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case SAGEKV_ERR_BOUNDS: return "checked build: an index outside its buffer was skipped";
    case SAGEKV_ERR_DEVICE: return "the context belongs to another device than the current one";
    default: return "unknown error code";
  }
}

int sagekv_last_cuda_error(const sagekv_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

}  // extern "C"
