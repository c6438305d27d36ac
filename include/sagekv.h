/*
 * sagekv.h -- C interface of the SAGE-KV hot path (arXiv 2503.08879, Section 2)
 * for NVIDIA B200 (sm_100a).
 *
 * The method, per transformer layer, after the prompt has been prefilled:
 *   Step 1  split the KV cache of N tokens into  sink [0,S) | eviction region
 *           [S,S+E) | recent window [S+E,N-1) | last token N-1,  E = N-1-S-R;
 *   Step 2  score the eviction region with the last token's query and keep,
 *           for every query head, the k best-scoring tokens;
 *   Step 3  build the reduced cache  C = Concat(sink, selected, recent, last);
 *   Step 4  decode on C; every new token's (k,v) enters the recent window and
 *           the oldest entry of the window leaves.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer unless its comment says "host".
 *     The library never takes ownership of a caller's buffer.
 *   - bf16 tensors are passed as `void*` / `const void*` (16-bit elements);
 *     head_dim is innermost and contiguous; head_dim must be 128.
 *   - `sagekv_strides` are in ELEMENTS.  Base pointers must be 16-byte aligned
 *     and every stride a multiple of 8 elements.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL
 *     is the default stream).  No call synchronises, and none of the three hot
 *     calls allocates.  Calls that share a context must be issued on one stream
 *     (or otherwise ordered): they share the context's scratch memory.
 *   - Return value: SAGEKV_OK (0) or a negative SAGEKV_ERR_* code.  Argument
 *     errors are found on the host before anything is launched.
 *   - A query head h reads KV head h / G, G = n_q_heads / n_kv_heads <= 8.
 *   - A context belongs to the device that was current in sagekv_create; every
 *     later call on it must find the same device current (SAGEKV_ERR_DEVICE
 *     otherwise).
 */
#ifndef SAGEKV_H_
#define SAGEKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SAGEKV_OK = 0,
  SAGEKV_ERR_INVALID = -1,     /* null pointer, negative size, S+R+1 > N, k % G != 0 ... */
  SAGEKV_ERR_ALIGN = -2,       /* pointer or stride breaks the alignment rules above     */
  SAGEKV_ERR_UNSUPPORTED = -3, /* head_dim != 128, G > 8, size beyond the context's max  */
  SAGEKV_ERR_CUDA = -4,        /* a CUDA runtime call failed (see sagekv_last_cuda_error) */
  SAGEKV_ERR_NOMEM = -5,       /* scratch allocation failed in sagekv_create             */
  SAGEKV_ERR_TOO_LARGE = -6,   /* problem exceeds the fixed scratch of sagekv_score_static */
  SAGEKV_ERR_TIMEOUT = -7,     /* sagekv_status: a bounded wait inside a kernel ran out  */
  SAGEKV_ERR_BOUNDS = -8,      /* sagekv_status, checked build: an out-of-range index was skipped */
  SAGEKV_ERR_DEVICE = -9       /* the context was created on another device than the current one */
};

typedef struct sagekv_ctx sagekv_ctx; /* opaque; owns only its scratch memory */

typedef struct {
  int32_t n_q_heads;    /* H_q                                              */
  int32_t n_kv_heads;   /* H_kv, divides H_q                                */
  int32_t head_dim;     /* d_h, must be 128                                 */
  int32_t batch;        /* independent sequences per call                   */
  float softmax_scale;  /* 0 => 1/sqrt(head_dim)                            */
} sagekv_shape;

typedef struct {
  int64_t batch_stride; /* elements between consecutive batch entries       */
  int64_t head_stride;  /* elements between consecutive KV heads            */
  int64_t token_stride; /* elements between consecutive tokens (>= head_dim)*/
} sagekv_strides;

/* Description of one layer's reduced cache.  Filled by sagekv_select_compact,
 * read by sagekv_decode_attn.  Host struct; `d_step` is a device pointer to one
 * int32 owned by the caller: the number of tokens appended so far. */
typedef struct {
  int32_t n_init;    /* S                                                    */
  int32_t k_q;       /* tokens kept per query head (after clamping to E)     */
  int32_t n_sel;     /* G * k_q selected slots per KV head                   */
  int32_t n_recent;  /* R                                                    */
  int32_t ring_len;  /* R + 1: the recent tokens and the last token          */
  int32_t len;       /* L = S + n_sel + R + 1 rows per KV head               */
  int32_t *d_step;   /* device int32, reset to 0 by sagekv_select_compact    */
} sagekv_cache_state;

/* Create / destroy a context for one shape.  `max_ctx` bounds N, `max_len`
 * bounds the reduced-cache length L of later calls; scratch for the score
 * partials and the split-K partials is allocated here (cudaMalloc on the
 * current device) and freed by sagekv_destroy.  Errors: INVALID, UNSUPPORTED,
 * NOMEM.  `*out` is NULL on failure. */
int sagekv_create(sagekv_ctx **out, const sagekv_shape *shape, int64_t max_ctx, int32_t max_len);
int sagekv_destroy(sagekv_ctx *ctx);

/* Appendix A.2, "Hyper-parameter settings": token budget B and query-group
 * number G give sink window B/4, k = B/(2G) kept tokens per query head and
 * recent window B/4.  When 2G does not divide B (the appendix's Qwen2.5 case,
 * G = 7: k = 512, recent = 8192 - 2048 - 7*512 = 2560) k is the largest power
 * of two not above B/(2G) and the slots left over go to the recent window:
 * n_recent = B - n_init - G*k_q always.  Host-only; outputs are host pointers.
 * Errors: INVALID for B < 4, G < 1 or a null pointer. */
int sagekv_budget_split(int32_t B, int32_t G, int32_t *n_init, int32_t *k_q, int32_t *n_recent);

/* Section 2, Step 2, first half: the last token's query scores every token of
 * the eviction region.  For every batch entry b, query head h and
 * eviction-region offset i in [0,E):
 *     s = scale * <q_last[b,h,:], K[b, h/G, S+i, :]>
 *     scores[b,h,i] = exp(s - max_j s_j) / sum_j exp(s_j - max_j s_j),  j in [0,E)
 * (a softmax over the eviction region only; every row sums to 1).
 *   q_last  bf16 [batch, H_q, 128], contiguous.
 *   K       bf16 [batch, H_kv, n_ctx, 128] addressed through `ks`.
 *   scores  fp32 [batch*H_q rows], row r at scores + r*scores_row_stride;
 *           scores_row_stride >= E and a multiple of 4, base 16-byte aligned.
 * bf16 products are accumulated in fp32.  E == 0 writes nothing.  Nothing
 * outside the E scores of each row is written, unless the caller has asked for
 * a hint with sagekv_set_select_hint (see there).
 * Errors: INVALID (null, n_init+n_recent+1 > n_ctx, stride < E), ALIGN,
 * UNSUPPORTED (n_ctx above the context's max_ctx), CUDA. */
int sagekv_score(sagekv_ctx *ctx, const void *q_last, const void *K, sagekv_strides ks,
                 int64_t n_ctx, int32_t n_init, int32_t n_recent,
                 float *scores, int64_t scores_row_stride, void *stream);

/* Section 2, Step 2, second half, and Step 3.  `k` is the number of selected
 * slots per KV head; it must be a multiple of G and every query head keeps
 * k_q = min(k/G, E) tokens (Step 2 selects per query head, one group of kept
 * tokens for each of the H_q heads; Appendix A.2 counts G*k selected slots in
 * the budget).  Per score row the k_q largest scores are
 * kept; of equal scores the lower position wins; the kept positions are written
 * in ascending order (token order is maintained, Appendix A.2).
 *   idx     int32 [batch, H_q, k_q] contiguous: absolute positions in [S,S+E).
 *   Kc, Vc  bf16 [batch, H_kv, >= L, 128] through `cs`; row layout per KV head g
 *           [0,S) sink | G segments of k_q rows, segment j = idx of head g*G+j |
 *           R recent tokens | last token,     L = S + G*k_q + R + 1
 *           (Step 3: C = Concat(S, E_topk, R, P_N)).  Rows are bit-exact copies.
 *   state   host struct, filled on return; state->d_step must already point to
 *           a device int32, which is set to 0 on the stream.
 *   K, V    bf16 [batch, H_kv, n_ctx, 128] through `ks`.  Only the kept, sink,
 *           recent and last rows are read, so K and V may also be left in
 *           pinned (device-addressable) host memory: the gather then moves
 *           just those rows over the bus.
 *   scores  fp32 rows as written by sagekv_score (any finite numbers select
 *           correctly).  Only the E scores of each row are read, unless the
 *           caller has asked for a hint with sagekv_set_select_hint.
 * Scores are compared as IEEE numbers (-0 equals +0); they must not be NaN.
 * Errors: INVALID (null, k < 0, k % G != 0, bad partition), ALIGN,
 * UNSUPPORTED (L above the context's max_len), CUDA. */
int sagekv_select_compact(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride,
                          const void *K, const void *V, sagekv_strides ks,
                          int64_t n_ctx, int32_t n_init, int32_t n_recent, int32_t k,
                          int32_t *idx, void *Kc, void *Vc, sagekv_strides cs,
                          sagekv_cache_state *state, void *stream);

/* Section 2, Step 4: decoding on the reduced cache, the recent window rolling
 * (a new token's key and value take the place of the window's oldest entry, so
 * the cache keeps its length).  With t = *state->d_step:
 * if k_new / v_new are non-NULL they overwrite row S + n_sel + (t mod ring_len)
 * of every KV head (row S + n_sel is the oldest recent token after compaction)
 * and *d_step becomes t+1; with both NULL nothing is appended.  Then
 *     out[b,h,:] = softmax(scale * q[b,h,:] . Kview^T) . Vview
 * where the view of head h = g*G+j is sink + segment j + window, i.e.
 * S + k_q + R + 1 rows, the reduced-cache length Step 3 states.
 *   q       bf16 [batch, H_q, 128];  k_new, v_new  bf16 [batch, H_kv, 128]
 *   out     bf16 [batch, H_q, 128];  lse  fp32 [batch, H_q] or NULL (natural-log
 *           of the softmax denominator, max included)
 * The cache is streamed once in split-K partitions whose partial results are
 * merged by log-sum-exp inside the same launch; products and sums are fp32,
 * softmax weights are rounded to bf16 before they multiply V.
 * Errors: INVALID (null, exactly one of k_new/v_new NULL), ALIGN,
 * UNSUPPORTED (state->len above the context's max_len), CUDA. */
int sagekv_decode_attn(sagekv_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                       void *Kc, void *Vc, sagekv_strides cs, const sagekv_cache_state *state,
                       void *out, float *lse, void *stream);

/* How sagekv_decode_attn launches overlap with the kernel before them on the
 * stream.  Step 4 runs once per layer and per generated token, so at batch 1 the
 * launch-to-launch gap is a large share of its cost.  (The score launches are
 * always plain; sagekv_set_select_overlap covers select+compact.)
 *   0  (default) plain launch: starts when the previous kernel has finished.
 *   1  programmatic dependent launch: the kernel may be scheduled while its
 *      predecessor drains, and waits on the device for the predecessor to
 *      finish before it reads or writes anything.  Always safe.
 *   2  as 1, but the rows of the reduced cache are requested BEFORE that wait.
 *      Only for callers who guarantee that the kernel directly before a
 *      sagekv_decode_attn call on the stream does not write the Kc / Vc passed
 *      to that call (for example a decode call for another layer, or work that
 *      only produces q, k_new, v_new).  q, k_new, v_new and the step counter
 *      are still read after the wait.
 * Errors: INVALID for a null context or a mode outside 0..2. */
int sagekv_set_overlap(sagekv_ctx *ctx, int mode);

/* Which kernel sagekv_decode_attn launches.  Both compute the same thing to the
 * same tolerance (Section 2, Step 4).
 *   0  (default) the library's choice: 1.
 *   1  warp-level tensor-core instructions fed through shared-memory loads; every
 *      cache length.
 *   2  the tensor cores' own path (operands read from shared memory by the tensor
 *      core, accumulators in tensor memory) where it applies: one cluster per KV
 *      head and at most 22 tiles of 16 rows per CTA (reduced caches up to 2816
 *      rows with clusters of 8); longer caches run as 1.  With the 4 to 8 query
 *      heads of a KV head as the only useful columns it is the slower one
 *      (measured: the tensor core spends one clock per operand row and k-step
 *      however few columns there are), and it is kept as a checked alternative.
 * Errors: INVALID for a null context or a variant outside 0..2. */
int sagekv_set_decode_variant(sagekv_ctx *ctx, int variant);

/* The same choice for the launches of sagekv_select_compact, sagekv_select_topk
 * and the pooled selection (Section 2, Steps 2 and 3), which run once per layer
 * after prefill and last a few microseconds each, so that with many layers queued
 * on a stream the gaps between them weigh as much as the work.
 *   0  (default) plain launch.
 *   1  programmatic dependent launch; the kernel waits on the device for its
 *      predecessor before it reads or writes anything a program can observe (it
 *      may ask for the candidate list to be brought into L2 earlier).  Always safe.
 *   2  as 1, but with a trusted candidate list (select hint mode 2) the wait is
 *      put off until the kernel's first WRITE: the list, K and V are read, and
 *      the selection is made, while the predecessor may still be running.  Only
 *      for callers who guarantee that the kernel directly before the call on the
 *      stream writes none of the call's inputs (scores with their lists, K, V):
 *      for example the select call of another layer, when the score calls of all
 *      layers were queued first.
 * Launches that do not start from a candidate list (select hint modes 0 and 1)
 * pass over the score rows and are always plain, whatever the mode.
 * Errors: INVALID for a null context or a mode outside 0..2. */
int sagekv_set_select_overlap(sagekv_ctx *ctx, int mode);

/* How the G query heads of a KV head share its selected slots.
 *   0  (default, the paper's reading: Step 2 selects per query head and the
 *      budget of Appendix A.2 counts G*k slots) every query head keeps its own
 *      k/G tokens and attends to the sink, its own segment and the window.
 *   1  pooled: sagekv_select_compact expects ONE score row per KV head
 *      (batch*H_kv rows, e.g. from sagekv_pool_scores), keeps the k best tokens
 *      of it (idx is [batch, H_kv, min(k,E)], k need not divide by G), and in
 *      sagekv_decode_attn every query head attends to all L rows of its KV
 *      head's cache.  The hints of sagekv_set_select_hint do not apply.
 * A reduced cache must be decoded in the mode it was built in.
 * Errors: INVALID (null context, unknown mode). */
int sagekv_set_group_mode(sagekv_ctx *ctx, int mode);

/* For group mode 1: pooled[b*H_kv + g][i] = sum over the G query heads h of KV
 * head g of scores[b*H_q + h][i], i in [0,E), added in head order in fp32.
 *   scores  fp32, batch*H_q rows of stride scores_row_stride, as sagekv_score
 *           writes them;  pooled  fp32, batch*H_kv rows of stride
 *           pooled_row_stride (>= E, a multiple of 4; base 16-byte aligned).
 * Errors: INVALID, ALIGN, UNSUPPORTED (n_ctx above max_ctx), DEVICE, CUDA. */
int sagekv_pool_scores(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride, int64_t n_ctx,
                       int32_t n_init, int32_t n_recent, float *pooled, int64_t pooled_row_stride, void *stream);

/* Section 3.1 "Baselines", StreamLLM_R, and Appendix A.1: the cache of a
 * sliding-window method that stores keys BEFORE rotary position embedding and
 * counts positions inside the kept window.  Builds the reduced cache of
 * sink + recent + last token (no selection: L = S + R + 1 rows per KV head)
 * from a pre-RoPE key cache, rotating the key that lands in row r by position r:
 *     a_i = r * rope_theta^(-2i/128),   i in [0,64)
 *     Kc[r][i]      = K[t][i] cos(a_i) - K[t][i+64] sin(a_i)
 *     Kc[r][i + 64] = K[t][i+64] cos(a_i) + K[t][i] sin(a_i)
 * (dimension i paired with i + 64), t = r for r < S, else n_ctx - L + r;
 * computed in double precision, rounded once to bf16.  V rows are copied
 * verbatim.  `state` is filled as by sagekv_select_compact with k = 0 and
 * *d_step is set to 0, so sagekv_decode_attn can run on the result; rows
 * appended later are stored as given (the caller rotates new keys).
 * Errors: INVALID (null, bad partition, rope_theta <= 1), ALIGN, UNSUPPORTED
 * (n_ctx above max_ctx, L above max_len), DEVICE, CUDA. */
int sagekv_compact_window_rope(sagekv_ctx *ctx, const void *K_pre, const void *V, sagekv_strides ks,
                               int64_t n_ctx, int32_t n_init, int32_t n_recent, float rope_theta,
                               void *Kc, void *Vc, sagekv_strides cs, sagekv_cache_state *state, void *stream);

/* ---- A Quest-style comparator (Section 3.1 "Baselines": a block-wise top-k
 * selection method; Section 3.2 compares memory efficiency with it).  It keeps
 * the FULL cache and selects blocks anew at every decode step; these three calls
 * are its selection half, on the same data layout as the method's own calls.
 *
 * sagekv_quest_build: per block of SAGEKV_QUEST_BLOCK = 16 consecutive tokens of
 * the eviction region (the last block may be shorter), the element-wise minimum
 * and maximum of the keys.  kmin, kmax  bf16 [batch, H_kv, n_blocks, 128]
 * contiguous, n_blocks = ceil(E / 16); exact (no rounding).  Built once.
 * Errors: INVALID, ALIGN, UNSUPPORTED (n_ctx above max_ctx), DEVICE, CUDA. */
#define SAGEKV_QUEST_BLOCK 16
int sagekv_quest_build(sagekv_ctx *ctx, const void *K, sagekv_strides ks, int64_t n_ctx, int32_t n_init,
                       int32_t n_recent, void *kmin, void *kmax, void *stream);

/* Per decode step: bounds[b*H_q + h][j] = scale * sum_c max(q[b,h,c]*kmin[b,h/G,j,c],
 * q[b,h,c]*kmax[b,h/G,j,c]), an upper bound of the attention logit of every token of
 * block j (fp32 products and sums).  bounds: batch*H_q rows of stride
 * bounds_row_stride >= n_blocks.  Errors: INVALID, ALIGN, DEVICE, CUDA. */
int sagekv_quest_bounds(sagekv_ctx *ctx, const void *q, const void *kmin, const void *kmax, int64_t n_blocks,
                        float *bounds, int64_t bounds_row_stride, void *stream);

/* The selection of sagekv_select_compact without the gather: per row of `scores`
 * (batch*H_q rows of n values, stride scores_row_stride, a multiple of 4; base
 * 16-byte aligned) the min(k_q, n) largest, lower index winning ties, written
 * ascending as 0-based indices to idx [batch*H_q, min(k_q, n)].  n may not exceed
 * the context's max_ctx.  Used for the comparator's block selection.
 * Errors: INVALID, ALIGN, UNSUPPORTED, DEVICE, CUDA. */
int sagekv_select_topk(sagekv_ctx *ctx, const float *scores, int64_t scores_row_stride, int64_t n,
                       int32_t k_q, int32_t *idx, void *stream);

/* Optional hint from the score step to the select step (no counterpart in the
 * paper; it changes no result).  Off by default: sagekv_score then writes, and
 * sagekv_select_compact reads, nothing but the E scores of each row, whatever
 * the row stride, so rows may be interleaved with other data of the caller.
 *   mode 0  off.
 *   mode 1  for rows of at least 14337 scores sagekv_score also writes, behind
 *           the E scores of every row (from float round_up(E,4) on), a 512-bin
 *           histogram of the maxima of 4096 groups of that row's scores and four
 *           tag words (516 32-bit words), and sagekv_select_compact takes its
 *           first threshold bound from that histogram instead of a pass over
 *           the scores.  It verifies the outcome, so scores changed in between,
 *           or any other content of those words, still select correctly, only
 *           slower.  The caller must give both calls a row stride of at least
 *           sagekv_scores_row_stride() and a buffer that spans
 *           batch*H_q * stride floats; both calls use the words only when the
 *           stride leaves room for them.
 *   mode 2  the caller also passes the `k` that the coming
 *           sagekv_select_compact calls will be given.  While it normalises a
 *           row of at least 14337 scores, sagekv_score then runs the first half
 *           of the selection on it (a bound not above the k/G-th largest score of
 *           the row, and every score at or above the bound as a candidate) and
 *           writes, behind the E scores of every row, eight tag words and the
 *           candidates in position order as 64-bit words, at most
 *           1.5*(k/G) + 256 of them; sagekv_scores_row_stride() gives the stride
 *           that leaves room.  sagekv_select_compact, called with the same k,
 *           buffer and stride, ranks that list instead of reading the row.
 *           It BELIEVES the list: the caller vouches that the scores, and the
 *           words behind them, are exactly what sagekv_score wrote.  Scores
 *           edited in between are not noticed (use mode 0 or 1 for scores from
 *           anywhere else).  With another k, a stride without the room, or
 *           shorter rows, both calls behave as in mode 0.  Same results as
 *           mode 0 on the scores sagekv_score wrote.
 * In modes 0 and 1 `k` is ignored.  The setting applies to later calls on the
 * context.  Errors: INVALID (null context, unknown mode, k < 0, k not a multiple
 * of G, mode 2 with k = 0). */
int sagekv_set_select_hint(sagekv_ctx *ctx, int mode, int32_t k);

/* Smallest scores_row_stride (in floats, a multiple of 4) that holds a row of
 * E = n_ctx - 1 - n_init - n_recent scores plus whatever the context's hint
 * mode keeps behind it.  Host-only.  Negative: SAGEKV_ERR_INVALID. */
int64_t sagekv_scores_row_stride(const sagekv_ctx *ctx, int64_t n_ctx, int32_t n_init, int32_t n_recent);

/* Device-side status of the context.  The kernels never trap: a wait on a copy
 * that does not arrive within its (generous) bound, or, in a library built
 * with -DSAGEKV_CHECKS, a global-memory index outside the extent the call was
 * given (the access is skipped), sets a bit in one int32 of context-owned device
 * memory and the kernel runs to its end.  This call copies that word to
 * *device_status (may be NULL), clears it, and returns sagekv_status_code() of
 * it.  It synchronises (a blocking 4-byte copy): call it after synchronising
 * the streams the context was used on, never inside a stream capture.
 * Errors: INVALID (null context), DEVICE, CUDA, or the word's own code. */
int sagekv_status(sagekv_ctx *ctx, int32_t *device_status);

/* The return code that belongs to a status word: SAGEKV_OK for 0,
 * SAGEKV_ERR_TIMEOUT if bit 0 is set, else SAGEKV_ERR_BOUNDS if bit 1 is set.
 * Host-only, needs no device. */
int sagekv_status_code(int32_t device_status);

/* 1 if the library was built with -DSAGEKV_CHECKS (index checks in every
 * kernel, slower), else 0. */
int sagekv_checked_build(void);

/* The score step without any allocation (the paper has no counterpart: this is
 * a deployment variant of sagekv_score, same arithmetic, same kernels, same
 * output).  It exists for programs that cannot call cudaMalloc when they reach
 * this step: inference servers hand nearly all device memory to their own
 * cache manager at start-up, so the cudaMalloc inside sagekv_create may fail
 * there, and it synchronises the whole device, which a serving loop with other
 * streams in flight cannot afford.  This call needs no context: the softmax
 * partials live in a fixed 256 KiB array inside the library image (present on
 * every GPU that loads the library, until the process ends).
 *   - Limit: batch * H_q * ceil(E / 256) <= 32768 partial entries; beyond it the
 *     call returns SAGEKV_ERR_TOO_LARGE and launches nothing (E = 131072-class
 *     contexts fit up to batch * H_q = 64).
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call outside any
 *     stream capture.  Later calls only launch.
 *   - All calls on a device share the array.  It needs no clearing (each entry
 *     is written before it is read within a call), but two calls whose kernels
 *     overlap on the GPU (different streams) race on it: keep them ordered.
 * Arguments, layouts, alignment rules and the other error codes are those of
 * sagekv_score, with `shape` taking the place of the context. */
int sagekv_score_static(const sagekv_shape *shape, const void *q_last, const void *K, sagekv_strides ks,
                        int64_t n_ctx, int32_t n_init, int32_t n_recent,
                        float *scores, int64_t scores_row_stride, void *stream);

/* Text for a return code; never NULL.  Static storage. */
const char *sagekv_strerror(int code);

/* The cudaError_t value of the most recent failing CUDA call made through
 * `ctx` (0 if none), for diagnosing SAGEKV_ERR_CUDA. */
int sagekv_last_cuda_error(const sagekv_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SAGEKV_H_ */
