// Shared device helpers and the internal launch interface of the SAGE-KV kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sagekv.h"

namespace sagekv {

constexpr int kHeadDim = 128;             // elements per row; a bf16 row is 256 bytes
constexpr int kMaxGroup = 8;              // G <= 8: one mma tile dimension holds a KV head's query heads
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ---- score ---------------------------------------------------------------
constexpr int kScoreWarps = 8;
constexpr int kScoreTokPerWarp = 32;      // two 16-token mma tiles in flight per warp
constexpr int kScoreChunk = kScoreWarps * kScoreTokPerWarp;   // tokens per CTA

struct ScoreParams {
  const uint16_t *q;       // [B, H_q, 128]
  const uint16_t *K;       // [B, H_kv, N, 128] through ks
  sagekv_strides ks;
  float *scores;           // [B*H_q rows]
  int64_t row_stride;
  float2 *partials;        // [B*H_q, n_chunks] (max, sum) in log2 units
  int n_chunks;
  int E, S, G, H_q, H_kv, B;
  float scale_log2;        // softmax scale * log2(e)
  bool sketch = false;     // leave the histogram of the group maxima behind each row that has room for it
  int64_t sketch_off = -1; // set by launch_score: where in a row it goes, or -1
  int list_k_q = 0;        // > 0: leave the candidate list for a select step with this k_q behind each row that has room
  int32_t *status = nullptr;   // status word of the context, or null (see kStatus*)
};
cudaError_t launch_score(const ScoreParams &p, int n_sm, cudaStream_t stream);

// ---- what the score step can leave behind each row for the select step -----------------------------------
// A row of E scores is cut into 8 slices of sketch_chunk(E) elements and each slice into 512 groups (16-byte
// vector v of the slice belongs to group v % 512, the last E % 4 elements to groups 0..2).  If the row has room
// for it, a histogram of the 4096 group maxima is stored at [sketch_offset(E), +512) of the row as 32-bit counts:
// 16 bins per octave, the top bin holding the row maximum, 32 octaves in all, lower maxima in bin 0.  Four
// words follow: a constant, E, the key of bin 0's lower edge >> kSketchShift, the key of the row maximum.  The
// k-th largest group maximum is a lower bound of the k-th largest score, so the select step finds its
// threshold bound by a scan of 512 counts.  It takes them only as a hint: any threshold that leaves at least
// k_q candidates is a valid one, and it checks.
constexpr int kSketchSlices = 8;
constexpr int kSketchGroups = 512;
constexpr int kSketchBins = 512;
constexpr int kSketchShift = 19;                               // key bits below a bin: 2^23 keys per octave / 16
constexpr int kSketchFloats = kSketchSlices * kSketchGroups;   // groups per row
constexpr int kSketchRoom = kSketchBins + 8;                   // 32-bit words reserved behind a row: the bins, four tag words, padding
constexpr uint32_t kSketchMagic = 0x53414745u;
constexpr int kSketchMinE = 7 * 2048 + 1;                      // rows long enough for clusters of 8 in the select step
inline __host__ __device__ int64_t sketch_offset(int64_t E) { return (E + 3) & ~(int64_t)3; }
inline __host__ __device__ int sketch_chunk(int64_t E) { return (int)((((E + kSketchSlices - 1) / kSketchSlices) + 3) & ~(int64_t)3); }
inline __host__ __device__ bool sketch_fits(int64_t E, int64_t row_stride) {
  return E >= kSketchMinE && row_stride >= sketch_offset(E) + kSketchRoom;
}

// ---- the candidate list the score step can leave behind each row for the select step ------------------------
// (hint mode 2, which the caller asks for together with the k of the coming select call.)  While it normalises a
// row the score step runs the first half of the select step's prefilter: a bound T0 not above the k_q-th largest
// score, and every score >= T0 as a candidate.  Behind the E scores (from float round_up(E,4) on): eight tag
// words, a constant, E, k_q, the number of candidates M, the key of T0, the key of the row maximum and two spare
// words, then the M candidates in position order as 64-bit words, (key << 32) | (2^32 - 1 - offset in the
// eviction region).  M = 0: no list (the prefilter did not apply to the row).  The select step ranks the list
// instead of scanning the row, and believes it: the caller vouches that the scores were not touched in between.
constexpr uint32_t kListMagic = 0x53414732u;
constexpr int kListTagWords = 8;
inline __host__ __device__ int list_cand_cap(int k_q) { return (k_q + k_q / 2 + 256) & ~1; }
inline __host__ __device__ int64_t list_room(int k_q) { return kListTagWords + 2 * (int64_t)list_cand_cap(k_q); }   // 32-bit words
// the prefilter runs on clusters of 8 CTAs of 512 threads: k_q small against the 4096 thread maxima, slices short
// enough for its tables
inline __host__ __device__ bool list_applies(int64_t E, int k_q, int64_t row_stride) {
  return E >= kSketchMinE && k_q >= 1 && 2 * (int64_t)k_q <= 8 * 512 && E <= (int64_t)8 * 16 * 8 * 512 * 4 &&
         row_stride >= sketch_offset(E) + list_room(k_q);
}

// ---- select + compact ------------------------------------------------------
struct SelectParams {
  const float *scores;
  int64_t row_stride;
  const uint16_t *K, *V;
  sagekv_strides ks;
  uint16_t *Kc, *Vc;
  sagekv_strides cs;
  int32_t *idx;            // [B, H_q, k_q]
  int32_t *d_step;
  int E, S, R, N, k_q, G, H_q, H_kv, B;
  int32_t *status = nullptr;   // status word of the context, or null
  bool sketch = false;         // the caller asked for the histograms behind the rows to be used (sagekv_set_select_hint)
  bool list = false;           // the caller vouches for the candidate lists behind the rows (hint mode 2)
  int pdl = 0;                 // 0 plain launch; 1 programmatic dependent launch; 2 also select before the dependency wait
};
cudaError_t launch_select_compact(const SelectParams &p, int n_sm, cudaStream_t stream);
cudaError_t select_compact_setup();   // one-time function attributes
// second pass of the score step in hint mode 2: normalise the rows and leave the candidate lists behind them
cudaError_t launch_score_finalize_candidates(const ScoreParams &p, cudaStream_t stream);

// ---- comparison paths (variants.cu) -----------------------------------------
struct WindowRopeParams {
  const uint16_t *K, *V;   // K before rotary embedding
  sagekv_strides ks;
  uint16_t *Kc, *Vc;
  sagekv_strides cs;
  int32_t *d_step;
  int32_t *status;
  int S, R, N, H_kv, B;
  float theta;
};
cudaError_t launch_compact_window_rope(const WindowRopeParams &p, int n_sm, cudaStream_t stream);
cudaError_t launch_pool_scores(const float *scores, int64_t row_stride, float *pooled, int64_t pooled_stride, int E, int G,
                               int n_groups, int n_sm, cudaStream_t stream);

constexpr int kDecodeDefaultVariant = 1;   // what sagekv_set_decode_variant(ctx, 0) stands for
constexpr int kQuestBlock = 16;   // tokens per block of the Quest-style summaries (SAGEKV_QUEST_BLOCK)
cudaError_t launch_quest_build(const uint16_t *K, sagekv_strides ks, uint16_t *kmin, uint16_t *kmax, int S, int E, int H_kv,
                               int B, int n_sm, cudaStream_t stream);
cudaError_t launch_quest_bounds(const uint16_t *q, const uint16_t *kmin, const uint16_t *kmax, float *u, int64_t u_stride,
                                int n_blocks, int G, int H_q, int H_kv, int B, float scale, int n_sm, cudaStream_t stream);

// ---- decode attention ------------------------------------------------------
constexpr int kDecodeWarps = 8;                                        // consumer warps per CTA (one more warp issues the copies)
constexpr int kDecodeMaxCluster = 8;                                   // CTAs per cluster (the portable limit)
constexpr int kDecodeSlots = 50;                                       // 4 KB slots of a CTA's staging area, one K or one V tile each: 200 KB (what fits beside the rest)
constexpr int kDecodeExtraClusters = 2;                                // clusters per head a launch may use beyond the fewest possible
constexpr int kDecodeMaxTiles = 44;                                    // most 16-row tiles a CTA takes: its K tiles must all be resident, and a warp keeps the scores of six
constexpr int kPartialStride = kMaxGroup * kHeadDim + 2 * kMaxGroup;   // floats per cluster result: O[8][128], m[8], l[8]

struct DecodeParams {
  const uint16_t *q;       // [B, H_q, 128]
  const uint16_t *k_new;   // [B, H_kv, 128] or null
  const uint16_t *v_new;
  uint16_t *Kc, *Vc;
  sagekv_strides cs;
  uint16_t *out;           // [B, H_q, 128]
  float *lse;              // [B, H_q] or null
  float *partials;         // [B*H_kv, clusters per head, kPartialStride]; used only with several clusters per head
  int32_t *tickets;        // [B*H_kv] arrival counters + [1] finished-heads counter, all 0 between launches
  int32_t *d_step;
  int32_t *status;         // the context's status word (see kStatus*)
  int S, k_q, n_sel, ring_len, L, G, H_q, H_kv, B;
  float scale_log2;
  int pdl_mode;            // 0 plain launch, 1 programmatic dependent launch, 2 also fetch the cache before the wait
  int variant;             // 1 warp-level mma kernel; 2 tensor-memory kernel where it applies
  int pooled;              // 1: every query head sees all selected rows of its KV head (k_q = n_sel), 0: its own segment
};

// What the one-time set-up of a device leaves behind (function attributes are set as a side effect).
struct DeviceInfo {
  int device;
  int n_sm;
  bool ready;
};
cudaError_t launch_decode(const DecodeParams &p, const DeviceInfo &dev, cudaStream_t stream);
cudaError_t decode_setup(DeviceInfo *dev);   // one-time, with the device current
void decode_geometry(int L, int heads, const DeviceInfo *dev, int *n_clusters, int *cluster_size, int *resident_tiles,
                     int *smem_bytes);

// ---- status word -------------------------------------------------------------
// One int32 in device memory per context, OR-ed into by the kernels, read by sagekv_status.
constexpr int kStatusWaitTimeout = 1;   // a bounded wait on a copy barrier gave up
constexpr int kStatusBounds = 2;        // checked build: an index outside its buffer was found and the access skipped

// In a build with -DSAGEKV_CHECKS every global-memory index of the kernels is compared with the extent the
// call was given; a violation sets kStatusBounds and the access is skipped (nothing traps).  Otherwise the
// condition is not evaluated.
#if defined(SAGEKV_CHECKS)
#define SAGEKV_OK_INDEX(status, cond) ((cond) ? true : (sagekv::note_bad_index(status), false))
#else
#define SAGEKV_OK_INDEX(status, cond) (true)
#endif

// ---- device helpers --------------------------------------------------------
#if defined(__CUDACC__)

__device__ __forceinline__ void note_bad_index(int32_t *status) {
  if (status != nullptr) atomicOr(status, kStatusBounds);
}

// 16-byte read-only load that does not linger in L1: cache rows are streamed once.
__device__ __forceinline__ uint4 ld_stream_v4(const void *ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

// plain 16-byte load (for rows another kernel on the stream may have just written)
__device__ __forceinline__ uint4 ld_v4(const void *ptr) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

__device__ __forceinline__ void st_v4(void *ptr, uint4 v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float &d0, float &d1, float &d2, float &d3, uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// order-preserving 32-bit key of a score: larger float <=> larger unsigned key; -0 and +0 share a key
__device__ __forceinline__ uint32_t score_key(float x) {
  const uint32_t u = __float_as_uint(x + 0.0f);         // -0 becomes +0: the two compare equal as numbers
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// merge two (max, sum) pairs of a running softmax kept in log2 units
__device__ __forceinline__ void merge_ml(float &m, float &l, float m2, float l2) {
  const float M = fmaxf(m, m2);
  if (M == -INFINITY) {
    l = 0.f;
  } else {
    l = l * fast_exp2(m - M) + l2 * fast_exp2(m2 - M);
  }
  m = M;
}

#endif  // __CUDACC__

}  // namespace sagekv
