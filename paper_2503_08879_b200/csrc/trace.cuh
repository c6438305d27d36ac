// Timeline of a launch (only in a build with -DSAGEKV_TRACE; the normal build contains none of it).
//
// Thread 0 of every CTA of a traced kernel notes the global timer at up to ten points and leaves the record in a
// ring in device memory; each source file that traces a kernel has a ring of its own and exports a reader for it
// (SAGEKV_TRACE_READER).  A stamp that has to follow a computation carries a (never true) dependence on its result,
// so that it cannot be scheduled ahead of it.  Words 10 and 11 of a record: the CTA's block index; gridDim.x in the
// low half and, in the high half, bits 4..35 of an address that tells the launches of a replayed sequence apart
// (launches that overlap cannot be told apart by time).
#pragma once

#include <cuda_runtime.h>

#include "sagekv.h"

#if defined(SAGEKV_TRACE)
namespace sagekv {
constexpr int kTraceSlots = 1 << 15, kTraceStamps = 12;
static __device__ unsigned long long g_trace[kTraceSlots][kTraceStamps];
static __device__ unsigned int g_trace_n;
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
}  // namespace sagekv
#define SAGEKV_TRACE_BEGIN unsigned long long trace_t[sagekv::kTraceStamps] = {0ull};
#define SAGEKV_STAMP(i) do { if (threadIdx.x == 0) trace_t[i] = sagekv::trace_now(); } while (0)
#define SAGEKV_STAMP_AFTER(i, val_) do { if (threadIdx.x == 0) trace_t[i] = sagekv::trace_now() + (unsigned long long)((val_) == 1.2345e-33f); } while (0)
#define SAGEKV_TRACE_END(tag_) do { if (threadIdx.x == 0) { \
    const unsigned int slot_ = atomicAdd(&sagekv::g_trace_n, 1u) % sagekv::kTraceSlots; \
    trace_t[10] = ((unsigned long long)blockIdx.x << 32) | ((unsigned long long)blockIdx.y << 16) | blockIdx.z; \
    trace_t[11] = (unsigned long long)gridDim.x | ((unsigned long long)(unsigned int)((unsigned long long)(tag_) >> 4) << 32); \
    for (int i_ = 0; i_ < sagekv::kTraceStamps; ++i_) sagekv::g_trace[slot_][i_] = trace_t[i_]; } } while (0)
// Defines `name(host, n_records)`: copies the records out (host buffer of 32768 x 12 64-bit words), returns how
// many CTAs were recorded since the last call, and starts a new recording.  Synchronises the device.
#define SAGEKV_TRACE_READER(name) \
  extern "C" int name(unsigned long long *host, unsigned int *n_records) { \
    if (cudaDeviceSynchronize() != cudaSuccess) return SAGEKV_ERR_CUDA; \
    unsigned int n = 0, zero = 0; \
    if (cudaMemcpyFromSymbol(&n, sagekv::g_trace_n, sizeof(n)) != cudaSuccess) return SAGEKV_ERR_CUDA; \
    if (cudaMemcpyFromSymbol(host, sagekv::g_trace, sizeof(unsigned long long) * sagekv::kTraceSlots * sagekv::kTraceStamps) != \
        cudaSuccess) \
      return SAGEKV_ERR_CUDA; \
    if (cudaMemcpyToSymbol(sagekv::g_trace_n, &zero, sizeof(zero)) != cudaSuccess) return SAGEKV_ERR_CUDA; \
    *n_records = n; \
    return SAGEKV_OK; \
  }
#else
#define SAGEKV_TRACE_BEGIN
#define SAGEKV_STAMP(i) do { } while (0)
#define SAGEKV_STAMP_AFTER(i, val_) do { } while (0)
#define SAGEKV_TRACE_END(tag_) do { } while (0)
#define SAGEKV_TRACE_READER(name)
#endif
