// Error text, device queries and the entry points that are not tied to one kernel.
#include <cstdio>
#include <cstring>

#include "llmem_host.h"
#include "ranges.cuh"

namespace llmem {

static thread_local char g_error[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof g_error, fmt, ap);
  va_end(ap);
}

void clear_error() { g_error[0] = '\0'; }

int sm_count() {
  static thread_local int cached_dev = -1, cached = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev != cached_dev) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    cached = v;
    cached_dev = dev;
  }
  return cached;
}

llmem_status check_launch(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return LLMEM_ERR_CUDA;
  }
  return LLMEM_OK;
}

// Issue-rate probe: every thread advances eight independent 32-bit chains, 64 counted
// instructions per loop iteration (the loop's own counter and branch are not counted), so
// that with 64 resident warps per SM the schedulers never lack an eligible warp.
// kKind 0: add / xor (the integer ALU), 1: multiply-add, 2: the two alternating.
template <int kKind>
__global__ void __launch_bounds__(256)
int_rate_kernel(unsigned int iters, unsigned int seed, unsigned long long* __restrict__ sink) {
  unsigned int a[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = seed * (unsigned int)(j + 1) + threadIdx.x;
  const unsigned int c = seed | 1u, m = (seed >> 3) | 3u;
  for (unsigned int i = 0; i < iters; ++i) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (kKind == 0) {
          asm volatile("add.u32 %0, %0, %1;" : "+r"(a[j]) : "r"(c));
          asm volatile("xor.b32 %0, %0, %1;" : "+r"(a[j]) : "r"(m));
        } else if (kKind == 1) {
          asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(m), "r"(c));
          asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(c), "r"(m));
        } else {
          asm volatile("add.u32 %0, %0, %1;" : "+r"(a[j]) : "r"(c));
          asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(m), "r"(c));
        }
      }
    }
  }
  unsigned int x = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) x ^= a[j];
  if (x == 0x9e3779b9u && sink) atomicAdd(sink, 1ull);  // keeps the chains alive
}

}  // namespace llmem

using namespace llmem;

extern "C" llmem_status llmem_selftest_int_rate(int kind, uint32_t iters, uint64_t* sink,
                                                int64_t* warp_instructions_out, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_selftest_int_rate");
  if (kind < 0 || kind > 2 || iters < 1 || iters > (1u << 20)) {
    set_error("llmem_selftest_int_rate: kind must be 0, 1 or 2 and iters in 1 .. 2^20");
    return LLMEM_ERR_ARG;
  }
  const unsigned grid = (unsigned)sm_count() * 8u;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const unsigned seed = 0x2404u + iters;
  unsigned long long* dsink = reinterpret_cast<unsigned long long*>(sink);
  if (kind == 0) int_rate_kernel<0><<<grid, 256, 0, s>>>(iters, seed, dsink);
  else if (kind == 1) int_rate_kernel<1><<<grid, 256, 0, s>>>(iters, seed, dsink);
  else int_rate_kernel<2><<<grid, 256, 0, s>>>(iters, seed, dsink);
  if (warp_instructions_out) *warp_instructions_out = (int64_t)grid * 8 * (int64_t)iters * 64;
  return check_launch("llmem_selftest_int_rate");
}

extern "C" const char* llmem_last_error(void) { return g_error; }

extern "C" int llmem_version(void) { return 100; }

extern "C" int llmem_checked_build(void) {
#ifdef LLMEM_DEBUG
  return 1;
#else
  return 0;
#endif
}

extern "C" size_t llmem_scratch_bytes(int op, int64_t n, int64_t total_events) {
  if (n < 0) n = 0;
  switch (op) {
    case LLMEM_OP_EVENT_COUNTS:
      // header + one partial sum per block of 1024 configurations
      return kScratchHeader + (size_t)((n + 1023) / 1024 + 1) * sizeof(int64_t);
    case LLMEM_OP_EXPAND:
      // the work counter alone for lists of long segments; the descriptor table of the
      // expansion by segment owners for lists of short ones
      return short_segment_list(n, total_events) ? expand_scan_scratch_bytes(n, total_events) : kScratchHeader;
    case LLMEM_OP_SCAN_PEAK:
      // header, block starts and a head and a tail partial per block of the list; for lists of
      // short segments also the list of parts of the longer ones
      return scan_scratch_bytes(n, total_events);
    case LLMEM_OP_EXPAND_SCAN:
      // the same, plus a descriptor per configuration when the segments are short
      return expand_scan_scratch_bytes(n, total_events);
    default:
      return 0;
  }
}

extern "C" llmem_status llmem_scratch_status(const void* scratch, void* cuda_stream) {
  clear_error();
  TraceRange trace("llmem_scratch_status");
  if (!scratch) {
    set_error("llmem_scratch_status: scratch is null");
    return LLMEM_ERR_ARG;
  }
  unsigned int word = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(&word, scratch, sizeof word, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    set_error("llmem_scratch_status: %s", cudaGetErrorString(e));
    return LLMEM_ERR_CUDA;
  }
  if (word >= 16) {
    set_error("index check %u of the checked build failed; the access was skipped", word - 16);
    return LLMEM_ERR_CHECK;
  }
  if (word != 0) {
    set_error("a bounded device-side wait gave up (status word %u)", word);
    return LLMEM_ERR_TIMEOUT;
  }
  return LLMEM_OK;
}
