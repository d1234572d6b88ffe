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

}  // namespace llmem

using namespace llmem;

extern "C" const char* llmem_last_error(void) { return g_error; }

extern "C" int llmem_version(void) { return 100; }

extern "C" size_t llmem_scratch_bytes(int op, int64_t n, int64_t total_events) {
  (void)total_events;
  if (n < 0) n = 0;
  switch (op) {
    case LLMEM_OP_EVENT_COUNTS:
      // header + one partial sum per block of 1024 configurations
      return kScratchHeader + (size_t)((n + 1023) / 1024 + 1) * sizeof(int64_t);
    case LLMEM_OP_EXPAND:
      // header only: the work counter
      return kScratchHeader;
    case LLMEM_OP_SCAN_PEAK:
    case LLMEM_OP_EXPAND_SCAN:
      // header, block starts and a head and a tail partial per block of the list
      return kStreamScratchBytes;
    default:
      return 0;
  }
}

extern "C" llmem_status llmem_scratch_status(const void* scratch, void* cuda_stream) {
  clear_error();
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
  if (word != 0) {
    set_error("a bounded device-side wait gave up (status word %u)", word);
    return LLMEM_ERR_TIMEOUT;
  }
  return LLMEM_OK;
}
