// Host-side helpers shared by the translation units of the library: error text,
// argument checks, launch geometry.
#pragma once

#include <cstdarg>
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include "../../include/llmem.h"

namespace llmem {

// Records the text returned by llmem_last_error() for the calling thread.
void set_error(const char* fmt, ...);
void clear_error();

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// An NVTX range around an entry point's host side (argument checks and launches), so that a
// timeline shows which library call queued which kernels.  Costs a function call through a
// null pointer check when no tool is attached.
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// Number of SMs of the current device (cached per thread; 148 on B200).
int sm_count();

// Returns LLMEM_ERR_CUDA and records the text if the last launch failed.
llmem_status check_launch(const char* what);

// Layout of the scratch buffer used by llmem_scan_peak and llmem_event_counts:
// a 256-byte header whose first word is the device status, then the payload.
constexpr size_t kScratchHeader = 256;
// Byte offset, inside the header, of the 64-bit counter from which the warps of a streaming
// kernel claim their next block of work.
constexpr size_t kWorkCounterOffset = 64;

// Scratch of llmem_expand_scan: header, block starts, partials and, for lists of short
// segments, one descriptor per configuration (defined with the kernel).
size_t expand_scan_scratch_bytes(long long n, long long total_events);
// Scratch of llmem_scan_peak: the same header, block starts and partials and, for lists of short
// segments, the list of parts of the longer ones (defined with the kernels).
size_t scan_scratch_bytes(long long n, long long total_events);
// Lists whose segments are short on average are expanded by segment owners (fused.cu), which
// need that scratch; the others chunk by chunk.
bool short_segment_list(long long n, long long total_events);

}  // namespace llmem
