// Shared host-side helpers of the library's translation units (argument checks,
// error text) and a few device utilities.  Not part of the public interface.
#pragma once

#include <cuda_runtime.h>
#include <cstdint>
#include <cstdio>

#include "spec.h"

#define SPEC_HIDDEN __attribute__((visibility("hidden")))
#define SPEC_EXPORT extern "C" __attribute__((visibility("default")))

namespace spec {

// Records the reason of a failure for spec_last_error() and returns `code`.
SPEC_HIDDEN int fail(int code, const char* fmt, ...);
// Geometry checks common to every entry point (NULL, ranges, divisibility).
SPEC_HIDDEN int check_problem(const spec_problem* p);
// SPEC_OK when the current device is compute capability 10.x.
SPEC_HIDDEN int check_device();
// Number of SMs of the current device.
SPEC_HIDDEN int sm_count();
// Upper bound of any sequence's length known on the host.
SPEC_HIDDEN inline int max_seq_len(const spec_problem* p) {
  if (!p->cu_seqlens) return p->n_in;
  return (p->n_in > 0 && p->n_in < p->total_tokens) ? p->n_in : p->total_tokens;
}
SPEC_HIDDEN inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

// Workspace layout (bytes), shared by spec_workspace_bytes and the calls.
struct WorkspacePlan {
  int score_ctas;          // persistent grid of the scoring kernels
  size_t partial_off, partial_bytes;   // per-segment row statistics (pass 1)
  size_t rowc_off, rowc_bytes;         // per-row softmax constants
  size_t token_off, token_bytes;       // SpecPC token scores (two vectors of total_tokens floats)
  size_t sel_head_off, sel_head_bytes; // streaming selection: sel_head_words words per (sequence, layer, KV head) unit
  int sel_head_words;                  // four words, then one candidate count per chunk
  size_t sel_cand_off, sel_cand_bytes; // streaming selection: candidate (key, position) pairs
  int64_t sel_row_entries;             // candidate entries per (layer, KV head) row
  size_t total;
};
SPEC_HIDDEN WorkspacePlan plan_workspace(const spec_problem* p);
// Streaming selection: every chunk of a sequence owns a segment of the candidate array as long as
// the chunk itself (at most kSelChunkMax positions, at least kSelChunkMin), so a sequence needs
// its length plus a partial chunk; the chunks' candidate counts sit in the unit's header.
constexpr int kSelChunkMax = 2048;
constexpr int kSelChunkMin = 1024;
constexpr int kSelCandSlack = 2 * kSelChunkMax;

#define SPEC_CUDA_OK(expr)                                                              \
  do {                                                                                  \
    cudaError_t e__ = (expr);                                                           \
    if (e__ != cudaSuccess)                                                             \
      return ::spec::fail(SPEC_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__));     \
  } while (0)

// Token range of sequence s.
__device__ __forceinline__ void seq_range(const int32_t* cu, int n_in, int s, int& begin, int& n) {
  if (cu) {
    begin = cu[s];
    n = cu[s + 1] - begin;
    if (n < 0) n = 0;
  } else {
    begin = 0;
    n = n_in;
  }
}

__device__ __forceinline__ void report(int32_t* status_word, int code) {
  if (status_word) atomicCAS(status_word, 0, code);
}

}  // namespace spec
