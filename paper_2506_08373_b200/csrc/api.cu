// Argument validation, error text and workspace sizing shared by all entry points.
#include <cstdarg>
#include <cstring>

#include "common.cuh"

namespace spec {

static thread_local char g_error[512] = "no error";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof g_error, fmt, ap);
  va_end(ap);
  return code;
}

int check_problem(const spec_problem* p) {
  if (!p) return fail(SPEC_ERR_BAD_ARG, "problem is NULL");
  if (p->n_seq < 1 || p->n_seq > 1024) return fail(SPEC_ERR_BAD_ARG, "n_seq=%d outside [1, 1024]", p->n_seq);
  if (p->total_tokens < 0) return fail(SPEC_ERR_BAD_ARG, "total_tokens=%d is negative", p->total_tokens);
  if (!p->cu_seqlens) {
    if (p->n_seq != 1) return fail(SPEC_ERR_BAD_ARG, "cu_seqlens is NULL but n_seq=%d", p->n_seq);
    if (p->n_in < 0 || p->n_in > p->total_tokens)
      return fail(SPEC_ERR_BAD_ARG, "n_in=%d outside [0, total_tokens=%d]", p->n_in, p->total_tokens);
  } else if (p->n_in < 0) {
    return fail(SPEC_ERR_BAD_ARG, "n_in=%d is negative (with cu_seqlens it is an upper bound of the sequence lengths, or 0)", p->n_in);
  }
  if (p->n_layers < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1)
    return fail(SPEC_ERR_BAD_ARG, "n_layers, n_q_heads and n_kv_heads must be >= 1");
  if (p->n_q_heads % p->n_kv_heads != 0)
    return fail(SPEC_ERR_BAD_ARG, "n_q_heads=%d is not a multiple of n_kv_heads=%d", p->n_q_heads, p->n_kv_heads);
  if (p->head_dim != 64 && p->head_dim != 128)
    return fail(SPEC_ERR_UNSUPPORTED, "head_dim=%d (supported: 64, 128)", p->head_dim);
  if (p->n_lookahead < 0 || p->n_window < 0 || p->n_lookahead + p->n_window < 1)
    return fail(SPEC_ERR_BAD_ARG, "n_lookahead=%d, n_window=%d: need both >= 0 and at least one query row",
                p->n_lookahead, p->n_window);
  if ((int64_t)p->n_seq * p->n_layers * p->n_kv_heads > (1 << 24))
    return fail(SPEC_ERR_UNSUPPORTED, "more than 2^24 (sequence, layer, KV head) units");
  return SPEC_OK;
}

int check_device() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(SPEC_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return fail(SPEC_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
  if (major != 10)
    return fail(SPEC_ERR_UNSUPPORTED, "device %d has compute capability %d.x; this library is sm_100a only", dev, major);
  return SPEC_OK;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
  if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < 64) cached[dev] = n;
  return n;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WorkspacePlan plan_workspace(const spec_problem* p) {
  WorkspacePlan w;
  memset(&w, 0, sizeof w);
  const int64_t R = p->n_lookahead + p->n_window;
  const int64_t M = R * (p->n_q_heads / p->n_kv_heads);
  const int64_t n_units = (int64_t)p->n_seq * p->n_layers * p->n_kv_heads;
  // Key tiles of 128: every sequence adds at most one ragged tile.
  const int64_t tokens = p->cu_seqlens ? p->total_tokens : p->n_in;
  const int64_t tiles_lh = tokens / 128 + p->n_seq;
  int64_t ctas = (int64_t)p->n_layers * p->n_kv_heads * tiles_lh;
  const int sms = sm_count();
  if (ctas > sms) ctas = sms;
  if (ctas < 1) ctas = 1;
  w.score_ctas = (int)ctas;
  size_t off = 0;
  w.partial_off = off;
  w.partial_bytes = (size_t)(n_units + ctas) * 4 * (size_t)M * 2 * sizeof(float);   // four epilogue warpgroups
  off = align_up(off + w.partial_bytes, 256);
  w.rowc_off = off;
  w.rowc_bytes = (size_t)p->n_seq * p->n_layers * p->n_q_heads * (size_t)R * sizeof(float);
  off = align_up(off + w.rowc_bytes, 256);
  w.token_off = off;
  w.token_bytes = 2 * (size_t)(p->total_tokens > 0 ? p->total_tokens : 1) * sizeof(float);   // token scores, and their average pool
  off = align_up(off + w.token_bytes, 256);
  w.sel_head_off = off;
  w.sel_head_words = 4 + max_seq_len(p) / kSelChunkMin + 2;
  w.sel_head_bytes = (size_t)n_units * w.sel_head_words * sizeof(int32_t);
  off = align_up(off + w.sel_head_bytes, 256);
  // candidates of sequence s of a row start at entry cu[s] + s*kSelCandSlack and may fill n_s + kSelCandSlack entries
  w.sel_row_entries = (((int64_t)p->total_tokens + 1) & ~(int64_t)1) + (int64_t)p->n_seq * kSelCandSlack + 8;
  w.sel_cand_off = off;
  w.sel_cand_bytes = (size_t)w.sel_row_entries * (size_t)p->n_layers * p->n_kv_heads * 8;
  off = align_up(off + w.sel_cand_bytes, 256);
  w.total = off;
  return w;
}

}  // namespace spec

SPEC_EXPORT size_t spec_workspace_bytes(const spec_problem* problem) {
  if (spec::check_problem(problem) != SPEC_OK) return 0;
  return spec::plan_workspace(problem).total;
}

SPEC_EXPORT const char* spec_last_error(void) { return spec::g_error; }
