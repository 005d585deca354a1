/*
 * spec.h -- C ABI of the B200 (sm_100a) lookahead-importance library.
 *
 * The library implements the data-parallel hot path of draft-based approximate
 * inference: SpecKV's lookahead importance scoring, pooling, top-C_max selection
 * and K/V compaction (Algorithm 1, lines 8-15; Eq. 1), and the SpecPC keep set
 * built on the same scores (Algorithm 2, lines 7-10).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller (any memory the
 *     device can address: device memory, or page-locked host memory mapped into
 *     the device's address space, which suits a source that is read sparsely,
 *     such as v in spec_compact_kv).  The library never allocates, frees or
 *     retains them.  Scratch memory is passed in as
 *     `workspace` (size from spec_workspace_bytes); its contents are undefined
 *     on entry and on return.
 *   - Work is enqueued asynchronously on `stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream).  The int32 return value is a
 *     spec_status: argument errors are detected on the host before anything is
 *     launched; launch failures map to SPEC_ERR_CUDA.  Nothing throws, aborts
 *     or prints; spec_last_error() gives a human-readable reason.
 *   - `status_word` (optional device int32, caller zeroes it) receives a
 *     negative spec_status if a kernel gave up on a bounded wait; read it after
 *     synchronising the stream.  The outputs of that call are then undefined.
 *   - There is no CPU fallback: on a device that is not compute capability
 *     10.x every compute entry point returns SPEC_ERR_UNSUPPORTED.
 *   - Calls that share a workspace or an output buffer must not overlap on the
 *     GPU; calls on one stream are ordered and need no host synchronisation
 *     between them.
 *
 * Notation (the paper's): n_in prompt length, R = n_window + n_lookahead query
 * rows per query head, G = n_q_heads / n_kv_heads, M = G*R query rows that
 * share one KV head, d = head_dim, L = n_layers, T = total_tokens.
 */
#ifndef SPEC_H_
#define SPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPEC_OK = 0,
  SPEC_ERR_BAD_ARG = -1,        /* NULL pointer, size out of range, inconsistent arguments */
  SPEC_ERR_ALIGNMENT = -2,      /* pointer or stride not 16-byte aligned */
  SPEC_ERR_UNSUPPORTED = -3,    /* shape outside the implemented range, or not an sm_100 device */
  SPEC_ERR_WORKSPACE = -4,      /* workspace NULL or smaller than spec_workspace_bytes() */
  SPEC_ERR_CUDA = -5,           /* a CUDA runtime / driver call failed */
  SPEC_ERR_TIMEOUT = -6         /* device side: a bounded wait expired (status_word only) */
} spec_status;

/* Reduction over query rows (spec_score) or over layers and heads (specpc_token_select). */
typedef enum {
  SPEC_REDUCE_SUM = 0,          /* Eq. 1 up to the constant 1/rows */
  SPEC_REDUCE_MAX = 1           /* Algorithm 1 line 9 / Algorithm 2 line 7 (MaxReduce) */
} spec_reduce;

typedef enum {
  SPEC_POOL_MAX = 0,            /* hyper-parameter table: SpecKV pools with Max, k = 7 */
  SPEC_POOL_AVG = 1,            /* Algorithm 1 line 10 / Algorithm 2 line 8 as printed (AvgPool1D) */
  SPEC_POOL_AVG_THEN_MAX = 2    /* specpc_token_select only: Algorithm 2 lines 8-9 in the printed order,
                                   AvgPool1D(pool_k) then MaxPool1D(n_neighbor) BEFORE the selection, so
                                   that exactly c_max tokens (plus the window) are kept; nothing is widened
                                   afterwards */
} spec_pool;

/*
 * Problem geometry shared by all calls.
 *
 * Keys and values live on a packed token axis of extent total_tokens; sequence s
 * owns tokens cu_seqlens[s] .. cu_seqlens[s+1]-1 (n_s of them; cu_seqlens is a
 * DEVICE array of n_seq+1 non-decreasing int32 with cu_seqlens[n_seq] <=
 * total_tokens).  cu_seqlens == NULL means one sequence covering tokens
 * [0, n_in).  With cu_seqlens given, the sequence lengths are only known on
 * the device; n_in is then the caller's upper bound on every n_s (it sizes
 * shared memory and picks launch shapes; 0 = no bound known, total_tokens is
 * assumed).  A sequence longer than a non-zero bound is not processed: the
 * selection calls report SPEC_ERR_BAD_ARG in status_word and return empty
 * lists for it.  Element (layer, kv_head, token, c) of K is at
 *   k + layer*k_stride_layer + kv_head*k_stride_head + token*k_stride_token + c
 * (strides in elements, bf16; the head_dim axis is contiguous); V likewise.
 * K/V base pointers and strides*2 bytes must be multiples of 16 bytes.
 */
typedef struct {
  int32_t n_seq;                /* >= 1 (<= 1024) */
  const int32_t* cu_seqlens;    /* device [n_seq+1] or NULL */
  int32_t n_in;                 /* cu_seqlens == NULL: the prompt length; else an upper bound of every n_s, or 0 */
  int32_t total_tokens;         /* T */
  int32_t n_layers, n_q_heads, n_kv_heads, head_dim;   /* head_dim in {64, 128}; n_q_heads % n_kv_heads == 0 */
  int32_t n_lookahead, n_window;                        /* R >= 1; n_lookahead may be 0 (SnapKV special case) */
  float softmax_scale;          /* > 0; Eq. 1 uses 1/sqrt(head_dim) */
  int64_t k_stride_layer, k_stride_head, k_stride_token;
  int64_t v_stride_layer, v_stride_head, v_stride_token;
} spec_problem;

/* Bytes of scratch that any of the calls below may need for this problem (0 on a bad problem). */
size_t spec_workspace_bytes(const spec_problem* problem);

/* Reason of the calling thread's last non-OK return (static storage, never NULL). */
const char* spec_last_error(void);

/*
 * Importance scores -- Eq. 1; Algorithm 1 lines 8-9 (CrossAttention of the window
 * and lookahead queries against the prompt keys, reduced over query rows).
 *
 * For every (sequence, layer, KV head) the M = G*R query rows of the GQA group are
 * scored against the sequence's keys with a per-row softmax of
 * softmax_scale * <q, k>, and the probabilities are reduced over the M rows:
 *   SPEC_REDUCE_SUM: scores[j] = sum_i w_i p_i[j]     SPEC_REDUCE_MAX: max_i w_i p_i[j]
 * The M x n_s probability matrix is never written to memory.
 *
 *  q           [n_seq, n_layers, n_q_heads, R, head_dim] bf16, contiguous, 16-byte aligned; rows are
 *              the n_window last prompt tokens in prompt order, then the lookahead tokens
 *              (Algorithm 1 line 8, "[X_m: ; Y]")
 *  k           bf16, see spec_problem
 *  row_weight  optional device float[R], w >= 0 (Algorithm 2 lines 4-6); NULL = all ones
 *  causal_window  0: every row sees every key it is given.  1: window row r only sees keys up to
 *              its own prompt position n_s - n_window + r.
 *  scores_out  [n_layers, n_kv_heads, T] fp32; the whole buffer is overwritten (tokens that no
 *              sequence covers are set to 0)
 * Query rows: up to M*head_dim = 81920 (M <= 640 at head_dim 128, 1280 at 64) are scored in one
 * sweep over the keys and the result is bit-reproducible from run to run; a larger M (a long
 * lookahead, a wide GQA group) is scored in ceil(M / that many) sweeps over equal groups of rows,
 * whose contributions are added in scores_out (SUM then rounds in an order that may differ between
 * runs, within the fp32 tolerance).
 */
int32_t spec_score(const spec_problem* problem, const void* q, const void* k, const float* row_weight,
                   int32_t reduce, int32_t causal_window, float* scores_out, void* workspace,
                   size_t workspace_bytes, int32_t* status_word, void* stream);

/*
 * Pooling + top-C_max selection -- Algorithm 1 lines 10 and 13.
 *
 * Per (sequence, layer, KV head), with e = n_s - min(n_forced_tail, n_s) eligible positions
 * [0, e): pooled[j] = pool over scores[j - pool_k/2 .. j - pool_k/2 + pool_k - 1] clipped to
 * [0, e) (stride 1; AVG divides by pool_k), the min(c_max - forced, e) positions with the largest
 * pooled value are kept (equal values: the lower position wins), and the forced tail [e, n_s) is
 * always kept (Algorithm 1 line 13: the last n_window KV pairs).  n_forced_tail = 0 selects the
 * plain top-c_max over all n_s positions.
 *
 *  scores     [n_layers, n_kv_heads, T] fp32, non-negative
 *  idx_out    [n_seq, n_layers, n_kv_heads, c_max] int32, ascending sequence-local positions,
 *             padded with -1 when fewer than c_max positions exist
 *  count_out  optional [n_seq, n_layers, n_kv_heads] int32 number of valid entries
 * Requires 1 <= pool_k <= 255, 0 <= n_forced_tail <= c_max, c_max >= 1.
 * workspace is optional (NULL, 0): the lists are the same either way.  With a workspace of
 * spec_workspace_bytes() the default pooling (SPEC_POOL_MAX, pool_k = 7) takes its fastest path
 * for sequences beyond 16384 positions, which parks candidate positions there; shorter
 * sequences with that pooling are selected in shared memory alone and need none.
 */
int32_t spec_pool_topk(const spec_problem* problem, const float* scores, int32_t pool, int32_t pool_k,
                       int32_t c_max, int32_t n_forced_tail, int32_t* idx_out, int32_t* count_out,
                       void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/*
 * Cache indices and vertical indices from one sweep -- Algorithm 1 lines 10, 11 and 13.
 *
 * Sparse prefill wants two index sets from the same pooled scores of a head: i_cache (line 13,
 * exactly what spec_pool_topk returns for c_max and n_forced_tail) and i_vert = topk(s, n_vert)
 * (line 11; the hyper-parameter table uses n_vert = 2048), the key columns every query attends
 * to in a Vertical-Slash kernel.  This call reads and pools the scores once and selects both
 * budgets from the resident pooled keys.  i_vert is taken over the eligible positions [0, e)
 * only (in Algorithm 1 the window keys carry no score); no tail is appended to it.
 *
 *  idx_out, count_out        as in spec_pool_topk
 *  vert_idx_out              [n_seq, n_layers, n_kv_heads, n_vert] int32, ascending sequence-local
 *                            positions (one sorted int32 list per head, the form a Vertical-Slash
 *                            kernel takes its vertical indices in), padded with -1
 *  vert_count_out            optional [n_seq, n_layers, n_kv_heads] int32, min(n_vert, e)
 * Requires n_vert >= 1 and the argument rules of spec_pool_topk (workspace optional, as there).
 */
int32_t spec_pool_topk_vert(const spec_problem* problem, const float* scores, int32_t pool, int32_t pool_k,
                            int32_t c_max, int32_t n_forced_tail, int32_t* idx_out, int32_t* count_out,
                            int32_t n_vert, int32_t* vert_idx_out, int32_t* vert_count_out,
                            void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/*
 * K/V compaction -- Algorithm 1 line 15 (cache <- K[i_cache], V[i_cache]).
 *
 * Row c of the compacted cache of (sequence s, layer, KV head) is source token
 * cu_seqlens[s] + idx[s, layer, head, c]; rows whose idx is -1 are zero-filled.  Rows are copied
 * bit-exactly.  v / v_out may both be NULL to gather K only.
 *
 *  block_table == NULL: k_out, v_out are [n_seq, n_layers, n_kv_heads, c_max, head_dim] bf16.
 *  block_table != NULL: k_out, v_out are page pools [n_layers, n_pages, n_kv_heads, page_size,
 *             head_dim]; slot c of sequence s goes to page block_table[s, c / page_size] (device
 *             int32 [n_seq, ceil(c_max / page_size)], assigned by the caller, each id in
 *             [0, n_pages)), row c % page_size.  Ids out of range are skipped and reported as
 *             SPEC_ERR_BAD_ARG in status_word.
 */
int32_t spec_compact_kv(const spec_problem* problem, const void* k, const void* v, const int32_t* idx,
                        int32_t c_max, void* k_out, void* v_out, const int32_t* block_table,
                        int32_t page_size, int32_t n_pages, int32_t* status_word, void* stream);

/*
 * SpecPC keep set -- Algorithm 2 lines 7-10.
 *
 * Per sequence: token score t[j] = reduce over all layers and KV heads of scores[l, h, j]
 * (`layer_head_reduce`; skip the first l_skip layers by offsetting `scores` and shrinking
 * problem->n_layers), pooled as in spec_pool_topk, top-c_max positions selected, every selected
 * position widened to [i - n_neighbor, i + n_neighbor] inside the eligible range, the forced tail
 * (the always-kept window) added, and the distinct positions written in ascending order.
 *
 *  scores      [n_layers, n_kv_heads, T] fp32 from spec_score on the draft model's Q/K
 *  keep_out    [n_seq, keep_capacity] int32, ascending, padded with -1
 *  n_keep_out  [n_seq] int32
 * keep_capacity must be >= min(max_len, c_max*(2*n_neighbor+1) + n_forced_tail) where max_len is
 * n_in when it is given (see spec_problem) and total_tokens otherwise (with
 * SPEC_POOL_AVG_THEN_MAX: min(max_len, c_max + n_forced_tail)); else SPEC_ERR_BAD_ARG.
 */
int32_t specpc_token_select(const spec_problem* problem, const float* scores, int32_t layer_head_reduce,
                            int32_t pool, int32_t pool_k, int32_t c_max, int32_t n_neighbor,
                            int32_t n_forced_tail, int32_t* keep_out, int32_t keep_capacity,
                            int32_t* n_keep_out, void* workspace, size_t workspace_bytes,
                            int32_t* status_word, void* stream);

/*
 * Prompt compression for the SpecKV-PC cascade -- Section 4.3 (SpecPC first cuts the prompt to
 * the kept tokens, then SpecKV runs on the compressed prompt).
 *
 * Gathers, for every layer and KV head, the K (and V) rows of the tokens in `keep` and packs the
 * sequences back to back: cu_seqlens_out[s] = n_keep[0] + ... + n_keep[s-1] is computed on the
 * device, so no host synchronisation is needed between specpc_token_select and the SpecKV calls
 * on the compressed prompt (pass cu_seqlens_out as the new problem's cu_seqlens, out_tokens as
 * its total_tokens and keep_capacity as its n_in bound).
 *
 *  keep            [n_seq, keep_capacity] int32 sequence-local positions, ascending (entries
 *                  beyond n_keep[s] are ignored)
 *  n_keep          [n_seq] int32
 *  k_out, v_out    [n_layers, n_kv_heads, out_tokens, head_dim] bf16; rows past the packed total
 *                  are left untouched.  v and v_out may both be NULL
 *  cu_seqlens_out  [n_seq + 1] int32, written by the call
 * A position outside its sequence, n_keep outside [0, keep_capacity] or a packed total above
 * out_tokens is skipped and reported as SPEC_ERR_BAD_ARG in status_word.
 */
int32_t spec_gather_tokens(const spec_problem* problem, const void* k, const void* v, const int32_t* keep,
                           int32_t keep_capacity, const int32_t* n_keep, void* k_out, void* v_out,
                           int32_t out_tokens, int32_t* cu_seqlens_out, int32_t* status_word, void* stream);

/*
 * specpc_token_select for callers that cannot allocate device memory.
 *
 * (No counterpart in the paper: this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option -- inside an inference server
 * whose memory pool already owns the whole device, while such a server measures its free memory,
 * or in a plugin that only ever sees the tensors of one request.  Such a caller has no buffer to
 * pass as `workspace`, so this variant keeps its only scratch, one fp32 token score per packed
 * token, in an array that is part of the library itself.  The call allocates nothing and frees
 * nothing; inputs and outputs are still the caller's.
 *
 * Limits and rules
 *   - total_tokens <= SPEC_STATIC_MAX_TOKENS, else SPEC_ERR_UNSUPPORTED (the message names the
 *     limit).  The array costs SPEC_STATIC_MAX_TOKENS * 4 bytes (1 MiB) of device memory on
 *     every GPU that loads the library, for the life of the process.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.  The array itself comes into
 *     being when the library's device code is first loaded on a device, which may be that same
 *     first call: make it before a memory pool claims the rest of the device.  The address is
 *     remembered per device; after cudaDeviceReset it is stale and the process must not call
 *     this entry point again.
 *   - SPEC_POOL_AVG_THEN_MAX is not offered (it needs a second vector): SPEC_ERR_UNSUPPORTED.
 *   - All calls on a device share the one array.  It keeps whatever the last call left there;
 *     each call rewrites every element it later reads, so results never depend on earlier
 *     calls -- but two calls that overlap on the GPU (different streams, no dependency) race
 *     on it.  Order them.
 * Otherwise arguments and results are those of specpc_token_select, minus the workspace.
 */
#define SPEC_STATIC_MAX_TOKENS 262144
int32_t specpc_token_select_static(const spec_problem* problem, const float* scores, int32_t layer_head_reduce,
                                   int32_t pool, int32_t pool_k, int32_t c_max, int32_t n_neighbor,
                                   int32_t n_forced_tail, int32_t* keep_out, int32_t keep_capacity,
                                   int32_t* n_keep_out, int32_t* status_word, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_H_ */
