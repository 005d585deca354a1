// K/V compaction (Algorithm 1 line 15): gather the selected rows of K and V into a
// contiguous or paged cache with 16-byte vector copies.  HBM-bound: every byte is
// read once and written once; the index list is read once per row.
#include "common.cuh"

namespace spec {

struct CompactParams {
  const uint16_t* k;
  const uint16_t* v;
  uint16_t* k_out;
  uint16_t* v_out;
  const int32_t* idx;
  const int32_t* cu;
  const int32_t* block_table;
  int64_t ksl, ksh, kst, vsl, vsh, vst;
  int n_in, L, H, c_max, page_size, n_pages, pages_per_seq;
  int blocks_per_unit;
  int32_t* status;
};

constexpr int kCompactThreads = 256;
constexpr int kRowsPerCta = 64;

__device__ __forceinline__ int4 ld_stream(const int4* p) {
  int4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ void st_stream(int4* p, int4 v) {
  asm volatile("st.global.cs.v4.s32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// VPR = 16-byte vectors per row (head_dim*2/16).  A group of VPR adjacent lanes copies one
// row; a CTA copies kRowsPerCta destination rows of one (sequence, layer, KV head) for both
// K and V.  All loads of a thread are issued before its stores.
template <int VPR, bool HAS_V>
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(CompactParams p) {
  constexpr int ROWS_PER_PASS = kCompactThreads / VPR;
  constexpr int PASSES = kRowsPerCta / ROWS_PER_PASS;
  const int unit = blockIdx.x / p.blocks_per_unit;
  const int rb = blockIdx.x % p.blocks_per_unit;
  const int h = unit % p.H;
  const int l = (unit / p.H) % p.L;
  const int s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int lane_v = threadIdx.x % VPR;
  const int row_in_pass = threadIdx.x / VPR;
  const int c0 = rb * kRowsPerCta;

  int4 kv[PASSES], vv[PASSES];
  int64_t dst[PASSES];
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {
    const int c = c0 + i * ROWS_PER_PASS + row_in_pass;
    dst[i] = -1;
    kv[i] = make_int4(0, 0, 0, 0);
    vv[i] = make_int4(0, 0, 0, 0);
    if (c >= p.c_max) continue;
    const int t = p.idx[(int64_t)unit * p.c_max + c];
    if (t >= n) { report(p.status, SPEC_ERR_BAD_ARG); continue; }
    if (p.block_table) {
      const int page = p.block_table[(int64_t)s * p.pages_per_seq + c / p.page_size];
      if (page < 0 || page >= p.n_pages) { report(p.status, SPEC_ERR_BAD_ARG); continue; }
      dst[i] = ((((int64_t)l * p.n_pages + page) * p.H + h) * p.page_size + c % p.page_size) * (VPR * 8);
    } else {
      dst[i] = ((int64_t)unit * p.c_max + c) * (VPR * 8);
    }
    if (t >= 0) {
      const int64_t tok = (int64_t)begin + t;
      kv[i] = ld_stream(reinterpret_cast<const int4*>(p.k + l * p.ksl + h * p.ksh + tok * p.kst) + lane_v);
      if (HAS_V) vv[i] = ld_stream(reinterpret_cast<const int4*>(p.v + l * p.vsl + h * p.vsh + tok * p.vst) + lane_v);
    }
  }
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {
    if (dst[i] < 0) continue;
    st_stream(reinterpret_cast<int4*>(p.k_out + dst[i]) + lane_v, kv[i]);
    if (HAS_V) st_stream(reinterpret_cast<int4*>(p.v_out + dst[i]) + lane_v, vv[i]);
  }
}

// ------------------------------------------------------------ prompt compression ----
//
// SpecKV-PC (Section 4.3): the prompt is first cut down to the tokens SpecPC keeps, then SpecKV
// runs on the compressed prompt.  The keep list is per sequence and its length is only known on
// the device, so the compressed K/V are packed by a prefix sum of the lengths computed here.

struct GatherParams {
  const uint16_t* k;
  const uint16_t* v;
  uint16_t* k_out;
  uint16_t* v_out;
  const int32_t* keep;
  const int32_t* n_keep;
  const int32_t* cu;
  int32_t* cu_out;
  int64_t ksl, ksh, kst, vsl, vsh, vst;
  int n_in, n_seq, L, H, keep_capacity, out_tokens, blocks_per_unit;
  int32_t* status;
};

// cu_out[s] = n_keep[0] + ... + n_keep[s-1] (one thread: n_seq <= 1024).
__global__ void keep_offsets_kernel(GatherParams p) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int acc = 0;
  p.cu_out[0] = 0;
  for (int s = 0; s < p.n_seq; ++s) {
    int n = p.n_keep[s];
    if (n < 0 || n > p.keep_capacity) { report(p.status, SPEC_ERR_BAD_ARG); n = 0; }
    acc += n;
    p.cu_out[s + 1] = acc;
  }
  if (acc > p.out_tokens) report(p.status, SPEC_ERR_BAD_ARG);
}

template <int VPR, bool HAS_V>
__global__ void __launch_bounds__(kCompactThreads) gather_tokens_kernel(GatherParams p) {
  constexpr int ROWS_PER_PASS = kCompactThreads / VPR;
  constexpr int PASSES = kRowsPerCta / ROWS_PER_PASS;
  const int unit = blockIdx.x / p.blocks_per_unit;
  const int rb = blockIdx.x % p.blocks_per_unit;
  const int h = unit % p.H;
  const int l = (unit / p.H) % p.L;
  const int s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int kept = min(max(p.n_keep[s], 0), p.keep_capacity);
  const int out0 = p.cu_out[s];
  const int lane_v = threadIdx.x % VPR;
  const int row_in_pass = threadIdx.x / VPR;
  const int c0 = rb * kRowsPerCta;
  if (c0 >= kept) return;

  int4 kv[PASSES], vv[PASSES];
  int64_t dst[PASSES];
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {
    const int c = c0 + i * ROWS_PER_PASS + row_in_pass;
    dst[i] = -1;
    if (c >= kept || out0 + c >= p.out_tokens) continue;
    const int t = p.keep[(int64_t)s * p.keep_capacity + c];
    if (t < 0 || t >= n) { report(p.status, SPEC_ERR_BAD_ARG); continue; }
    dst[i] = (((int64_t)l * p.H + h) * p.out_tokens + out0 + c) * (VPR * 8);
    const int64_t tok = (int64_t)begin + t;
    kv[i] = ld_stream(reinterpret_cast<const int4*>(p.k + l * p.ksl + h * p.ksh + tok * p.kst) + lane_v);
    if (HAS_V) vv[i] = ld_stream(reinterpret_cast<const int4*>(p.v + l * p.vsl + h * p.vsh + tok * p.vst) + lane_v);
  }
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {
    if (dst[i] < 0) continue;
    st_stream(reinterpret_cast<int4*>(p.k_out + dst[i]) + lane_v, kv[i]);
    if (HAS_V) st_stream(reinterpret_cast<int4*>(p.v_out + dst[i]) + lane_v, vv[i]);
  }
}

}  // namespace spec

SPEC_EXPORT int32_t spec_compact_kv(const spec_problem* pr, const void* k, const void* v, const int32_t* idx,
                                    int32_t c_max, void* k_out, void* v_out, const int32_t* block_table,
                                    int32_t page_size, int32_t n_pages, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!k || !k_out || !idx) return fail(SPEC_ERR_BAD_ARG, "k, k_out and idx must not be NULL");
  if ((v == nullptr) != (v_out == nullptr)) return fail(SPEC_ERR_BAD_ARG, "v and v_out must both be given or both be NULL");
  if (c_max < 1) return fail(SPEC_ERR_BAD_ARG, "c_max=%d must be >= 1", c_max);
  if (block_table && (page_size < 1 || n_pages < 1))
    return fail(SPEC_ERR_BAD_ARG, "paged output needs page_size >= 1 and n_pages >= 1 (got %d, %d)", page_size, n_pages);
  if (!aligned16(k) || !aligned16(k_out) || !aligned16(v) || !aligned16(v_out))
    return fail(SPEC_ERR_ALIGNMENT, "k, v, k_out and v_out must be 16-byte aligned");
  const int64_t strides[6] = {pr->k_stride_layer, pr->k_stride_head, pr->k_stride_token,
                              pr->v_stride_layer, pr->v_stride_head, pr->v_stride_token};
  for (int i = 0; i < (v ? 6 : 3); ++i)
    if (strides[i] < 0 || (strides[i] * 2) % 16 != 0)
      return fail(SPEC_ERR_ALIGNMENT, "K/V strides must be non-negative multiples of 8 elements");
  rc = check_device();
  if (rc != SPEC_OK) return rc;

  CompactParams p;
  p.k = static_cast<const uint16_t*>(k);
  p.v = static_cast<const uint16_t*>(v);
  p.k_out = static_cast<uint16_t*>(k_out);
  p.v_out = static_cast<uint16_t*>(v_out);
  p.idx = idx;
  p.cu = pr->cu_seqlens;
  p.block_table = block_table;
  p.ksl = pr->k_stride_layer; p.ksh = pr->k_stride_head; p.kst = pr->k_stride_token;
  p.vsl = pr->v_stride_layer; p.vsh = pr->v_stride_head; p.vst = pr->v_stride_token;
  p.n_in = pr->n_in; p.L = pr->n_layers; p.H = pr->n_kv_heads; p.c_max = c_max;
  p.page_size = block_table ? page_size : 1;
  p.n_pages = n_pages;
  p.pages_per_seq = block_table ? (c_max + page_size - 1) / page_size : 0;
  p.blocks_per_unit = (c_max + kRowsPerCta - 1) / kRowsPerCta;
  p.status = status_word;
  const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;
  const int64_t blocks = n_units * p.blocks_per_unit;
  if (blocks > 0x7fffffffLL) return fail(SPEC_ERR_UNSUPPORTED, "too many rows to gather in one call");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool d128 = pr->head_dim == 128;
  if (v) {
    if (d128) compact_kernel<16, true><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
    else      compact_kernel<8, true><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
  } else {
    if (d128) compact_kernel<16, false><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
    else      compact_kernel<8, false><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
  }
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}

SPEC_EXPORT int32_t spec_gather_tokens(const spec_problem* pr, const void* k, const void* v, const int32_t* keep,
                                       int32_t keep_capacity, const int32_t* n_keep, void* k_out, void* v_out,
                                       int32_t out_tokens, int32_t* cu_seqlens_out, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!k || !k_out || !keep || !n_keep || !cu_seqlens_out)
    return fail(SPEC_ERR_BAD_ARG, "k, k_out, keep, n_keep and cu_seqlens_out must not be NULL");
  if ((v == nullptr) != (v_out == nullptr)) return fail(SPEC_ERR_BAD_ARG, "v and v_out must both be given or both be NULL");
  if (keep_capacity < 1 || out_tokens < 1) return fail(SPEC_ERR_BAD_ARG, "keep_capacity=%d and out_tokens=%d must be >= 1", keep_capacity, out_tokens);
  if (!aligned16(k) || !aligned16(k_out) || !aligned16(v) || !aligned16(v_out))
    return fail(SPEC_ERR_ALIGNMENT, "k, v, k_out and v_out must be 16-byte aligned");
  const int64_t strides[6] = {pr->k_stride_layer, pr->k_stride_head, pr->k_stride_token,
                              pr->v_stride_layer, pr->v_stride_head, pr->v_stride_token};
  for (int i = 0; i < (v ? 6 : 3); ++i)
    if (strides[i] < 0 || (strides[i] * 2) % 16 != 0)
      return fail(SPEC_ERR_ALIGNMENT, "K/V strides must be non-negative multiples of 8 elements");
  rc = check_device();
  if (rc != SPEC_OK) return rc;

  GatherParams p;
  p.k = static_cast<const uint16_t*>(k);
  p.v = static_cast<const uint16_t*>(v);
  p.k_out = static_cast<uint16_t*>(k_out);
  p.v_out = static_cast<uint16_t*>(v_out);
  p.keep = keep; p.n_keep = n_keep; p.cu = pr->cu_seqlens; p.cu_out = cu_seqlens_out;
  p.ksl = pr->k_stride_layer; p.ksh = pr->k_stride_head; p.kst = pr->k_stride_token;
  p.vsl = pr->v_stride_layer; p.vsh = pr->v_stride_head; p.vst = pr->v_stride_token;
  p.n_in = pr->n_in; p.n_seq = pr->n_seq; p.L = pr->n_layers; p.H = pr->n_kv_heads;
  p.keep_capacity = keep_capacity; p.out_tokens = out_tokens;
  p.blocks_per_unit = (keep_capacity + kRowsPerCta - 1) / kRowsPerCta;
  p.status = status_word;
  const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;
  const int64_t blocks = n_units * p.blocks_per_unit;
  if (blocks > 0x7fffffffLL) return fail(SPEC_ERR_UNSUPPORTED, "too many rows to gather in one call");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  keep_offsets_kernel<<<1, 32, 0, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  const bool d128 = pr->head_dim == 128;
  if (v) {
    if (d128) gather_tokens_kernel<16, true><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
    else      gather_tokens_kernel<8, true><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
  } else {
    if (d128) gather_tokens_kernel<16, false><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
    else      gather_tokens_kernel<8, false><<<(unsigned)blocks, kCompactThreads, 0, st>>>(p);
  }
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}
