// K/V compaction (Algorithm 1 line 15): gather the selected rows of K and V into a
// contiguous or paged cache.  HBM-bound: every byte is read once and written once; the index
// list is read once per row.  Two kernels: compact_bulk_kernel moves rows with bulk
// asynchronous copies through shared memory (no registers are tied up while rows are in
// flight, and a contiguous destination is written with one large copy per CTA);
// compact_kernel moves them with 16-byte vector loads and stores and serves sources outside
// device memory (V left in page-locked host memory).
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

// ------------------------------------------------------ rows by bulk asynchronous copy ----

#ifndef SPEC_BULK_ROWS
#define SPEC_BULK_ROWS 16
#endif
constexpr int kBulkRows = SPEC_BULK_ROWS;         // destination rows per CTA
constexpr int kBulkThreads = kBulkRows < 32 ? 32 : kBulkRows;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// A CTA gathers kBulkRows destination rows of one (sequence, layer, KV head) for K and V: one
// bulk copy per source row into shared memory, all in flight together, then bulk copies out (a
// contiguous destination takes one per tensor, a paged one takes one per row).  Small CTAs
// and many of them: 16 rows per CTA measured best (8 to 256 tried), at 0.95 of the copy
// bandwidth on the 128K workload.
template <bool HAS_V>
__global__ void __launch_bounds__(kBulkThreads) compact_bulk_kernel(CompactParams p, int row_bytes) {
  extern __shared__ __align__(128) uint8_t rows_sm[];      // [K | V][kBulkRows][row_bytes]
  __shared__ uint64_t bar;
  const int unit = blockIdx.x / p.blocks_per_unit;
  const int rb = blockIdx.x % p.blocks_per_unit;
  const int h = unit % p.H;
  const int l = (unit / p.H) % p.L;
  const int s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int tid = threadIdx.x;
  const int c0 = rb * kBulkRows;
  const int n_rows = min(kBulkRows, p.c_max - c0);
  const uint32_t bar_a = smem_addr(&bar);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_a), "r"(kBulkRows) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  uint8_t* k_sm = rows_sm;
  uint8_t* v_sm = rows_sm + (size_t)kBulkRows * row_bytes;
  int64_t page_dst = -1;                                   // paged: element offset of my row in the pools
  if (tid < kBulkRows) {
    const int c = c0 + tid;
    int t = -1;
    bool skip = c >= p.c_max;                              // no such destination row
    if (!skip) {
      t = p.idx[(int64_t)unit * p.c_max + c];
      if (t >= n) { report(p.status, SPEC_ERR_BAD_ARG); t = -1; }
      if (p.block_table) {
        const int page = p.block_table[(int64_t)s * p.pages_per_seq + c / p.page_size];
        if (page < 0 || page >= p.n_pages) { report(p.status, SPEC_ERR_BAD_ARG); skip = true; }
        else page_dst = ((((int64_t)l * p.n_pages + page) * p.H + h) * p.page_size + c % p.page_size) * (row_bytes / 2);
      }
    }
    if (!skip && t >= 0) {
      const int64_t tok = (int64_t)begin + t;
      const uint32_t bytes = (uint32_t)row_bytes * (HAS_V ? 2u : 1u);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_addr(k_sm + (size_t)tid * row_bytes)), "l"(p.k + l * p.ksl + h * p.ksh + tok * p.kst), "r"((uint32_t)row_bytes), "r"(bar_a)
                   : "memory");
      if (HAS_V)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(v_sm + (size_t)tid * row_bytes)), "l"(p.v + l * p.vsl + h * p.vsh + tok * p.vst), "r"((uint32_t)row_bytes), "r"(bar_a)
                     : "memory");
    } else {
      // a row that is not gathered (index -1, or nothing to write) reads as zero
      int4* kz = reinterpret_cast<int4*>(k_sm + (size_t)tid * row_bytes);
      int4* vz = reinterpret_cast<int4*>(v_sm + (size_t)tid * row_bytes);
      for (int i = 0; i < row_bytes / 16; ++i) {
        kz[i] = make_int4(0, 0, 0, 0);
        if (HAS_V) vz[i] = make_int4(0, 0, 0, 0);
      }
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_a) : "memory");
      if (skip) page_dst = -1;
    }
  }
  uint32_t ok = 0;
  for (uint32_t tries = 0; tries < (1u << 20) && !ok; ++tries)
    asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\nselp.u32 %0, 1, 0, q;\n}"
                 : "=r"(ok) : "r"(bar_a) : "memory");
  if (!ok) report(p.status, SPEC_ERR_TIMEOUT);
  // the zero rows were written through the generic proxy, the copies out read through the async proxy
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (!ok) return;                                         // (a copy that never landed: nothing is written)
  if (p.block_table == nullptr) {
    if (tid == 0 || (HAS_V && tid == 1)) {
      uint16_t* out = tid == 0 ? p.k_out : p.v_out;
      const uint8_t* src = tid == 0 ? k_sm : v_sm;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                   ::"l"(out + ((int64_t)unit * p.c_max + c0) * (row_bytes / 2)), "r"(smem_addr(src)), "r"((uint32_t)(n_rows * row_bytes)) : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
  } else if (tid < kBulkRows && page_dst >= 0) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(p.k_out + page_dst), "r"(smem_addr(k_sm + (size_t)tid * row_bytes)), "r"((uint32_t)row_bytes) : "memory");
    if (HAS_V)
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                   ::"l"(p.v_out + page_dst), "r"(smem_addr(v_sm + (size_t)tid * row_bytes)), "r"((uint32_t)row_bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
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
  // Bulk copies only between device memory: a source in page-locked host memory goes through plain loads.
  bool all_device = true;
  const void* ptrs[4] = {k, v, k_out, v_out};
  for (int i = 0; i < 4 && all_device; ++i) {
    if (!ptrs[i]) continue;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, ptrs[i]) != cudaSuccess) { cudaGetLastError(); all_device = false; }
    else if (at.type != cudaMemoryTypeDevice) all_device = false;
  }
  if (all_device) {
    const int row_bytes = pr->head_dim * 2;
    const size_t smem = (size_t)kBulkRows * row_bytes * (v ? 2 : 1);
    p.blocks_per_unit = (c_max + kBulkRows - 1) / kBulkRows;
    const int64_t bulk_blocks = n_units * p.blocks_per_unit;
    if (bulk_blocks > 0x7fffffffLL) return fail(SPEC_ERR_UNSUPPORTED, "too many rows to gather in one call");
    if (smem > 48 * 1024) {
      static int set[64] = {0};
      int dev = 0;
      SPEC_CUDA_OK(cudaGetDevice(&dev));
      if (dev >= 0 && dev < 64 && !__atomic_load_n(&set[dev], __ATOMIC_ACQUIRE)) {
        SPEC_CUDA_OK(cudaFuncSetAttribute(compact_bulk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024));
        SPEC_CUDA_OK(cudaFuncSetAttribute(compact_bulk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024));
        __atomic_store_n(&set[dev], 1, __ATOMIC_RELEASE);
      }
    }
    if (v) compact_bulk_kernel<true><<<(unsigned)bulk_blocks, kBulkThreads, smem, st>>>(p, row_bytes);
    else   compact_bulk_kernel<false><<<(unsigned)bulk_blocks, kBulkThreads, smem, st>>>(p, row_bytes);
  } else if (v) {
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
