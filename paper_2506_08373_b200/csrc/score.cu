// Lookahead importance scoring (Eq. 1; Algorithm 1 lines 8-9) on tcgen05 tensor cores.
//
// score[j] = reduce_i softmax_j(scale * q_i . k_j) over the M = G*R query rows that share a
// KV head.  The M x n probability matrix never leaves the SM:
//   pass 1   S = Q K^T per 128-key tile (query rows on TMEM lanes): running row max and
//            sum-exp, kept per thread, written per (CTA, unit) segment;
//   merge    combines the segments' statistics into one constant per row,
//            c_i = log2e*scale*max_i + log2 Z_i - log2 w_i;
//   pass 2   S^T = K Q^T per tile (keys on TMEM lanes, query rows on columns):
//            p = exp2(scale*log2e*S - c_i), reduced over columns thread-locally, one reduction per key
//            and warpgroup.
// Both passes are persistent, warp-specialised kernels: warp 0 feeds K tiles (and the unit's Q)
// with TMA into a shared-memory ring, two threads issue tcgen05.mma into TMEM, and four epilogue
// warpgroups (16 warps, four per SM sub-partition) drain the accumulators with tcgen05.ld and
// do the exponentials.  Every warpgroup owns one 128-column TMEM buffer.  A work item is
// 128 x 128 logits: 128 query rows x the 128 keys of a tile in pass 1, the 128 keys of a tile x
// a chunk of 128 query rows in pass 2.  Key tiles alternate between the two pairs of
// warpgroups (each pair has its own issuing thread); within a pair the items of a tile
// alternate between its two warpgroups, which start alternately from tile to tile.  A
// warpgroup drains an item whole, four 32-column loads with the arithmetic in between, and
// hands the buffer back after the last load, so the four warps that share an SM
// sub-partition run out of step with one another.
// The exponential is the scarce resource (16 MUFU results per clock per SM against 32 logits per
// clock from the tensor cores), so a fixed share of the elements is evaluated on the FMA pipes
// instead (range reduction + cubic polynomial, relative error 7.5e-5), and the surrounding
// arithmetic uses the packed two-lane fp32 instructions to halve its issue slots.  Warpgroups
// never synchronise inside a unit: pass 1 writes their statistics as separate partials; in
// pass 2 a key tile belongs to one pair, whose two warpgroups add their per-key sums (over the
// chunks each of them drained) into the zero-filled output with one reduction each (two
// addends, so the result does not depend on their order).  More query rows than fit in shared
// memory are scored in several launches over groups of rows (ScoreParams::row0), each adding
// into the same output.
// The global key-tile space (layer, KV head, sequence, tile) is cut into equal contiguous
// ranges, one per CTA.
//
// Every wait on an mbarrier is bounded in time; on expiry the CTA reports SPEC_ERR_TIMEOUT
// through the status word, lets its copies land, frees its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include <algorithm>

namespace spec {

constexpr int kEpilogueWarpgroups = 4;
constexpr int kEpilogueThreads = kEpilogueWarpgroups * 128;
constexpr int kMmaWarpB = 2 + kEpilogueThreads / 32;    // second MMA-issuing warp, after the epilogue warps
constexpr int kThreads = 64 + kEpilogueThreads + 32;
#ifndef SPEC_POLY_PAIRS_1
#define SPEC_POLY_PAIRS_1 4
#endif
#ifndef SPEC_POLY_PAIRS_2
#define SPEC_POLY_PAIRS_2 4
#endif
// of the 16 element pairs in a 32-element block, evaluated on the FMA pipes (pass 1, pass 2)
constexpr int kPolyPairs1 = SPEC_POLY_PAIRS_1, kPolyPairs2 = SPEC_POLY_PAIRS_2;
constexpr int kBufCols = 128;                 // TMEM columns of a pass-2 accumulator buffer (pass 1 uses two of 256)
constexpr int kTileKeys = 128;
constexpr int kMaxStages = 8;
constexpr int kMaxMTiles = 10;
constexpr int kNumBars = 2 * kMaxStages + 2 + 8;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
#ifndef SPEC_SUSPEND_HINT_NS
#define SPEC_SUSPEND_HINT_NS 100000
#endif
constexpr uint32_t kSuspendHintNs = SPEC_SUSPEND_HINT_NS;

struct ScoreParams {
  const int32_t* cu;
  const float* row_weight;
  float* partial;       // [n_units + n_ctas][4 warpgroups][M][2]  (max in log2 domain, sum-exp)
  float* rowc;          // [n_seq*L*Hq*R]  minus the per-row constant
  float* scores;        // [L, Hkv, T]
  int32_t* status;
  long long T;
  int n_in, n_seq, L, Hq, Hkv, G, R, M, M_pad, d;   // M, M_pad: the query rows of this launch, rows [row0, row0 + M) of every unit
  int row0;
  int causal, n_window;  // causal != 0: window row r sees keys up to position n - n_window + r only
  int n_stages, n_chunks, cw_last;   // pass 2: chunks of 128 query rows, the last of cw_last (64 or 128)
  int reduce;
  float a;              // softmax_scale * log2(e)
  uint32_t q_bytes, stage_bytes;
};

// ------------------------------------------------------------------ PTX wrappers ------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One arrival for the whole warp, after a warp-wide (.sync.aligned) instruction has completed
// for all lanes: predicated, no branch.
__device__ __forceinline__ void arrive_lane0(uint64_t* bar, int lane) {
  asm volatile("{\n.reg .pred p;\nsetp.eq.s32 p, %1, 0;\n@p mbarrier.arrive.shared::cta.b64 _, [%0];\n}"
               ::"r"(smem_u32(bar)), "r"(lane) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when another role has given up or the time limit passed.  The
// suspend-time hint lets the hardware park the thread until the phase completes instead of
// spinning in the issue slots the epilogue warps need.
__device__ __forceinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t addr = smem_u32(bar);
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(addr), "r"(parity), "r"(kSuspendHintNs) : "memory");
    if (ok) return true;
    if ((it & 7u) == 0) {                                   // every failed wait already lasted up to the hint
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

// The common case, a phase that has already completed, costs one non-blocking test inline.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  if (ok) return true;
  return mbar_wait_slow(bar, parity, abort_flag);
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int x, int y, int z, int w, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulation, issued by one thread.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane, complete on return (the load and
// the wait for it are one statement, so no use of the registers can be scheduled in between).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor: K-major operand, rows of 64 bf16 (128 bytes) with the
// 128-byte swizzle TMA writes; 8-row groups are 1024 bytes apart.  Only the start address
// (bits 0-13, in 16-byte units) differs between the operands of this kernel, so the issuing
// thread keeps the low word per operand and adds offsets to it; the high word is constant.
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4)        // stride byte offset between 8-row groups
                             | (1u << 14)                 // descriptor version of this architecture
                             | (2u << 29);                // 128-byte swizzle
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr) {
  return ((saddr & 0x3FFFFu) >> 4) | (1u << 16);          // leading byte offset (unused for swizzled K-major)
}
__device__ __forceinline__ uint64_t desc_at(uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; }
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__device__ __forceinline__ uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// ------------------------------------------------------------- work decomposition -----

struct Seg {
  int unit;        // ordinal (layer*Hkv + head)*n_seq + seq
  int s, l, h;
  int begin, n;    // token range of the sequence
  int t0, nt;      // first key tile of the unit handled here, number of tiles
};

struct SegIter {
  long long g, g_end;
  int TT;
};

// Tile-count prefix over sequences, tp[0..n_seq].
__device__ void build_tile_prefix(const ScoreParams& p, int* tp) {
  int acc = 0;
  tp[0] = 0;
  for (int s = 0; s < p.n_seq; ++s) {
    int b, n;
    seq_range(p.cu, p.n_in, s, b, n);
    acc += (n + kTileKeys - 1) / kTileKeys;
    tp[s + 1] = acc;
  }
}

__device__ __forceinline__ SegIter seg_begin(const ScoreParams& p, const int* tp, int n_ctas, int cta) {
  SegIter it;
  it.TT = tp[p.n_seq];
  const long long N = (long long)p.L * p.Hkv * it.TT;
  const long long P = (N + n_ctas - 1) / n_ctas;
  it.g = P * cta;
  it.g_end = it.g + P < N ? it.g + P : N;
  return it;
}

__device__ bool seg_next(SegIter& it, const ScoreParams& p, const int* tp, Seg& sg) {
  if (it.g >= it.g_end) return false;
  const int lh = (int)(it.g / it.TT);
  const int rem = (int)(it.g % it.TT);
  int lo = 0, hi = p.n_seq;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tp[mid] <= rem) lo = mid; else hi = mid;
  }
  sg.s = lo;
  sg.l = lh / p.Hkv;
  sg.h = lh % p.Hkv;
  sg.unit = lh * p.n_seq + lo;
  sg.t0 = rem - tp[lo];
  const long long left = it.g_end - it.g;
  const int in_unit = tp[lo + 1] - rem;
  sg.nt = left < in_unit ? (int)left : in_unit;
  seq_range(p.cu, p.n_in, lo, sg.begin, sg.n);
  it.g += sg.nt;
  return true;
}

// ------------------------------------------------------------------ epilogue math -----

// The packed fp32 instructions (two lanes per instruction) through the float2 intrinsics.
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 2^x for both lanes on the MUFU unit.
__device__ __forceinline__ float2 ex2_mufu2(float2 x) {
  return make_float2(ex2(x.x), ex2(x.y));
}
// 2^x for both lanes without the MUFU unit: x = n + f with n = round(x), |f| <= 1/2 (adding
// 1.5 * 2^23 leaves n in the low mantissa bits), 2^f by a cubic with relative error 7.5e-5,
// then n is added into the exponent field.  x is clamped at -125 so the exponent cannot wrap.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
  x = make_float2(fmaxf(x.x, -125.f), fmaxf(x.y, -125.f));
  const float2 xr = __fadd2_rn(x, splat2(12582912.f));
  const float2 n = __fadd2_rn(xr, splat2(-12582912.f));
  const float2 f = __ffma2_rn(n, splat2(-1.f), x);
  float2 q = __ffma2_rn(f, splat2(0.0551713221f), splat2(0.2426105440f));
  q = __ffma2_rn(q, f, splat2(0.6932609677f));
  q = __ffma2_rn(q, f, splat2(0.9999281168f));
  return make_float2(__uint_as_float(__float_as_uint(q.x) + (__float_as_uint(xr.x) << 23)),
                     __uint_as_float(__float_as_uint(q.y) + (__float_as_uint(xr.y) << 23)));
}
// Pair i (0..15) of a 32-element block: NP of them, evenly spread, avoid the MUFU unit.
template <int NP>
__device__ __forceinline__ float2 ex2_pair(float2 x, int i) {
  return (i * NP) / 16 != ((i + 1) * NP) / 16 ? ex2_poly2(x) : ex2_mufu2(x);
}

// Pass 1: fold 32 logits of one row into the running (max, sum-exp), log2 domain.  At least one
// of the 32 logits is valid.
template <bool MASKED>
__device__ __forceinline__ void stats_update(const uint32_t (&r)[32], int valid, float a, float& m, float& z) {
  float v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    v[i] = __uint_as_float(r[i]);
    if (MASKED && i >= valid) v[i] = -INFINITY;
  }
  float g[11];
#pragma unroll
  for (int i = 0; i < 10; ++i) g[i] = max3(v[3 * i], v[3 * i + 1], v[3 * i + 2]);
  g[10] = fmaxf(v[30], v[31]);
  const float g0 = max3(g[0], g[1], g[2]), g1 = max3(g[3], g[4], g[5]), g2 = max3(g[6], g[7], g[8]);
  const float gm = max3(max3(g0, g1, g2), g[9], g[10]);
  const float mn = fmaxf(m, gm * a);                       // a > 0
  z *= ex2(m - mn);                                        // first block: 0 * 2^-inf = 0
  m = mn;
  const float2 a2 = splat2(a), neg2 = splat2(-mn);
  float2 s0 = splat2(0.f), s1 = splat2(0.f);
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    s0 = __fadd2_rn(s0, ex2_pair<kPolyPairs1>(__ffma2_rn(make_float2(v[2 * i], v[2 * i + 1]), a2, neg2), i));
    s1 = __fadd2_rn(s1, ex2_pair<kPolyPairs1>(__ffma2_rn(make_float2(v[2 * i + 2], v[2 * i + 3]), a2, neg2), i + 1));
  }
  z += (s0.x + s0.y) + (s1.x + s1.y);
}

// Pass 2: probabilities of 32 query rows for this thread's key, reduced into acc (two packed
// partial sums, or two packed maxima).
template <bool MAXRED>
__device__ __forceinline__ void prob_accumulate(const uint32_t (&r)[32], const float* __restrict__ negc, float2 a2, float2 (&acc)[2]) {
  const float4* c4 = reinterpret_cast<const float4*>(negc);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 c = c4[i];
    const float2 p0 = ex2_pair<kPolyPairs2>(__ffma2_rn(make_float2(__uint_as_float(r[4 * i + 0]), __uint_as_float(r[4 * i + 1])), a2, make_float2(c.x, c.y)), 2 * i);
    const float2 p1 = ex2_pair<kPolyPairs2>(__ffma2_rn(make_float2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), a2, make_float2(c.z, c.w)), 2 * i + 1);
    if (MAXRED) {
      acc[0].x = max3(acc[0].x, p0.x, p0.y);               // one maximum per chain: the four are merged at the end
      acc[1].x = max3(acc[1].x, p1.x, p1.y);
    } else {
      acc[0] = __fadd2_rn(acc[0], p0);
      acc[1] = __fadd2_rn(acc[1], p1);
    }
  }
}

// The same for a key tile that reaches into the causal window: the probability of query row
// (row0 + i) for this thread's key (position `key` of a sequence of n) is dropped when the row
// is window row r < n_window and the key lies after the row's own position n - n_window + r.
// Plain scalar code: only the last tile or two of a sequence come here.
template <bool MAXRED>
__device__ __forceinline__ void prob_accumulate_causal(const uint32_t (&r)[32], const float* __restrict__ negc, float a,
                                                       float2 (&acc)[2], int row0, int R, int n_window, int n, int key) {
  int rr = row0 % R;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float pr = ex2(fmaf(__uint_as_float(r[i]), a, negc[i]));
    if (rr < n_window && key > max(n - n_window + rr, 0)) pr = 0.f;
    if (MAXRED) acc[0].x = fmaxf(acc[0].x, pr); else acc[0].x += pr;
    if (++rr == R) rr = 0;
  }
}

// ------------------------------------------------------------------ the kernel --------

template <int PASS, bool MAXRED>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, const ScoreParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr int BUFCOLS = kBufCols;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* k_sm = smem;
  uint8_t* q_sm = smem + (size_t)p.n_stages * p.stage_bytes;
  float* c_sm = reinterpret_cast<float*>(q_sm + p.q_bytes);
  int* tp = reinterpret_cast<int*>(c_sm + p.M_pad);
  uint64_t* bars = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(tp + p.n_seq + 1) + 7) & ~(uintptr_t)7);
  uint64_t* k_full = bars;
  uint64_t* k_empty = bars + kMaxStages;
  uint64_t* q_full = bars + 2 * kMaxStages;
  uint64_t* q_empty = q_full + 1;
  uint64_t* t_full = q_full + 2;
  uint64_t* t_empty = t_full + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  if ((smem_u32(smem) & 1023u) != 0) {      // the swizzled tiles need 1024-byte alignment
    if (tid == 0) report(p.status, SPEC_ERR_ALIGNMENT);
    return;
  }
  if (tid == 0) {
    *abort_flag = 0;
    build_tile_prefix(p, tp);
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
  }
  if (tid == 32) {
    // pass 1: one MMA thread, every buffer drained by all 16 epilogue warps;
    // pass 2: two MMA threads release a stage, a buffer is drained by the 8 warps of one pair
    for (int i = 0; i < kMaxStages; ++i) { mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 2); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 2);
    for (int i = 0; i < 4; ++i) { mbar_init(&t_full[i], 1); mbar_init(&t_empty[i], 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_kh = p.d / 64;                               // 64-element halves of the contraction
  const uint32_t q_half_bytes = (uint32_t)p.M_pad * 128u;
  // K ring: [64-element half of the contraction][stage][128 keys x 128 bytes]
  const uint32_t k_half_bytes = (uint32_t)p.n_stages * (128u * 128u);

  if (warp == 0) {
    // ------------------------------------------------ TMA producer ----
    if (lane == 0) {
      SegIter it = seg_begin(p, tp, gridDim.x, blockIdx.x);
      Seg sg;
      uint32_t kit = 0, nseg = 0;
      bool ok = true;
      while (ok && seg_next(it, p, tp, sg)) {
        if (nseg > 0) ok = mbar_wait(q_empty, (nseg - 1) & 1, abort_flag);   // previous unit's MMAs retired
        if (!ok) break;
        ++nseg;
        mbar_expect_tx(q_full, p.q_bytes);
        const int qrow0 = ((sg.s * p.L + sg.l) * p.Hq + sg.h * p.G) * p.R;
        for (int kh = 0; kh < n_kh; ++kh)
          for (int rb = 0; rb < p.M_pad / 128; ++rb)
            tma_load_2d(q_sm + kh * q_half_bytes + rb * (128 * 128), &tm_q, kh * 64, qrow0 + p.row0 + rb * 128, q_full);
        for (int t = 0; t < sg.nt; ++t, ++kit) {
          const int stage = kit % p.n_stages;
          const uint32_t par = (kit / p.n_stages) & 1;
          ok = mbar_wait(&k_empty[stage], par ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(&k_full[stage], p.stage_bytes);
          uint8_t* dst = k_sm + (size_t)stage * (128 * 128);
          const int row = sg.begin + (sg.t0 + t) * kTileKeys;
          for (int kh = 0; kh < n_kh; ++kh)
            tma_load_4d(dst + kh * k_half_bytes, &tm_k, kh * 64, row, sg.h, sg.l, &k_full[stage]);
        }
      }
    }
  } else if (warp == 1 || warp == kMmaWarpB) {
    // ------------------------------------------------ MMA issuers -----
    // Two issuing threads, one per warpgroup pair.  An issuing thread is a serial chain of
    // barrier waits and tcgen05.mma instructions (each holds the thread for about 60 cycles),
    // so one thread alone leaves the tensor pipe idle for more than half of the time.  Thread s
    // feeds pair s only: the buffers 2s and 2s + 1 of that pair's two warpgroups.  Both threads
    // wait for every key tile and commit to its "empty" barrier, whether or not they used it,
    // so that every phase of those barriers sees exactly two arrivals.
    if (lane == 0) {
      const int strm = warp == 1 ? 0 : 1;
      SegIter it = seg_begin(p, tp, gridDim.x, blockIdx.x);
      Seg sg;
      uint32_t kit = 0, nseg = 0;
      bool ok = true;
      const uint32_t idesc_full = make_idesc(128);
      const uint32_t idesc_last = make_idesc(PASS == 1 ? 128 : p.cw_last);
      const int n_sub = PASS == 1 ? p.M_pad / 128 : p.n_chunks;
      const uint32_t q_lo0 = desc_lo(smem_u32(q_sm)), k_lo0 = desc_lo(smem_u32(k_sm));
      const uint32_t q_half16 = q_half_bytes >> 4;
      const uint32_t k_half16 = k_half_bytes >> 4;
      uint32_t uses[2] = {0u, 0u};                            // items issued into each of my pair's two buffers
      while (ok && seg_next(it, p, tp, sg)) {
        ok = mbar_wait(q_full, nseg & 1, abort_flag);
        if (!ok) break;
        ++nseg;
        tc_fence_after();
        // A key tile belongs to the pair with the parity of its index in the segment; within the
        // pair, sub-item `sub` (a block of 128 query rows) of the pair's k-th tile goes to the
        // warpgroup (sub + k) & 1, whose private 128-column buffer receives it.
        for (int t = 0; t < sg.nt && ok; ++t, ++kit) {
          const int stage = kit % p.n_stages;
          ok = mbar_wait(&k_full[stage], (kit / p.n_stages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + stage * ((128 * 128) >> 4);
          if ((t & 1) == strm) {
            for (int sub = 0; sub < n_sub; ++sub) {
              const int h = (sub + (t >> 1)) & 1;
              const int buf = strm * 2 + h;
              ok = mbar_wait(&t_empty[buf], (uses[h] & 1) ^ 1, abort_flag);
              if (!ok) break;
              ++uses[h];
              tc_fence_after();
              const uint32_t d_tmem = tmem_base + buf * BUFCOLS;
              const uint32_t q_lo = q_lo0 + sub * ((128 * 128) >> 4);
              const uint32_t idesc = (PASS == 2 && sub == n_sub - 1) ? idesc_last : idesc_full;
#pragma unroll
              for (int kh = 0; kh < 2; ++kh) {
                if (kh < n_kh) {
#pragma unroll
                  for (int ks = 0; ks < 4; ++ks) {
                    if (PASS == 1) tc_mma(d_tmem, desc_at(q_lo + kh * q_half16 + ks * 2), desc_at(k_lo + kh * k_half16 + ks * 2), idesc, (kh | ks) != 0);
                    else tc_mma(d_tmem, desc_at(k_lo + kh * k_half16 + ks * 2), desc_at(q_lo + kh * q_half16 + ks * 2), idesc, (kh | ks) != 0);
                  }
                }
              }
              tc_commit(&t_full[buf]);
            }
          }
          if (ok) tc_commit(&k_empty[stage]);      // arrives once my MMAs on this stage (if any) retire
        }
        if (ok) tc_commit(q_empty);
      }
    }
  } else if (warp < kMmaWarpB) {
    // ------------------------------------------------ epilogue --------
    const int wg = (warp - 2) >> 2;                        // warpgroup 0..3
    const int pair = wg >> 1;                              // pairs take alternate key tiles
    const int half = wg & 1;                               // column half of the pair's buffer
    const int quarter = warp & 3;                          // TMEM lane quarter this warp may read
    const int row_in_tile = quarter * 32 + lane;
    const int et = tid - 64;                               // 0..511 among epilogue threads
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
    SegIter it = seg_begin(p, tp, gridDim.x, blockIdx.x);
    Seg sg;
    bool ok = true;
    uint32_t ra[32];
    uint32_t used = 0;                                       // items drained from my warpgroup's buffer
    const uint32_t my_taddr = lane_base + wg * BUFCOLS;
    if (PASS == 1) {
      // Work item = 128 query rows (on lanes) x the 128 keys of a tile, all of it mine.
      const int n_mt = p.M_pad / 128;
      float mrun[kMaxMTiles], zrun[kMaxMTiles];
      while (ok && seg_next(it, p, tp, sg)) {
#pragma unroll
        for (int i = 0; i < kMaxMTiles; ++i) { mrun[i] = -INFINITY; zrun[i] = 0.f; }
        for (int t = pair; t < sg.nt && ok; t += 2) {
          const int key0 = (sg.t0 + t) * kTileKeys;                                // first key of the tile
          const int nv = min(kTileKeys, sg.n - key0);                              // valid keys of the tile
          const bool in_window = p.causal && key0 + kTileKeys > sg.n - p.n_window;    // warp-uniform
          const bool plain = nv >= kTileKeys && !in_window;
          for (int mt = ((t >> 1) + half) & 1; mt < n_mt && ok; mt += 2) {
            ok = mbar_wait(&t_full[wg], used & 1, abort_flag);
            if (!ok) break;
            ++used;
            tc_fence_after();
            float m = mrun[mt], z = zrun[mt];
            if (plain) {
              // every row sees all 128 keys: no masks, no per-row arithmetic
              tmem_ld32(my_taddr, ra);
              stats_update<false>(ra, 32, p.a, m, z);
              tmem_ld32(my_taddr + 32, ra);
              stats_update<false>(ra, 32, p.a, m, z);
              tmem_ld32(my_taddr + 64, ra);
              stats_update<false>(ra, 32, p.a, m, z);
              tmem_ld32(my_taddr + 96, ra);
              tc_fence_before();
              arrive_lane0(&t_empty[wg], lane);               // all reads done: the buffer can be refilled
              stats_update<false>(ra, 32, p.a, m, z);
            } else {
              int vis = nv;                                    // keys of the tile that this thread's row may see
              if (in_window) {
                const int rr = (p.row0 + mt * 128 + row_in_tile) % p.R;
                if (rr < p.n_window) vis = min(nv, max(sg.n - p.n_window + rr, 0) + 1 - key0);
              }
#pragma unroll 1
              for (int c = 0; c < 4; ++c) {
                if (c * 32 >= nv) break;                                    // warp-uniform
                tmem_ld32(my_taddr + c * 32, ra);
                if (vis - c * 32 > 0) stats_update<true>(ra, min(vis - c * 32, 32), p.a, m, z);
              }
              tc_fence_before();
              arrive_lane0(&t_empty[wg], lane);
            }
            mrun[mt] = m;
            zrun[mt] = z;
          }
        }
        if (ok) {
          float* dst = p.partial + ((size_t)(sg.unit + blockIdx.x) * kEpilogueWarpgroups + wg) * p.M * 2;
          for (int mt = 0; mt < n_mt; ++mt) {
            const int row = mt * 128 + row_in_tile;
            if (row < p.M) {
              dst[row * 2 + 0] = mrun[mt];
              dst[row * 2 + 1] = zrun[mt];
            }
          }
        }
      }
    } else {
      // Work item = one key tile (keys on lanes) x one chunk of 128 query rows, all of it mine; the
      // chunks of a tile alternate between the two warpgroups of the pair.
      const float2 a2 = splat2(p.a);
      // Every epilogue thread passes the two barriers of every segment, also after a wait has
      // given up, so that no warp is left waiting at them.
      while (seg_next(it, p, tp, sg)) {
        const int qrow0 = ((sg.s * p.L + sg.l) * p.Hq + sg.h * p.G) * p.R;
        asm volatile("bar.sync 1, 512;" ::: "memory");          // previous unit's constants no longer read
        for (int i = et; i < p.M_pad; i += kEpilogueThreads) c_sm[i] = i < p.M ? p.rowc[qrow0 + p.row0 + i] : -INFINITY;
        asm volatile("bar.sync 1, 512;" ::: "memory");
        float* out = p.scores + ((long long)sg.l * p.Hkv + sg.h) * p.T + sg.begin;
        for (int t = pair; t < sg.nt && ok; t += 2) {
          float2 acc[2] = {splat2(0.f), splat2(0.f)};
          const int key = (sg.t0 + t) * kTileKeys + row_in_tile;
          const bool in_window = p.causal && (sg.t0 + t + 1) * kTileKeys > sg.n - p.n_window;   // warp-uniform
          bool any = false;
          for (int ch = ((t >> 1) + half) & 1; ch < p.n_chunks; ch += 2) {
            ok = mbar_wait(&t_full[wg], used & 1, abort_flag);
            if (!ok) break;
            ++used;
            any = true;
            tc_fence_after();
            const int cw = ch == p.n_chunks - 1 ? p.cw_last : 128;            // my columns: 64 or 128
            const float* negc = c_sm + ch * 128;
            const int row0 = p.row0 + ch * 128;                 // query row of my first column
            const int nb = cw >> 5;                             // blocks of 32 columns: 2 or 4
#pragma unroll 1
            for (int c = 0; c < nb; ++c) {
              tmem_ld32(my_taddr + c * 32, ra);
              if (c == nb - 1) {
                tc_fence_before();
                arrive_lane0(&t_empty[wg], lane);
              }
              if (!in_window) prob_accumulate<MAXRED>(ra, negc + c * 32, a2, acc);
              else prob_accumulate_causal<MAXRED>(ra, negc + c * 32, p.a, acc, row0 + c * 32, p.R, p.n_window, sg.n, key);
            }
          }
          if (!ok) break;
          if (any && key < sg.n) {
            // The output was zero-filled; the two warpgroups of the pair contribute once per key.
            const float v0 = acc[0].x, v1 = acc[0].y, v2 = acc[1].x, v3 = acc[1].y;
            if (MAXRED) {
              const float v = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
              asm volatile("red.global.max.u32 [%0], %1;" ::"l"(out + key), "r"(__float_as_uint(v)) : "memory");
            } else {
              const float v = (v0 + v1) + (v2 + v3);
              asm volatile("red.global.add.f32 [%0], %1;" ::"l"(out + key), "f"(v) : "memory");
            }
          }
        }
      }
    }
  }

  if (*abort_flag) {
    if (tid == 0) report(p.status, SPEC_ERR_TIMEOUT);
    __nanosleep(200000);                                     // let copies already in flight land
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

// Combines the per-segment statistics of every query row into its softmax constant.
__global__ void __launch_bounds__(128) merge_kernel(const ScoreParams p, int n_ctas) {
  __shared__ int sh_before, sh_total;
  const int unit = blockIdx.x;
  const int lh = unit / p.n_seq, s = unit % p.n_seq;
  if (threadIdx.x == 0) { sh_before = 0; sh_total = 0; }
  __syncthreads();
  int before = 0, total = 0;
  for (int i = threadIdx.x; i < p.n_seq; i += blockDim.x) {
    int b, n;
    seq_range(p.cu, p.n_in, i, b, n);
    const int tiles = (n + kTileKeys - 1) / kTileKeys;
    total += tiles;
    if (i < s) before += tiles;
  }
  atomicAdd(&sh_before, before);
  atomicAdd(&sh_total, total);
  __syncthreads();
  int b, n;
  seq_range(p.cu, p.n_in, s, b, n);
  const int tiles = (n + kTileKeys - 1) / kTileKeys;
  if (tiles == 0) return;
  const long long TT = sh_total;
  const long long N = (long long)p.L * p.Hkv * TT;
  const long long P = (N + n_ctas - 1) / n_ctas;
  const long long u0 = (long long)lh * TT + sh_before;
  const int b0 = (int)(u0 / P), b1 = (int)((u0 + tiles - 1) / P);
  const int l = lh / p.Hkv, h = lh % p.Hkv;
  const int qrow0 = ((s * p.L + l) * p.Hq + h * p.G) * p.R;
  for (int i = threadIdx.x; i < p.M; i += blockDim.x) {
    float m = -INFINITY;
    const int s0 = (unit + b0) * kEpilogueWarpgroups, s1 = (unit + b1) * kEpilogueWarpgroups + kEpilogueWarpgroups - 1;   // one partial per warpgroup and CTA
    for (int c = s0; c <= s1; ++c) m = fmaxf(m, p.partial[((size_t)c * p.M + i) * 2]);
    float z = 0.f;
    for (int c = s0; c <= s1; ++c) {
      const float pm = p.partial[((size_t)c * p.M + i) * 2];
      const float pz = p.partial[((size_t)c * p.M + i) * 2 + 1];
      if (pm > -INFINITY) z += pz * exp2f(pm - m);
    }
    float c = m + log2f(z);
    if (p.row_weight) c -= log2f(p.row_weight[(p.row0 + i) % p.R]);
    p.rowc[qrow0 + p.row0 + i] = -c;
  }
}

// ------------------------------------------------------------------ host side ---------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace spec

SPEC_EXPORT int32_t spec_score(const spec_problem* pr, const void* q, const void* k, const float* row_weight,
                               int32_t reduce, int32_t causal_window, float* scores_out, void* workspace,
                               size_t workspace_bytes, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!q || !k || !scores_out) return fail(SPEC_ERR_BAD_ARG, "q, k and scores_out must not be NULL");
  if (reduce != SPEC_REDUCE_SUM && reduce != SPEC_REDUCE_MAX) return fail(SPEC_ERR_BAD_ARG, "reduce=%d is not a spec_reduce value", reduce);
  if (causal_window != 0 && causal_window != 1) return fail(SPEC_ERR_BAD_ARG, "causal_window=%d must be 0 or 1", causal_window);
  if (!(pr->softmax_scale > 0.f) || !(pr->softmax_scale < 1e30f)) return fail(SPEC_ERR_BAD_ARG, "softmax_scale must be positive and finite");
  if (!aligned16(q) || !aligned16(k)) return fail(SPEC_ERR_ALIGNMENT, "q and k must be 16-byte aligned");
  const int d = pr->head_dim;
  if (pr->k_stride_token < d || pr->k_stride_head < d || pr->k_stride_layer < d ||
      (pr->k_stride_token * 2) % 16 || (pr->k_stride_head * 2) % 16 || (pr->k_stride_layer * 2) % 16)
    return fail(SPEC_ERR_ALIGNMENT, "K strides must be multiples of 8 elements and at least head_dim");
  const int R = pr->n_lookahead + pr->n_window;
  const int G = pr->n_q_heads / pr->n_kv_heads;
  const int M = G * R;
  // The query rows of a unit stay resident in shared memory; more than fit (G*R*head_dim > 81920) are
  // scored in several launches over equal groups of rows, whose contributions add up in scores_out.
  const int rows_max = std::min(81920 / d, kMaxMTiles * 128) / 128 * 128;
  const int n_groups = (M + rows_max - 1) / rows_max;
  const int rows_group = ((M + n_groups - 1) / n_groups + 127) / 128 * 128;
  const WorkspacePlan wp = plan_workspace(pr);
  if (!workspace || workspace_bytes < wp.total)
    return fail(SPEC_ERR_WORKSPACE, "workspace of %zu bytes given, %zu needed", workspace_bytes, wp.total);
  rc = check_device();
  if (rc != SPEC_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the whole output is overwritten: tokens that no sequence covers read as 0, and pass 2 adds into it
  const size_t out_bytes = (size_t)pr->n_layers * pr->n_kv_heads * (size_t)pr->total_tokens * sizeof(float);
  if (out_bytes) SPEC_CUDA_OK(cudaMemsetAsync(scores_out, 0, out_bytes, st));
  const int64_t tokens = pr->cu_seqlens ? pr->total_tokens : pr->n_in;
  if (tokens == 0) return SPEC_OK;

  EncodeTiledFn encode = encode_fn();
  if (!encode) return fail(SPEC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");

  CUtensorMap tm_q, tm_k;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)pr->n_seq * pr->n_layers * pr->n_q_heads * R};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t es[2] = {1, 1};
    CUresult r = encode(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPEC_ERR_CUDA, "tensor map for q could not be encoded (CUresult %d)", (int)r);
  }
  {
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)pr->total_tokens, (cuuint64_t)pr->n_kv_heads, (cuuint64_t)pr->n_layers};
    const cuuint64_t strides[3] = {(cuuint64_t)pr->k_stride_token * 2, (cuuint64_t)pr->k_stride_head * 2, (cuuint64_t)pr->k_stride_layer * 2};
    const cuuint32_t box[4] = {64, 128, 1, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = encode(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPEC_ERR_CUDA, "tensor map for k could not be encoded (CUresult %d)", (int)r);
  }

  ScoreParams p;
  p.cu = pr->cu_seqlens;
  p.row_weight = row_weight;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.partial = reinterpret_cast<float*>(ws + wp.partial_off);
  p.rowc = reinterpret_cast<float*>(ws + wp.rowc_off);
  p.scores = scores_out;
  p.status = status_word;
  p.T = pr->total_tokens;
  p.n_in = pr->n_in; p.n_seq = pr->n_seq; p.L = pr->n_layers; p.Hq = pr->n_q_heads; p.Hkv = pr->n_kv_heads;
  p.G = G; p.R = R; p.d = d;
  p.reduce = reduce;
  p.causal = causal_window;
  p.n_window = pr->n_window;
  p.a = (float)((double)pr->softmax_scale * 1.4426950408889634);
  p.stage_bytes = (uint32_t)kTileKeys * d * 2;

  const int n_ctas = wp.score_ctas;
  const unsigned n_units = (unsigned)(pr->n_seq * pr->n_layers * pr->n_kv_heads);
  auto pass1 = score_kernel<1, false>;
  auto pass2 = reduce == SPEC_REDUCE_MAX ? score_kernel<2, true> : score_kernel<2, false>;
  // The kernels may use all of an SM's shared memory; the attribute is set once per device (it is per
  // function and context, so setting it per call would race between host threads).
  {
    static int set[64] = {0};
    int dev = 0;
    SPEC_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return fail(SPEC_ERR_UNSUPPORTED, "device ordinal %d is not supported", dev);
    if (!__atomic_load_n(&set[dev], __ATOMIC_ACQUIRE)) {
      SPEC_CUDA_OK(cudaFuncSetAttribute(score_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
      SPEC_CUDA_OK(cudaFuncSetAttribute(score_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
      SPEC_CUDA_OK(cudaFuncSetAttribute(score_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
      __atomic_store_n(&set[dev], 1, __ATOMIC_RELEASE);
    }
  }
  for (int g = 0; g < n_groups; ++g) {
    p.row0 = g * rows_group;
    p.M = std::min(rows_group, M - p.row0);
    p.M_pad = (p.M + 127) / 128 * 128;
    const int M64 = (p.M + 63) / 64 * 64;                  // pass 2 splits each chunk's columns in two halves of 32 or 64
    p.n_chunks = (M64 + 127) / 128;
    p.cw_last = M64 - (p.n_chunks - 1) * 128;
    p.q_bytes = (uint32_t)p.M_pad * d * 2;
    const int small = p.M_pad * 4 + (pr->n_seq + 1) * 4 + 8 + kNumBars * 8 + 16;
    const int smem_max = 227 * 1024;
    int stages = (smem_max - (int)p.q_bytes - small) / (int)p.stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(SPEC_ERR_UNSUPPORTED, "not enough shared memory for two key stages (%d rows, head_dim=%d)", p.M, d);
    p.n_stages = stages;
    int smem = stages * (int)p.stage_bytes + (int)p.q_bytes + small;
    if (smem < 120 * 1024) smem = 120 * 1024;             // one CTA per SM: each CTA owns the whole TMEM
    pass1<<<n_ctas, kThreads, smem, st>>>(tm_q, tm_k, p);
    SPEC_CUDA_OK(cudaGetLastError());
    merge_kernel<<<n_units, 128, 0, st>>>(p, n_ctas);
    SPEC_CUDA_OK(cudaGetLastError());
    pass2<<<n_ctas, kThreads, smem, st>>>(tm_q, tm_k, p);
    SPEC_CUDA_OK(cudaGetLastError());
  }
  return SPEC_OK;
}
