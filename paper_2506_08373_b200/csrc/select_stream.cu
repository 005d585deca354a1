// Streaming pool + top-C selection for the default pooling (Algorithm 1 lines 10, 11 and 13 with
// the hyper-parameter table's Max pool of width 7), used when the caller provides a workspace.
//
// Three kernels on the caller's stream; no CTA ever waits for another:
//   1. sample_floor_kernel, one CTA per (sequence, layer, KV head) unit: pools one 32-byte sector
//      out of every 32..128 positions (a sector holds the whole width-7 window of its fourth
//      score) and takes, from a two-level histogram of the sampled keys (top 11 bits, then the
//      next 11), the key a few standard deviations below the rank the budget corresponds to.
//      That key is a floor under the final threshold with overwhelming probability, and it does
//      not depend on where in the unit the large scores sit (rising, falling or concentrated
//      scores cost the same).
//   2. stream_sweep_kernel, one small CTA per (unit, chunk of 2048 positions), sixteen to an SM: the
//      chunk is staged in shared memory with one bulk asynchronous copy and pooled from there
//      (three 16-byte reads per four positions, nothing written back); the positions at or above
//      the floor go, as (key, position) pairs, to the chunk's own segment of the unit's candidate
//      array in the workspace.  The scores are read from global memory once.
//   3. stream_finish_kernel, one CTA per unit: three radix passes (11 + 11 + 10 bits) over the
//      candidates, held in shared memory, find the exact threshold key; winners and ties are
//      marked in position bitmaps and written out in ascending position, ties to the lower
//      position.  A second budget (the vertical indices) is selected from the same candidates.
// If the floor was too high or too low for the candidate array (fewer candidates than the budget,
// or more than fit: only with massively tied scores), the finishing CTA falls back to the generic
// selection that recomputes pooled keys from global memory.  The result is exact in every case.
//
// Units of up to 16384 positions, a few to an SM, skip the workspace and the three launches:
// unit_select_kernel stages a unit in shared memory and does the same three steps in one CTA.
#include "select_common.cuh"

#include <algorithm>

namespace spec {

constexpr int kStreamBins = 2048;
constexpr int kSweepThreads = 64;
constexpr int kSweepWarps = kSweepThreads / 32;
constexpr int kMaxStepsPerWarp = 8;              // 128-position steps a sweeping warp keeps in registers
constexpr int kMaxSamples = 4096;
constexpr uint32_t kNoSelection = 0xFFFFFFFFu;   // floor value of a unit that keeps everything or nothing

struct StreamParams {
  const float* scores;
  const int32_t* cu;
  int64_t T;
  int n_in, L, H, n_forced, c_max, n_vert;
  int chunk;                  // positions per sweeping CTA (multiple of 128)
  int chunks_max;             // CTAs per unit
  int bitmap_words;           // words of one position bitmap of the finishing CTA
  int max_len;                // the host's bound on any sequence length (sizes the grid and shared memory)
  int held_cap;               // candidates the finishing CTA can hold in shared memory
  int32_t* head;              // [units][head_words]: floor key, unused, unused, failure flag, then a candidate count per chunk
  int head_words;
  uint2* cand;                // candidate (key, position) pairs
  int64_t row_entries;        // candidate entries per (layer, KV head) row
  int32_t* idx_out;
  int32_t* count_out;
  int32_t* vert_out;
  int32_t* vert_count_out;
  int32_t* status;
};

struct UnitGeom {
  int s, l, h, begin, n, forced, e;
  bool over;                  // longer than the host's bound: treated as empty and reported
  int take[2];
  const float* src;
  int64_t cand_off;
  int cand_cap;
};

__device__ __forceinline__ UnitGeom unit_geom_of(const StreamParams& p, int s, int row);

__device__ __forceinline__ UnitGeom unit_geom(const StreamParams& p, int unit) {
  const int rows = p.H * p.L;
  return unit_geom_of(p, unit / rows, unit % rows);
}

// row = layer * H + head
__device__ __forceinline__ UnitGeom unit_geom_of(const StreamParams& p, int s, int row) {
  UnitGeom g;
  g.s = s;
  g.l = g.h = 0;                                          // only their combination, `row`, is used
  seq_range(p.cu, p.n_in, g.s, g.begin, g.n);
  g.over = g.n > p.max_len;
  if (g.over) g.n = 0;
  g.forced = min(p.n_forced, g.n);
  g.e = g.n - g.forced;
  g.take[0] = max(min(p.c_max - g.forced, g.e), 0);
  g.take[1] = max(min(p.n_vert, g.e), 0);
  g.src = p.scores + (int64_t)row * p.T + g.begin;
  // even, so that a segment starts on a 16-byte boundary
  g.cand_off = (int64_t)row * p.row_entries + ((g.begin + 1) & ~1) + (int64_t)g.s * kSelCandSlack;
  g.cand_cap = g.n + kSelCandSlack;
  return g;
}

__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// From the sampled keys (0 = no sample) and the histogram of their leading 11 bits to the floor: about
// tk / 2^shift of the samples lie above the threshold; the floor is taken four standard deviations
// further down the sample, with the next 11 bits resolved among the samples of that bin.  0 when the
// sample is too small to tell.  Called by all threads of the CTA.
__device__ __forceinline__ uint32_t floor_from_samples(const uint32_t* skey, int n_groups, uint32_t* hist, int tk, int shift,
                                                       int* wsum, int* out2) {
  const int tid = threadIdx.x;
  const float m_exp = (float)tk / (float)(1 << shift);
  const int rho = (int)(m_exp + 4.f * sqrtf(m_exp) + 8.f);
  int fb, ab;
  if (!locate_bin(hist + tid * (kStreamBins / kSelThreads), kStreamBins / kSelThreads, rho, wsum, out2, fb, ab)) return 0u;
  for (int b = tid; b < kStreamBins; b += kSelThreads) hist[b] = 0;
  __syncthreads();
  for (int m = tid; m < n_groups; m += kSelThreads) {
    const uint32_t key = skey[m];
    if (key != 0 && (key >> 21) == (uint32_t)fb) atomicAdd(&hist[(key >> 10) & 2047u], 1u);
  }
  int dg = 0, ab2 = 0;
  locate_bin(hist + tid * (kStreamBins / kSelThreads), kStreamBins / kSelThreads, rho - ab, wsum, out2, dg, ab2);
  return ((uint32_t)fb << 21) | ((uint32_t)dg << 10);
}

// ---------------------------------------------------------------- 1. the floor -------

__global__ void __launch_bounds__(kSelThreads) sample_floor_kernel(const StreamParams p) {
  __shared__ uint32_t hist[kStreamBins];
  __shared__ uint32_t skey[kMaxSamples];
  __shared__ int wsum[32];
  __shared__ int out2[4];
  const int unit = blockIdx.x, tid = threadIdx.x;
  // The sweep is launched as a programmatic dependent: its CTAs may start now and issue the copies of
  // their chunks; they wait for this grid to finish before they read the floor.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const UnitGeom g = unit_geom(p, unit);
  const int tk = max(g.take[0], g.take[1]);
  const bool selects = (g.take[0] > 0 && g.take[0] < g.e) || (g.take[1] > 0 && g.take[1] < g.e);
  uint32_t floor_key = kNoSelection;
  if (selects) {
    floor_key = 0;
    for (int b = tid; b < kStreamBins; b += kSelThreads) hist[b] = 0;
    // x = position + mis8 puts every multiple of eight on a 32-byte boundary of global memory
    const int mis8 = (int)((reinterpret_cast<uintptr_t>(g.src) >> 2) & 7u);
    const int X = g.e + mis8;
    int shift = g.e >= 65536 ? 7 : g.e >= 16384 ? 6 : 5;             // one sample per 2^shift positions
    while (((X >> shift) + 1) > kMaxSamples) ++shift;
    const int spg = 1 << (shift - 3);                                // sectors per sample group
    const int n_sectors = (X + 7) >> 3;
    const int n_groups = (n_sectors + spg - 1) / spg;                // <= kMaxSamples
    __syncthreads();
    for (int m = tid; m < n_groups; m += kSelThreads) {
      uint32_t hsh = ((uint32_t)unit * 0x9E3779B1u) ^ ((uint32_t)m * 0x85EBCA6Bu);
      hsh ^= hsh >> 15; hsh *= 0x2C1B3C6Du; hsh ^= hsh >> 12;
      const int q = m * spg + (int)(hsh % (uint32_t)min(spg, n_sectors - m * spg));
      const int p0 = q * 8 - mis8;                                   // position of the sector's first score
      const int centre = p0 + 3;
      uint32_t key = 0;                                              // 0: no sample here (below every real key's top bits)
      if (centre >= 0 && centre < g.e) {
        float v[8];
        if (p0 >= 0 && p0 + 8 <= g.e) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(g.src + p0));
          const float4 b = __ldg(reinterpret_cast<const float4*>(g.src + p0 + 4));
          v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = (p0 + i >= 0 && p0 + i < g.e) ? __ldg(g.src + p0 + i) : -INFINITY;
        }
        key = to_key(fmax3(fmax3(v[0], v[1], v[2]), fmax3(v[3], v[4], v[5]), v[6]));   // pooled value of the centre
        atomicAdd(&hist[key >> 21], 1u);
      }
      skey[m] = key;
    }
    floor_key = floor_from_samples(skey, n_groups, hist, tk, shift, wsum, out2);
  }
  if (tid == 0) {
    if (g.over) report(p.status, SPEC_ERR_BAD_ARG);
    int32_t* hd = p.head + (int64_t)unit * p.head_words;
    hd[0] = (int32_t)floor_key;
    hd[1] = 0;
    hd[2] = 0;
    hd[3] = 0;
  }
}

// ---------------------------------------------------------------- 2. the sweep -------

// Where a sweeping CTA's work item (one chunk of one unit) lies and what it copies in bulk.
struct SweepItem {
  UnitGeom g;
  int32_t* hd;
  uint32_t floor_key;
  int chunk_id, mis, X, x0, x1, n_steps, xa, total, bx0, bx1;
  bool active, bulk;
};

__device__ __forceinline__ SweepItem sweep_item(const StreamParams& p, int s, int row, int chunk_id) {
  SweepItem t;
  t.chunk_id = chunk_id;
  t.g = unit_geom_of(p, s, row);
  t.hd = p.head + ((int64_t)s * (p.H * p.L) + row) * p.head_words;
  t.floor_key = 0;                                         // read by the caller once the copy is under way
  t.mis = (int)((reinterpret_cast<uintptr_t>(t.g.src) >> 2) & 3u);
  t.X = t.g.e + t.mis;                                     // x = position + mis: multiples of four are 16-byte boundaries
  t.x0 = t.chunk_id * p.chunk;
  t.x1 = min(t.x0 + p.chunk, t.X);
  t.active = t.x1 > t.x0;
  t.n_steps = t.active ? (t.x1 - t.x0 + 127) >> 7 : 0;
  // staged: [x0 - 4, x0 + n_steps * 128 + 4); the 16-byte aligned interior of the unit comes by bulk copy
  t.xa = t.x0 - 4;
  t.total = t.n_steps * 128 + 8;
  t.bx0 = max(t.xa, t.mis ? 4 : 0);
  t.bx1 = min(t.xa + t.total, t.X & ~3);
  t.bulk = t.active && t.bx1 > t.bx0;
  if (!t.bulk) t.bx0 = t.bx1 = t.xa + t.total;
  return t;
}

// Pools my warp's steps straight from shared memory; bit 4k + u of the returned mask marks the
// candidates (pooled value at or above the floor) among my four positions of step k.  EDGE: the
// chunk holds slots that are not positions of the unit (only the chunks at either end do).  NW: the
// warps that share the chunk, step by step in turn.
template <bool EDGE, int NW>
__device__ __forceinline__ uint32_t sweep_steps(const SweepItem& t, const float* raw, float floor_f, int warp, int lane) {
  const float4* base4 = reinterpret_cast<const float4*>(raw + 4);
  uint32_t mask = 0;
#pragma unroll
  for (int k = 0; k < kMaxStepsPerWarp; ++k) {
    const int st = warp + k * NW;
    if (st < t.n_steps) {
      const float4* at = base4 + st * 32 + lane;
      const float4 pv = at[-1], cv = at[0], nv = at[1];
      const float x[10] = {pv.y, pv.z, pv.w, cv.x, cv.y, cv.z, cv.w, nv.x, nv.y, nv.z};
      // the four windows share x[3..6]; neighbouring windows share a pair on either side
      const float mid = fmax3(x[3], x[4], fmaxf(x[5], x[6])), l12 = fmaxf(x[1], x[2]), r78 = fmaxf(x[7], x[8]);
      const float v[4] = {fmax3(mid, x[0], l12), fmax3(mid, l12, x[7]), fmax3(mid, x[2], r78), fmax3(mid, r78, x[9])};
      const int pp0 = t.x0 + st * 128 + lane * 4 - t.mis;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        bool c = !(v[u] < floor_f);
        if (EDGE) c = c && pp0 + u >= 0 && pp0 + u < t.g.e;
        if (c) mask |= 1u << (4 * k + u);
      }
    }
  }
  return mask;
}

// One CTA per (unit, chunk).  Many small CTAs share an SM, so that the bulk copies of some overlap
// the pooling of others (fatter CTAs, and persistent double-buffered ones, were slower).
__global__ void __launch_bounds__(kSweepThreads, 16) stream_sweep_kernel(const StreamParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __shared__ int wsum[kSweepWarps];
  __shared__ uint64_t mbar;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  SweepItem t = sweep_item(p, blockIdx.z, blockIdx.y, blockIdx.x);
  if (!t.active) return;
  float* raw = reinterpret_cast<float*>(smem_raw);
  const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&mbar);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (t.bulk) {
      const uint32_t bytes = (uint32_t)(t.bx1 - t.bx0) * 4u;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"((uint32_t)__cvta_generic_to_shared(raw + (t.bx0 - t.xa))), "l"(t.g.src + (t.bx0 - t.mis)), "r"(bytes), "r"(bar_a)
                   : "memory");
    }
  }
  for (int i = tid; i < t.total; i += kSweepThreads) {
    const int x = t.xa + i;
    if (x >= t.bx0 && x < t.bx1) { i += ((t.bx1 - x - 1) / kSweepThreads) * kSweepThreads; continue; }   // the bulk-copied part
    const int pp = x - t.mis;
    raw[i] = (pp >= 0 && pp < t.g.e) ? __ldg(t.g.src + pp) : -INFINITY;
  }
  // The floor is fetched while the copy is in flight.  A unit that keeps everything or nothing needs no sweep,
  // but its copy is awaited all the same: shared memory must not be given up with a copy under way.
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the floors are written by the grid before this one
  t.floor_key = (uint32_t)__ldcg(t.hd);
  __syncthreads();                                         // the barrier is initialised; the edges are in place
  if (t.bulk) {
    uint32_t ok = 0;
    for (uint32_t tries = 0; tries < (1u << 20) && !ok; ++tries)
      asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\nselp.u32 %0, 1, 0, q;\n}"
                   : "=r"(ok) : "r"(bar_a) : "memory");
    if (!ok) {                                             // the copy never landed: the unit is handed to the generic path
      report(p.status, SPEC_ERR_TIMEOUT);
      atomicExch(t.hd + 3, 1);
    }
  }
  if (t.floor_key == kNoSelection) return;
  const float floor_f = key_to_float(t.floor_key);
  const bool edge = t.x0 < t.mis || t.x0 + t.n_steps * 128 > t.X;
  uint32_t mask = edge ? sweep_steps<true, kSweepWarps>(t, raw, floor_f, warp, lane) : sweep_steps<false, kSweepWarps>(t, raw, floor_f, warp, lane);
  // ---- my candidates go to my own segment of the unit's array, their number to the unit's header
  const int mine = __popc(mask);
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  int before = incl - mine, n_cta = 0;
#pragma unroll
  for (int w = 0; w < kSweepWarps; ++w) {
    const int c = wsum[w];
    if (w < warp) before += c;
    n_cta += c;
  }
  if (tid == 0) t.hd[4 + t.chunk_id] = n_cta;              // a segment is as long as the chunk: it cannot overflow
  // Few positions are candidates: each lane walks its own, pooling them again from the staged scores.
  uint2* dst = p.cand + t.g.cand_off + (int64_t)t.chunk_id * p.chunk + before;
  while (mask) {
    const int b = __ffs(mask) - 1;
    mask &= mask - 1;
    const int j = (warp + (b >> 2) * kSweepWarps) * 128 + lane * 4 + (b & 3);     // position within the chunk
    const float* w7 = raw + 4 + j - 3;
    const float v = fmax3(fmax3(w7[0], w7[1], w7[2]), fmax3(w7[3], w7[4], w7[5]), w7[6]);
    *dst++ = make_uint2(to_key(v), (uint32_t)(t.x0 + j - t.mis));
  }
}

// ------------------------------------------------------------- 3. the finishing CTA --

// Shared-memory views of a finishing CTA.
struct FinishMem {
  uint32_t* hist;             // kStreamBins words
  const uint2* cand;          // the unit's candidates, (key, position); position kNoSelection marks padding
  uint32_t* map_gt;           // two position bitmaps of bitmap_words words each, 16-byte aligned; the same
  uint32_t* map_eq;           // memory is the scratch of the generic selection
  int bitmap_words;
  int* wsum;                  // 32 ints
  int* out2;                  // 4 ints
  int* lead;                  // 2 x 9 ints, zero on entry
};

// The exact selection of a unit from its candidates (every position whose pooled key is at or above
// floor_key): three radix passes (11 + 11 + 10 bits) find the threshold key; winners and ties are
// marked in position bitmaps and written out in ascending position, ties to the lower position.  A
// second budget (the vertical indices) is selected from the same candidates.  failed, or fewer
// candidates than a budget: that budget takes the generic selection, which recomputes pooled keys
// from global memory.  maps_dirty: the bitmaps were not cleared by the caller.  Called by all
// threads of the CTA.
__device__ __forceinline__ void finish_unit(const StreamParams& p, const UnitGeom& g, int unit, const FinishMem& fm, int n_cand,
                                            int n_real, bool failed, bool maps_dirty, uint32_t floor_key) {
  const int tid = threadIdx.x;
  const uint2* cand = fm.cand;
  uint32_t* hist = fm.hist;
  uint32_t* map_gt = fm.map_gt;
  uint32_t* map_eq = fm.map_eq;
  int* wsum = fm.wsum;
  int* out2 = fm.out2;
  const int n_budgets = p.n_vert > 0 ? 2 : 1;
  for (int b = 0; b < n_budgets; ++b) {
    int32_t* idx = b == 0 ? p.idx_out + (int64_t)unit * p.c_max : p.vert_out + (int64_t)unit * p.n_vert;
    int32_t* cnt = b == 0 ? p.count_out : p.vert_count_out;
    const int width = b == 0 ? p.c_max : p.n_vert;
    const int tail = b == 0 ? g.forced : 0;
    const int tk = g.take[b];
    __syncthreads();
    if (tk > 0 && tk < g.e) {
      if (failed || n_real < tk) {
        __syncthreads();
        // generic selection: pooled keys recomputed from global memory in every pass
        SelectScratch sc;
        maps_dirty = true;
        sc.hist = map_gt;
        sc.misc = reinterpret_cast<int*>(sc.hist + kSelWarps * 256);
        KeySource key;
        key.scores = g.src;
        key.e = g.e; key.pool = SPEC_POOL_MAX; key.k = 7;
        key.keys = nullptr;
        uint32_t T;
        int need_eq;
        radix_select(key, g.e, tk, sc, T, need_eq);
        ordered_emit(key, g.e, T, need_eq, sc, [&](int rank, int j) { idx[rank] = j; });
      } else {
        // ---- exact threshold among the candidates
        uint32_t prefix = 0, mask = 0;
        int remaining = tk;
        int first_pass = 0;
        {
          // The leading 11 bits first, without a histogram: every candidate is at or above the floor,
          // so they fall into a few bins from the floor's bin up.  Every thread counts the eight
          // lowest of those bins (and everything higher together) in registers; the sums over the
          // CTA locate the digit unless the threshold lies higher still (then the histogram pass).
          const uint32_t fb = floor_key >> 21;
          // nine 7-bit counters packed in one word pair per thread (a thread sees at most
          // held_cap / 512 < 128 candidates)
          int* lead_b = fm.lead + 9 * b;
          unsigned long long packed = 0;
          for (int i = tid; i < n_cand; i += kSelThreads) {
            const uint2 ck = cand[i];
            if (ck.y == kNoSelection) continue;
            packed += 1ull << (7u * min((ck.x >> 21) - fb, 8u));
          }
          // one warp-wide reduction per counter, one shared-memory addition per warp and counter
#pragma unroll
          for (int b = 0; b < 9; ++b) {
            const uint32_t v = __reduce_add_sync(0xffffffffu, (uint32_t)((packed >> (7 * b)) & 127ull));
            if ((tid & 31) == 0 && v) atomicAdd(&lead_b[b], (int)v);
          }
          __syncthreads();
          int tot[9];
#pragma unroll
          for (int b = 0; b < 9; ++b) tot[b] = lead_b[b];
          if (tot[8] < remaining) {
            int above = tot[8], b = 7;
            for (; b > 0; --b) {
              if (above + tot[b] >= remaining) break;
              above += tot[b];
            }
            remaining -= above;
            prefix = (fb + (uint32_t)b) << 21;
            mask = 2047u << 21;
            first_pass = 1;
          }
        }
        for (int pass = first_pass; pass < 3; ++pass) {
          const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
          const uint32_t dmask = pass == 2 ? 1023u : 2047u;
          for (int i = tid; i < kStreamBins; i += kSelThreads) hist[i] = 0;
          __syncthreads();
          for (int i0 = 0; i0 < n_cand; i0 += kSelThreads) {
            const int i = i0 + tid;
            const uint2 ck = i < n_cand ? cand[i] : make_uint2(0u, kNoSelection);
            const uint32_t kk = ck.x;
            const bool in = ck.y != kNoSelection && (kk & mask) == prefix;
            const uint32_t dgt = (kk >> shift) & dmask;
            if (pass == 0) {
              // lanes of a warp with the same digit add once: the candidates share their leading bits
              const uint32_t act = __ballot_sync(0xffffffffu, in);
              if (in) {
                const uint32_t same = __match_any_sync(act, dgt);
                if ((tid & 31) == __ffs(same) - 1) atomicAdd(&hist[dgt], (uint32_t)__popc(same));
              }
            } else if (in) {
              atomicAdd(&hist[dgt], 1u);
            }
          }
          int dg = 0, ab = 0;
          locate_bin(hist + tid * (kStreamBins / kSelThreads), kStreamBins / kSelThreads, remaining, wsum, out2, dg, ab);
          remaining -= ab;
          prefix |= (uint32_t)dg << shift;
          mask |= dmask << shift;
        }
        const uint32_t T = prefix;
        const int need_eq = remaining;
        // ---- winners and ties into position bitmaps, then out in ascending position
        const int n_words = (g.e + 31) >> 5;
        if (maps_dirty) {                                    // the first selection found them cleared during the gather
          uint4* z4 = reinterpret_cast<uint4*>(map_gt);      // both bitmaps, adjacent, whole 16-byte words
          const int n4 = (fm.bitmap_words + ((n_words + 3) & ~3)) >> 2;
          for (int w = tid; w < n4; w += kSelThreads) z4[w] = make_uint4(0u, 0u, 0u, 0u);
          __syncthreads();
        }
        maps_dirty = true;
        for (int i = tid; i < n_cand; i += kSelThreads) {
          const uint2 c = cand[i];
          if (c.y == kNoSelection) continue;
          if (c.x > T) atomicOr(&map_gt[c.y >> 5], 1u << (c.y & 31));
          else if (c.x == T) atomicOr(&map_eq[c.y >> 5], 1u << (c.y & 31));
        }
        __syncthreads();
        // Output rank of a position = winners (and ties) before it: an exclusive count per group of
        // a few words, kept where the histogram was, plus the words of its own group up to its bit.
        int gshift = 0;                                                          // words per group = 2^gshift, two groups per thread
        while ((2 * kSelThreads << gshift) < n_words) ++gshift;
        const int gw = 1 << gshift;
        int* grp_gt = reinterpret_cast<int*>(hist);
        int* grp_eq = grp_gt + 2 * kSelThreads;
        int gt0 = 0, eq0 = 0, gt1 = 0, eq1 = 0;
        for (int w = 2 * tid * gw; w < min((2 * tid + 1) * gw, n_words); ++w) { gt0 += __popc(map_gt[w]); eq0 += __popc(map_eq[w]); }
        for (int w = (2 * tid + 1) * gw; w < min((2 * tid + 2) * gw, n_words); ++w) { gt1 += __popc(map_gt[w]); eq1 += __popc(map_eq[w]); }
        // one scan for both counts, 16 bits each (a finishing CTA holds fewer than 2^15 candidates)
        int tot_packed;
        const int sp = block_exclusive_scan((gt0 + gt1) | ((eq0 + eq1) << 16), wsum, tot_packed);
        const int sg = sp & 0xffff, sq = sp >> 16;
        grp_gt[2 * tid] = sg; grp_gt[2 * tid + 1] = sg + gt0;
        grp_eq[2 * tid] = sq; grp_eq[2 * tid + 1] = sq + eq0;
        __syncthreads();
        if (gshift == 2) {
          // groups of four words: a group of either bitmap is one 16-byte read
#pragma unroll 2
          for (int i = tid; i < n_cand; i += kSelThreads) {
            const uint2 c = cand[i];
            if (c.x < T || c.y == kNoSelection) continue;
            const int w = (int)(c.y >> 5), grp = w >> 2, sub = w & 3;
            const uint32_t below = (1u << (c.y & 31)) - 1u;
            const uint4 mg = reinterpret_cast<const uint4*>(map_gt)[grp], mq = reinterpret_cast<const uint4*>(map_eq)[grp];
            // words of the group before mine count whole, mine up to my bit, the rest not at all
            const uint32_t k0 = sub > 0 ? 0xffffffffu : (sub == 0 ? below : 0u);
            const uint32_t k1 = sub > 1 ? 0xffffffffu : (sub == 1 ? below : 0u);
            const uint32_t k2 = sub > 2 ? 0xffffffffu : (sub == 2 ? below : 0u);
            const uint32_t k3 = sub == 3 ? below : 0u;
            const int g_before = grp_gt[grp] + __popc(mg.x & k0) + __popc(mg.y & k1) + __popc(mg.z & k2) + __popc(mg.w & k3);
            const int q_before = grp_eq[grp] + __popc(mq.x & k0) + __popc(mq.y & k1) + __popc(mq.z & k2) + __popc(mq.w & k3);
            if (c.x > T) idx[g_before + min(q_before, need_eq)] = (int32_t)c.y;
            else if (q_before < need_eq) idx[g_before + q_before] = (int32_t)c.y;
          }
        } else {
#pragma unroll 2
          for (int i = tid; i < n_cand; i += kSelThreads) {
            const uint2 c = cand[i];
            if (c.x < T || c.y == kNoSelection) continue;
            const int w = (int)(c.y >> 5), grp = w >> gshift;
            const uint32_t below = (1u << (c.y & 31)) - 1u;
            int g_before = grp_gt[grp] + __popc(map_gt[w] & below), q_before = grp_eq[grp] + __popc(map_eq[w] & below);
            for (int ww = grp << gshift; ww < w; ++ww) { g_before += __popc(map_gt[ww]); q_before += __popc(map_eq[ww]); }
            if (c.x > T) idx[g_before + min(q_before, need_eq)] = (int32_t)c.y;
            else if (q_before < need_eq) idx[g_before + q_before] = (int32_t)c.y;
          }
        }
      }
    } else {
      for (int q = tid; q < tk; q += kSelThreads) idx[q] = q;        // every eligible position is kept
    }
    for (int q = tk + tid; q < width; q += kSelThreads) idx[q] = (q - tk < tail) ? g.e + (q - tk) : -1;
    if (cnt && tid == 0) cnt[unit] = tk + tail;
  }
}

// Shared memory of stream_finish_kernel: radix histogram, the candidates, two position bitmaps
// (or, instead of the bitmaps, the scratch of the generic selection).
__host__ __device__ inline size_t stream_finish_bytes(int bitmap_words, int held_cap) {
  const size_t maps = (size_t)bitmap_words * 8, generic = (size_t)(kSelWarps * 256 + 2 * kSelWarps + 8) * 4;
  return (size_t)kStreamBins * 4 + (size_t)held_cap * 8 + (maps > generic ? maps : generic);
}

__global__ void __launch_bounds__(kSelThreads, 3) stream_finish_kernel(const StreamParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __shared__ int wsum[32];
  __shared__ int out2[4];
  __shared__ int lead[2][9];                               // per budget: candidates per leading-digit bin above the floor's
  __shared__ uint64_t mbar;
  const int tid = threadIdx.x;
  const int unit = blockIdx.x;
  if (tid < 18) (&lead[0][0])[tid] = 0;
  const UnitGeom g = unit_geom(p, unit);
  const int32_t* hd = p.head + (int64_t)unit * p.head_words;
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the candidates are written by the grid before this one
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw);
  uint2* held = reinterpret_cast<uint2*>(hist + kStreamBins);
  uint32_t* map_gt = reinterpret_cast<uint32_t*>(held + p.held_cap);
  uint32_t* map_eq = map_gt + p.bitmap_words;
  const bool any_selects = (g.take[0] > 0 && g.take[0] < g.e) || (p.n_vert > 0 && g.take[1] > 0 && g.take[1] < g.e);
  // ---- gather the candidates of the unit's chunks
  int n_cand = 0, n_real = 0;                              // slots gathered (padding pairs included), real candidates
  bool failed = hd[3] != 0;
  if (any_selects) {
    const int mis = (int)((reinterpret_cast<uintptr_t>(g.src) >> 2) & 3u);
    const int n_chunks = (g.e + mis + p.chunk - 1) / p.chunk;          // <= kSelThreads, checked on the host
    const uint2* segs = p.cand + g.cand_off;
    const int raw_cnt = tid < n_chunks ? hd[4 + tid] : 0;
    const int my_cnt = (raw_cnt + 1) & ~1;                 // rounded up to a whole 16 bytes
    int total;
    const int mine_at = block_exclusive_scan(my_cnt, wsum, total);
    n_real = total - __syncthreads_count(raw_cnt & 1);     // every odd count was rounded up by one
    failed = failed || total > p.held_cap;
    if (!failed) {
      // One bulk asynchronous copy per chunk, all in flight together.  Bulk copies move multiples of
      // 16 bytes to 16-byte aligned places, so every chunk's candidates start at an even slot and
      // an odd count drags one stale pair along, marked as padding afterwards.
      const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&mbar);
      if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"((uint32_t)total * 8u) : "memory");
      }
      __syncthreads();
      if (my_cnt > 0) {
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"((uint32_t)__cvta_generic_to_shared(held + mine_at)), "l"(segs + (int64_t)tid * p.chunk),
                       "r"((uint32_t)my_cnt * 8u), "r"(bar_a) : "memory");
      }
      // while the copies are in flight: both position bitmaps (adjacent, whole 16-byte words) are cleared
      {
        uint4* z4 = reinterpret_cast<uint4*>(map_gt);
        const int n4 = (p.bitmap_words + ((((g.e + 31) >> 5) + 3) & ~3)) >> 2;
        for (int w = tid; w < n4; w += kSelThreads) z4[w] = make_uint4(0u, 0u, 0u, 0u);
      }
      uint32_t ok = total == 0;
      for (uint32_t tries = 0; tries < (1u << 20) && !ok; ++tries)
        asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\nselp.u32 %0, 1, 0, q;\n}"
                     : "=r"(ok) : "r"(bar_a) : "memory");
      if (__syncthreads_or(!ok)) {                         // the copies never landed: the generic path serves the unit
        if (tid == 0) report(p.status, SPEC_ERR_TIMEOUT);
        failed = true;
      } else {
        if (raw_cnt & 1) held[mine_at + raw_cnt] = make_uint2(0u, kNoSelection);   // padding pair
        n_cand = total;
      }
    }
  }
  FinishMem fm;
  fm.hist = hist; fm.cand = held; fm.map_gt = map_gt; fm.map_eq = map_eq; fm.bitmap_words = p.bitmap_words;
  fm.wsum = wsum; fm.out2 = out2; fm.lead = &lead[0][0];
  finish_unit(p, g, unit, fm, n_cand, n_real, failed, false, (uint32_t)hd[0]);
}

// ------------------------------------------- short units: the three steps in one CTA --

constexpr int kUnitSlots = kMaxStepsPerWarp * kSelWarps * 128;   // 16384: what 16 warps sweep with one mask word each
constexpr int kUnitRawWords = kUnitSlots + 32;                   // staged scores with their halo, a multiple of 16 bytes
constexpr int kUnitSampleShift = 4;                              // the floor's sample: one position in 16
constexpr int kUnitHeldMin = 2304;                               // the candidate area also serves the floor's histogram and
                                                                 // samples, and the generic selection's scratch

// One CTA per unit that fits in shared memory whole: the scores are staged by one bulk copy, the
// floor comes from a sample of the staged scores, the sweep leaves its candidates in shared memory
// and finish_unit selects from them.  No workspace, no second kernel, no trip through L2 for the
// candidates.  The memory is used twice: the floor's histogram and samples lie where the
// candidates go afterwards, and the finishing step's histogram and bitmaps where the scores were.
__global__ void __launch_bounds__(kSelThreads, 2) unit_select_kernel(const StreamParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __shared__ int wsum[32];
  __shared__ int out2[4];
  __shared__ int lead[2][9];
  __shared__ uint64_t mbar;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x;
  if (tid < 18) (&lead[0][0])[tid] = 0;
  const int rows = p.H * p.L;
  SweepItem t = sweep_item(p, unit / rows, unit % rows, 0);      // the whole unit is one chunk
  const UnitGeom& g = t.g;
  float* raw = reinterpret_cast<float*>(smem_raw);
  uint2* held = reinterpret_cast<uint2*>(raw + kUnitRawWords);
  const int tk = max(g.take[0], g.take[1]);
  const bool selects = (g.take[0] > 0 && g.take[0] < g.e) || (p.n_vert > 0 && g.take[1] > 0 && g.take[1] < g.e);
  if (tid == 0 && g.over) report(p.status, SPEC_ERR_BAD_ARG);

  bool failed = false, staged = true;
  int n_cand = 0;
  uint32_t floor_key = 0;
  if (t.active) {
    const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&mbar);
    if (tid == 0) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      if (t.bulk) {
        const uint32_t bytes = (uint32_t)(t.bx1 - t.bx0) * 4u;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"((uint32_t)__cvta_generic_to_shared(raw + (t.bx0 - t.xa))), "l"(g.src + (t.bx0 - t.mis)), "r"(bytes), "r"(bar_a)
                     : "memory");
      }
    }
    for (int i = tid; i < t.total; i += kSelThreads) {
      const int x = t.xa + i;
      if (x >= t.bx0 && x < t.bx1) { i += ((t.bx1 - x - 1) / kSelThreads) * kSelThreads; continue; }   // the bulk-copied part
      const int pp = x - t.mis;
      raw[i] = (pp >= 0 && pp < g.e) ? __ldg(g.src + pp) : -INFINITY;
    }
    uint32_t* hist = reinterpret_cast<uint32_t*>(held);
    uint32_t* skey = hist + kStreamBins;
    if (selects) for (int b = tid; b < kStreamBins; b += kSelThreads) hist[b] = 0;
    __syncthreads();                                         // the barrier is initialised; edges and zeros are in place
    if (t.bulk) {
      // Awaited also by a unit that keeps everything or nothing: shared memory is not given up, nor
      // used for anything else, with a copy under way.
      uint32_t ok = 0;
      for (uint32_t tries = 0; tries < (1u << 20) && !ok; ++tries)
        asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\nselp.u32 %0, 1, 0, q;\n}"
                     : "=r"(ok) : "r"(bar_a) : "memory");
      if (__syncthreads_or(!ok)) {                           // the copy never landed: the generic selection serves the unit
        if (tid == 0) report(p.status, SPEC_ERR_TIMEOUT);
        failed = true;
        staged = false;
      }
    }
    if (selects && !failed) {
      // ---- the floor, from one pooled position in every 16 of the staged scores
      const int n_groups = (g.e + (1 << kUnitSampleShift) - 1) >> kUnitSampleShift;
      for (int m = tid; m < n_groups; m += kSelThreads) {
        uint32_t hsh = ((uint32_t)unit * 0x9E3779B1u) ^ ((uint32_t)m * 0x85EBCA6Bu);
        hsh ^= hsh >> 15; hsh *= 0x2C1B3C6Du; hsh ^= hsh >> 12;
        const int q = (m << kUnitSampleShift) + (int)(hsh % (uint32_t)min(1 << kUnitSampleShift, g.e - (m << kUnitSampleShift)));
        const float* w7 = raw + 4 + (q + t.mis) - 3;         // slots outside the unit hold -inf
        const uint32_t key = to_key(fmax3(fmax3(w7[0], w7[1], w7[2]), fmax3(w7[3], w7[4], w7[5]), w7[6]));
        atomicAdd(&hist[key >> 21], 1u);
        skey[m] = key;
      }
      floor_key = floor_from_samples(skey, n_groups, hist, tk, kUnitSampleShift, wsum, out2);
      // ---- the sweep: candidates straight into shared memory
      const float floor_f = key_to_float(floor_key);
      const bool edge = t.mis > 0 || t.n_steps * 128 > t.X;
      uint32_t mask = edge ? sweep_steps<true, kSelWarps>(t, raw, floor_f, warp, lane) : sweep_steps<false, kSelWarps>(t, raw, floor_f, warp, lane);
      int total;
      int at = block_exclusive_scan(__popc(mask), wsum, total);
      if (total > p.held_cap) {
        failed = true;
      } else {
        n_cand = total;
        // step by step, the four pooled values again from three 16-byte reads (a walk over single
        // candidates would make the whole CTA wait for the thread with the most of them)
        const float4* base4 = reinterpret_cast<const float4*>(raw + 4);
#pragma unroll
        for (int k = 0; k < kMaxStepsPerWarp; ++k) {
          const uint32_t nib = (mask >> (4 * k)) & 15u;
          if (nib) {
            const int st = warp + k * kSelWarps;
            const float4* a4 = base4 + st * 32 + lane;
            const float4 pv = a4[-1], cv = a4[0], nv = a4[1];
            const float x[10] = {pv.y, pv.z, pv.w, cv.x, cv.y, cv.z, cv.w, nv.x, nv.y, nv.z};
            const float mid = fmax3(x[3], x[4], fmaxf(x[5], x[6])), l12 = fmaxf(x[1], x[2]), r78 = fmaxf(x[7], x[8]);
            const float v[4] = {fmax3(mid, x[0], l12), fmax3(mid, l12, x[7]), fmax3(mid, x[2], r78), fmax3(mid, r78, x[9])};
            const int j0 = st * 128 + lane * 4 - t.mis;                              // position of my first slot
#pragma unroll
            for (int u = 0; u < 4; ++u)
              if (nib & (1u << u)) held[at++] = make_uint2(to_key(v[u]), (uint32_t)(j0 + u));
          }
        }
      }
    }
  }
  __syncthreads();                                           // the staged scores are no longer read
  FinishMem fm;
  fm.cand = held;
  fm.bitmap_words = p.bitmap_words;
  fm.wsum = wsum; fm.out2 = out2; fm.lead = &lead[0][0];
  if (staged) {
    fm.hist = reinterpret_cast<uint32_t*>(raw);
    fm.map_gt = fm.hist + kStreamBins;
  } else {
    fm.hist = reinterpret_cast<uint32_t*>(held);             // unused by the generic selection
    fm.map_gt = reinterpret_cast<uint32_t*>(held);           // its scratch, away from the copy that may still land
  }
  fm.map_eq = fm.map_gt + p.bitmap_words;
  finish_unit(p, g, unit, fm, n_cand, n_cand, failed, true, floor_key);
}

// ------------------------------------------------------------------ host side ---------

// The one-CTA selection of short units.  *done = false: the shapes do not fit it.
static int run_unit_topk(const spec_problem* pr, const float* scores, int c_max, int n_forced_tail, int32_t* idx_out,
                         int32_t* count_out, int n_vert, int32_t* vert_out, int32_t* vert_count_out, int32_t* status_word,
                         cudaStream_t st, bool* done) {
  *done = false;
  const int max_len = max_seq_len(pr);
  // A unit is staged from the 16-byte boundary at or below its first score: up to three more slots,
  // none when every unit is known to start on such a boundary.
  const bool aligned = !pr->cu_seqlens && (reinterpret_cast<uintptr_t>(scores) & 15u) == 0 && pr->total_tokens % 4 == 0 &&
                       pr->n_in % 4 == 0;
  if (max_len < 1 || max_len + (aligned ? 0 : 3) > kUnitSlots) return SPEC_OK;
  const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;
  if (n_units < 1 || n_units > 0x7fffffff) return SPEC_OK;
  StreamParams p = {};
  p.scores = scores; p.cu = pr->cu_seqlens; p.T = pr->total_tokens; p.n_in = pr->n_in;
  p.L = pr->n_layers; p.H = pr->n_kv_heads; p.n_forced = n_forced_tail; p.c_max = c_max; p.n_vert = n_vert;
  p.chunk = kUnitSlots;
  p.chunks_max = 1;
  p.bitmap_words = ((max_len + 31) / 32 + 3) & ~3;
  p.max_len = max_len;
  // a denser sample than the streaming path's: the floor lets through about 1.6 times the budget
  p.held_cap = std::max((5 * std::max(c_max, n_vert) / 2 + 1024 + 3) & ~3, kUnitHeldMin);
  const size_t smem = (size_t)kUnitRawWords * 4 + (size_t)p.held_cap * 8;
  if (smem > (size_t)kSmemLimit - 1024) return SPEC_OK;
  p.idx_out = idx_out; p.count_out = count_out; p.vert_out = vert_out; p.vert_count_out = vert_count_out;
  p.status = status_word;
  static int set[64] = {0};
  int dev = 0;
  SPEC_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SPEC_OK;
  if (!__atomic_load_n(&set[dev], __ATOMIC_ACQUIRE)) {
    SPEC_CUDA_OK(cudaFuncSetAttribute(unit_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - 1024));
    __atomic_store_n(&set[dev], 1, __ATOMIC_RELEASE);
  }
  unit_select_kernel<<<(unsigned)n_units, kSelThreads, smem, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  *done = true;
  return SPEC_OK;
}

int run_stream_topk(const spec_problem* pr, const float* scores, int c_max, int n_forced_tail, int32_t* idx_out,
                    int32_t* count_out, int n_vert, int32_t* vert_out, int32_t* vert_count_out, void* workspace,
                    size_t workspace_bytes, int32_t* status_word, cudaStream_t st, bool* done) {
  *done = false;
  {
    // Short units, a few to an SM: one CTA does all of it.  Many more units than the GPU holds at once
    // are better streamed (the one-CTA kernel is a chain of latencies, the streaming one is not).
    const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;
    if (!workspace || n_units <= 592) {
      const int rc = run_unit_topk(pr, scores, c_max, n_forced_tail, idx_out, count_out, n_vert, vert_out, vert_count_out,
                                   status_word, st, done);
      if (rc != SPEC_OK || *done) return rc;
    }
  }
  if (!workspace) return SPEC_OK;
  const WorkspacePlan wp = plan_workspace(pr);
  if (workspace_bytes < wp.total) return SPEC_OK;
  const int max_len = max_seq_len(pr);
  if (max_len < 1) return SPEC_OK;
  const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;

  StreamParams p = {};
  p.scores = scores; p.cu = pr->cu_seqlens; p.T = pr->total_tokens; p.n_in = pr->n_in;
  p.L = pr->n_layers; p.H = pr->n_kv_heads; p.n_forced = n_forced_tail; p.c_max = c_max; p.n_vert = n_vert;
  // chunks of 4096 positions (a warp keeps its 8 steps of pooled values in registers), smaller
  // while that leaves SMs without a CTA
  int chunk = kSelChunkMax;
  static_assert(kSelChunkMax == kMaxStepsPerWarp * kSweepWarps * 128, "a sweeping warp keeps its steps in registers");
  while (chunk > kSelChunkMin && n_units * (((int64_t)max_len + 3 + chunk - 1) / chunk) < 1184) chunk >>= 1;
  p.chunk = chunk;
  p.chunks_max = (int)(((int64_t)max_len + 3 + chunk - 1) / chunk);
  if (p.chunks_max > kSelThreads) return SPEC_OK;          // the finishing CTA reads one segment count per thread
  p.bitmap_words = ((max_len + 31) / 32 + 3) & ~3;
  p.max_len = max_len;
  const size_t smem_sweep = (size_t)(chunk + 8 + 128) * 4;
  // the floor lets through about 1.6 to 2.5 times the budget (less for larger budgets)
  p.held_cap = (3 * std::max(c_max, n_vert) + 2048 + 3) & ~3;
  if (stream_finish_bytes(p.bitmap_words, p.held_cap) > (size_t)kSmemLimit - 1024) {
    // a large budget: what fits (the floor lets through about 1.6 times a budget of thousands)
    const int64_t room = ((int64_t)kSmemLimit - 1024 - (int64_t)stream_finish_bytes(p.bitmap_words, 0)) / 8;
    if (room < 2 * (int64_t)std::max(c_max, n_vert) + 2048) return SPEC_OK;   // too long or too large a budget for the finishing CTA
    p.held_cap = (int)(room & ~(int64_t)3);
  }
  const size_t smem_finish = stream_finish_bytes(p.bitmap_words, p.held_cap);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.head = reinterpret_cast<int32_t*>(ws + wp.sel_head_off);
  p.head_words = wp.sel_head_words;
  p.cand = reinterpret_cast<uint2*>(ws + wp.sel_cand_off);
  p.row_entries = wp.sel_row_entries;
  p.idx_out = idx_out; p.count_out = count_out; p.vert_out = vert_out; p.vert_count_out = vert_count_out;
  p.status = status_word;

  static int set[64] = {0};
  int dev = 0;
  SPEC_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SPEC_OK;
  if (!__atomic_load_n(&set[dev], __ATOMIC_ACQUIRE)) {
    SPEC_CUDA_OK(cudaFuncSetAttribute(stream_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - 1024));
    __atomic_store_n(&set[dev], 1, __ATOMIC_RELEASE);
  }
  sample_floor_kernel<<<(unsigned)n_units, kSelThreads, 0, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  if (pr->n_layers * pr->n_kv_heads > 65535) return SPEC_OK;   // rows are a grid dimension of the sweep
  const dim3 sweep_grid((unsigned)p.chunks_max, (unsigned)(pr->n_layers * pr->n_kv_heads), (unsigned)pr->n_seq);
  // The sweep and the finishing kernel are programmatic dependents of the kernel before them: they are
  // launched while it still runs and wait, in the kernel, where they first need its results.
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = st;
  cfg.attrs = pdl;
  cfg.numAttrs = 1;
  cfg.gridDim = sweep_grid;
  cfg.blockDim = dim3(kSweepThreads);
  cfg.dynamicSmemBytes = smem_sweep;
  SPEC_CUDA_OK(cudaLaunchKernelEx(&cfg, stream_sweep_kernel, p));
  cfg.gridDim = dim3((unsigned)n_units);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem_finish;
  SPEC_CUDA_OK(cudaLaunchKernelEx(&cfg, stream_finish_kernel, p));
  *done = true;
  return SPEC_OK;
}

}  // namespace spec
