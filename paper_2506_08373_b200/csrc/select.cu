// Pooling + exact top-C selection (Algorithm 1 lines 10 and 13) and the SpecPC keep set
// (Algorithm 2 lines 7-10).
//
// One CTA owns one (sequence, layer, KV head) unit (SpecPC: one sequence).  Pooled values
// are turned into order-preserving 32-bit keys; the C-th largest key is found by an MSB-first
// radix select with shared-memory histograms (one private histogram per warp, run-length
// aggregated updates), and the winners are emitted in ascending position by a chunked block
// scan, which also resolves ties at the threshold in favour of the lower position.  Keys are
// kept in shared memory when the unit fits; longer units recompute them from global memory in
// every pass.
#include "common.cuh"

namespace spec {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelVec = 4;                       // consecutive positions per thread in the ordered pass
constexpr int kSmemLimit = 227 * 1024;

// Monotone map float -> uint32 (larger float <=> larger key), valid for any sign.
__device__ __forceinline__ uint32_t to_key(float v) {
  const uint32_t b = __float_as_uint(v + 0.0f);            // -0.0 + 0.0 = +0.0: the two zeros tie, as they compare equal
  return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);   // negative: all bits flipped; else: sign bit set
}

// Pooled value of position j over the eligible range [0, e).
__device__ __forceinline__ float pooled_at(const float* __restrict__ s, int e, int j, int pool, int k) {
  int lo = j - (k >> 1);
  int hi = lo + k - 1;
  lo = lo < 0 ? 0 : lo;
  hi = hi > e - 1 ? e - 1 : hi;
  if (pool == SPEC_POOL_MAX) {
    float m = s[lo];
    for (int t = lo + 1; t <= hi; ++t) m = fmaxf(m, s[t]);
    return m;
  }
  float a = 0.f;
  for (int t = lo; t <= hi; ++t) a += s[t];
  return a / (float)k;
}

// Key source: shared-memory resident keys, or recomputation from the scores.
struct KeySource {
  const uint32_t* keys;       // non-NULL when resident
  const float* scores;
  int e, pool, k;
  __device__ __forceinline__ uint32_t operator()(int j) const {
    return keys ? keys[j] : to_key(pooled_at(scores, e, j, pool, k));
  }
};

struct SelectScratch {
  uint32_t* hist;             // [kSelWarps][256]
  int* misc;                  // [2*kSelWarps + 8]
};

// Finds the key T of the `need`-th largest element of key(0..e): count(key > T) < need <=
// count(key >= T).  Returns T and need_eq = need - count(key > T) (how many elements equal to
// T belong to the selection).  Requires 1 <= need <= e.  All threads of the CTA must call.
__device__ void radix_select(const KeySource& key, int e, int need, const SelectScratch& sc,
                             uint32_t& T_out, int& need_eq_out) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t prefix = 0, mask = 0;
  int remaining = need;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < kSelWarps * 256; i += kSelThreads) sc.hist[i] = 0;
    __syncthreads();
    uint32_t* myh = sc.hist + warp * 256;
    int run_d = -1, run_c = 0;
    for (int j = tid; j < e; j += kSelThreads) {
      const uint32_t kk = key(j);
      if ((kk & mask) == prefix) {
        const int dg = (kk >> shift) & 255;
        if (dg == run_d) {
          ++run_c;
        } else {
          if (run_c) atomicAdd(&myh[run_d], (uint32_t)run_c);
          run_d = dg;
          run_c = 1;
        }
      }
    }
    if (run_c) atomicAdd(&myh[run_d], (uint32_t)run_c);
    __syncthreads();
    if (tid < 256) {
      uint32_t tot = 0;
#pragma unroll
      for (int w = 0; w < kSelWarps; ++w) tot += sc.hist[w * 256 + tid];
      sc.hist[tid] = tot;
    }
    __syncthreads();
    if (warp == 0) {
      // lane owns bins [8*lane, 8*lane+8); suffix sums over lanes locate the digit.
      uint32_t b[8], s = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { b[i] = sc.hist[lane * 8 + i]; s += b[i]; }
      uint32_t suf = s;                                  // inclusive suffix sum over lanes >= lane
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += t;
      }
      const uint32_t above = suf - s;                    // elements in bins of higher lanes
      if (above < (uint32_t)remaining && (uint32_t)remaining <= suf) {
        uint32_t cum = above;
        int dg = 7;
        for (; dg > 0; --dg) {
          if (cum + b[dg] >= (uint32_t)remaining) break;
          cum += b[dg];
        }
        sc.misc[0] = lane * 8 + dg;
        sc.misc[1] = (int)cum;                           // elements strictly above the digit
      }
    }
    __syncthreads();
    const int dg = sc.misc[0];
    remaining -= sc.misc[1];
    prefix |= (uint32_t)dg << shift;
    mask |= 255u << shift;
    __syncthreads();
  }
  T_out = prefix;
  need_eq_out = remaining;
}

// Visits, in ascending position, every selected position j of [0, e): key > T, or key == T and
// fewer than need_eq equal keys precede it.  emit(rank, j) receives the 0-based rank in the
// ascending output.  Returns the number of selected positions.  All threads must call.
template <class Emit>
__device__ int ordered_emit(const KeySource& key, int e, uint32_t T, int need_eq, const SelectScratch& sc, Emit emit) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int base_gt = 0, base_eq = 0;
  int* wg = sc.misc + 8;
  int* we = sc.misc + 8 + kSelWarps;
  for (int c0 = 0; c0 < e; c0 += kSelThreads * kSelVec) {
    const int j0 = c0 + tid * kSelVec;
    uint32_t kk[kSelVec];
    int gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelVec; ++i) {
      const int j = j0 + i;
      kk[i] = j < e ? key(j) : 0u;
      if (j < e) { gt += kk[i] > T; eq += kk[i] == T; }
    }
    int sgt = gt, seq = eq;                               // inclusive warp scans
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, sgt, o);
      const int b = __shfl_up_sync(0xffffffffu, seq, o);
      if (lane >= o) { sgt += a; seq += b; }
    }
    if (lane == 31) { wg[warp] = sgt; we[warp] = seq; }
    __syncthreads();
    int pre_gt = base_gt + sgt - gt, pre_eq = base_eq + seq - eq, tot_gt = 0, tot_eq = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
      const int a = wg[w], b = we[w];
      if (w < warp) { pre_gt += a; pre_eq += b; }
      tot_gt += a;
      tot_eq += b;
    }
#pragma unroll
    for (int i = 0; i < kSelVec; ++i) {
      const int j = j0 + i;
      if (j < e) {
        if (kk[i] > T) {
          emit(pre_gt + min(pre_eq, need_eq), j);
          ++pre_gt;
        } else if (kk[i] == T) {
          if (pre_eq < need_eq) emit(pre_gt + pre_eq, j);
          ++pre_eq;
        }
      }
    }
    base_gt += tot_gt;
    base_eq += tot_eq;
    __syncthreads();
  }
  return base_gt + min(base_eq, need_eq);
}

struct TopkParams {
  const float* scores;
  const int32_t* cu;
  int32_t* idx_out;
  int32_t* count_out;
  int64_t T;
  int n_in, L, H, pool, pool_k, c_max, n_forced, cap;
};

// ------------------------------------------------------ streaming pool + top-C ------
//
// One CTA per (sequence, layer, KV head) unit, any length.  The unit's scores are read once.
// Every warp owns a contiguous range of positions and streams it on its own, kWarpStep
// positions per step, straight from global memory into registers (every lane loads its own
// eight scores with two 16-byte loads, the next steps' loads in flight while the current one
// is processed, and takes the three scores on either side from the neighbouring lanes by
// shuffle), with no CTA-wide barrier per step.  Every pooled key at or above a rising floor is
// counted in a shared histogram of the keys' top kTopBits bits and appended, in position order, to the warp's candidate list in
// shared memory; the floor is the bin that holds the C-th largest key of the positions seen so
// far and is raised at a few CTA-wide synchronisation points.  After the sweep the remaining
// bits are resolved by radix passes over the candidates only, and the winners are written in
// ascending position (warp lists are in position order and so is their concatenation).  If
// the candidates do not fit (many nearly equal scores, or c_max beyond a few thousand), the
// unit falls back to the generic multi-pass selection that recomputes keys from global memory.
constexpr int kPerThread = 8;                     // consecutive positions per thread and step
constexpr int kWarpStep = 32 * kPerThread;        // positions per warp and step
constexpr int kTopBits = 13;
constexpr int kTopBins = 1 << kTopBits;
constexpr int kTopHistWords = kTopBins + (kTopBins >> 8) * 4;   // four words of padding per 256 bins
constexpr int kCandCap = 7168;
constexpr int kWarpCap = kCandCap / kSelWarps;    // candidate entries per warp
constexpr int kFinBins = 1024;                    // histogram of the candidate passes (10 bits)

// Block-wide exclusive scan of one int per thread; total returned to every thread.
// wsum: kSelWarps ints of shared memory that no thread touches again before the CTA's next
// synchronisation after this call (callers alternate two buffers).  One __syncthreads.
__device__ __forceinline__ int block_exclusive_scan(int v, int* wsum, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  // every warp scans the kSelWarps (<= 32) warp totals itself
  int ws = lane < kSelWarps ? wsum[lane] : 0;
  int wincl = ws;
#pragma unroll
  for (int o = 1; o < kSelWarps; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, wincl, o);
    if (lane >= o) wincl += t;
  }
  total = __shfl_sync(0xffffffffu, wincl, kSelWarps - 1);
  const int before = __shfl_sync(0xffffffffu, wincl - ws, warp);
  return before + incl - v;
}

// Geometry of the sweep.  Positions are shifted by the unit's misalignment `mis` (0..3
// elements from a 16-byte boundary), x = position + mis, so that the positions of a thread and
// every 16-byte vector start on a 16-byte boundary of global memory.  Warp w streams
// x in [w * span, (w + 1) * span), span a multiple of kWarpStep.
struct SweepGeom {
  const float* src;       // score of position 0
  int e;                  // eligible positions [0, e)
  int mis, span, n_steps, pool, k;
};

__device__ __forceinline__ SweepGeom make_geom(const float* src, int e, int pool, int k) {
  SweepGeom g;
  g.src = src; g.e = e; g.pool = pool; g.k = k;
  g.mis = (int)((reinterpret_cast<uintptr_t>(src) >> 2) & 3u);
  const int per_warp = (e + g.mis + kSelWarps - 1) / kSelWarps;
  g.n_steps = (per_warp + kWarpStep - 1) / kWarpStep;
  g.span = g.n_steps * kWarpStep;
  return g;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Four scores starting at position p_first (a multiple of four elements from a 16-byte boundary);
// positions outside [0, e) read as -infinity.
__device__ __forceinline__ float4 load4(const SweepGeom& g, int p_first) {
  if (p_first >= 0 && p_first + 3 < g.e) return __ldg(reinterpret_cast<const float4*>(g.src + p_first));
  float t[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int pp = p_first + q;
    t[q] = (pp >= 0 && pp < g.e) ? __ldg(g.src + pp) : -INFINITY;
  }
  return make_float4(t[0], t[1], t[2], t[3]);
}

// Max-pool of width 7 for a lane's eight positions from its own eight scores w (elements 0..7),
// the three scores before them (l) and the three after them (r).
__device__ __forceinline__ void pool_max7_halo(const float (&l)[3], const float4 (&w4)[2], const float (&r)[3], float (&val)[kPerThread]) {
  const float x[14] = {l[0], l[1], l[2], w4[0].x, w4[0].y, w4[0].z, w4[0].w, w4[1].x, w4[1].y, w4[1].z, w4[1].w, r[0], r[1], r[2]};
  float t3[12];
#pragma unroll
  for (int i = 0; i < 12; ++i) t3[i] = fmax3(x[i], x[i + 1], x[i + 2]);
#pragma unroll
  for (int u = 0; u < kPerThread; ++u) val[u] = fmax3(t3[u], t3[u + 3], x[u + 6]);
}

// Word of bin b in the top-bits histogram: every lane of a warp scans 256 consecutive bins
// with 16-byte loads, and the padding staggers the lanes over the memory banks.
__device__ __forceinline__ int top_word(uint32_t b) { return (int)(b + ((b >> 8) << 2)); }

// Finds the bin holding the need-th largest element of a histogram whose bins are spread
// over the threads, bins_per_thread consecutive bins each starting at my_bins (need >= 1).  Returns the bin and
// the number of elements in higher bins to every thread; false (outputs untouched) when the
// histogram holds fewer than `need` elements.
__device__ __forceinline__ bool locate_bin(const uint32_t* my_bins, int bins_per_thread, int need, int* wsum, int* out2,
                                           int& bin, int& above) {
  const int b0 = threadIdx.x * bins_per_thread;
  __syncthreads();                                         // histogram complete, wsum free
  if (threadIdx.x == 0) out2[0] = -1;
  int mine = 0;
  for (int i = 0; i < bins_per_thread; ++i) mine += (int)my_bins[i];
  int total;
  const int below = block_exclusive_scan(mine, wsum, total);
  const int over = total - below - mine;                   // elements in bins above my range
  if (over < need && need <= over + mine) {
    int cum = over, b = bins_per_thread - 1;
    for (; b > 0; --b) {
      const int hcount = (int)my_bins[b];
      if (cum + hcount >= need) break;
      cum += hcount;
    }
    out2[0] = b0 + b;
    out2[1] = cum;
  }
  __syncthreads();
  const int found = out2[0];
  const int cum = out2[1];
  __syncthreads();
  if (found < 0) return false;
  bin = found;
  above = cum;
  return true;
}

// Shared memory: top histogram, candidate keys and positions, candidate-pass histogram, a few
// words of bookkeeping, then the parked groups (values and first positions) of all warps.
constexpr int kTopkPendOffset = (kTopHistWords * 4 + 2 * kCandCap * 4 + kFinBins * 4 + (2 * kSelWarps + 2 + 1) * 4 + 15) / 16 * 16;
constexpr int kTopkSmemBytes = kTopkPendOffset + kSelWarps * 32 * (kPerThread + 1) * 4;

__global__ void __launch_bounds__(kSelThreads, 2) pool_topk_kernel(TopkParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint32_t* top_hist = reinterpret_cast<uint32_t*>(smem_raw);            // histogram of the keys' top bits
  uint32_t* cand_key = top_hist + kTopHistWords;                        // [kSelWarps][kWarpCap]
  int32_t* cand_idx = reinterpret_cast<int32_t*>(cand_key + kCandCap);
  uint32_t* fin_hist = reinterpret_cast<uint32_t*>(cand_idx + kCandCap); // candidate passes
  int* wsum = reinterpret_cast<int*>(fin_hist + kFinBins);              // kSelWarps, then two results, then flags
  int* out2 = wsum + kSelWarps;
  int* wcnt = out2 + 2;                                                  // [kSelWarps] list lengths, then the overflow flag
  int* overflow = wcnt + kSelWarps;
  float* pend = reinterpret_cast<float*>(smem_raw + kTopkPendOffset);    // parked groups of all warps

  const int unit = blockIdx.x;
  const int h = unit % p.H, l = (unit / p.H) % p.L, s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int forced = min(p.n_forced, n);
  const int e = n - forced;
  const int take = min(p.c_max - forced, e);
  int32_t* idx = p.idx_out + (int64_t)unit * p.c_max;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const float* src = p.scores + ((int64_t)l * p.H + h) * p.T + begin;

  if (take > 0 && take < e) {
    const SweepGeom g = make_geom(src, e, p.pool, p.pool_k);
    for (int i = tid; i < kTopHistWords; i += kSelThreads) top_hist[i] = 0;
    if (tid == 0) *overflow = 0;
    __syncthreads();
    uint32_t* ck = cand_key + warp * kWarpCap;
    int32_t* ci = cand_idx + warp * kWarpCap;
    const bool max7 = g.pool == SPEC_POOL_MAX && g.k == 7;
    // ---- the sweep.  The take-th largest key of the positions seen so far can only be below
    // that of the whole unit, so the bin that holds it is a floor: keys under it are out.
    uint32_t floor_key = 0;
    uint32_t early_floor = 0;                                // highest floor taken from a part of the unit
    int cnt = 0;                                             // entries in my warp's list (warp-uniform)
    const int x_warp = warp * g.span + lane * kPerThread;

    // One step of my warp: the pooled values of positions p0 .. p0 + 7 of every lane.
    // Raises my warp's floor to the bin that holds the take-th largest of the keys counted so
    // far, read from the shared histogram without stopping the other warps.  Their updates can
    // only add keys, so the bin found is still a lower bound.
    auto warp_refloor = [&]() {
      constexpr int kBinsPerLane = kTopBins / 32;
      static_assert(kBinsPerLane == 256, "the padding of the histogram assumes 256 bins per lane");
      const uint32_t* hb = top_hist + lane * (kBinsPerLane + 4);
      int mine = 0;
      for (int i = 0; i < kBinsPerLane; i += 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(hb + i);
        mine += (int)(v.x + v.y + v.z + v.w);
      }
      int suffix = mine;                                     // keys in my bins and in those of higher lanes
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_down_sync(0xffffffffu, suffix, o);
        if (lane + o < 32) suffix += t;
      }
      const bool here = suffix - mine < take && take <= suffix;
      int bin = -1;
      if (here) {
        int cum = suffix - mine;
        bin = kBinsPerLane - 1;
        for (; bin > 0; --bin) {
          cum += (int)hb[bin];
          if (cum >= take) break;
        }
        bin += lane * kBinsPerLane;
      }
      const uint32_t who = __ballot_sync(0xffffffffu, here);
      if (who) {
        const uint32_t fk = (uint32_t)__shfl_sync(0xffffffffu, bin, __ffs(who) - 1) << (32 - kTopBits);
        if (fk > floor_key) floor_key = fk;
      }
    };

    // Ordered in-place filter of my warp's list against the current floor.
    auto filter_list = [&]() {
      int kept = 0;
      for (int r = 0; r < cnt; r += 32) {
        const int i = r + lane;
        const uint32_t kk = i < cnt ? ck[i] : 0u;
        const int32_t ix = i < cnt ? ci[i] : 0;
        const bool keep = i < cnt && kk >= floor_key;
        const uint32_t bal = __ballot_sync(0xffffffffu, keep);
        __syncwarp();                                      // every lane holds its entry before any is overwritten
        if (keep) { const int w = kept + __popc(bal & lt_mask); ck[w] = kk; ci[w] = ix; }
        kept += __popc(bal);
        __syncwarp();
      }
      cnt = kept;
    };

    // Groups (the eight pooled values of one lane and one step) that hold at least one key at
    // or above the floor are parked in a small per-warp buffer and dealt with 32 at a time,
    // one group per lane, so that the per-key work runs with full warps instead of once per
    // step for a handful of keys.
    float* pend_val = pend + warp * (32 * kPerThread);      // [32 groups][8 values]
    int* pend_p0 = reinterpret_cast<int*>(pend + kSelWarps * 32 * kPerThread) + warp * 32;
    int n_pend = 0;                                          // parked groups (warp-uniform)

    auto expand = [&]() {
      if (n_pend == 0) return;
      const bool have = lane < n_pend;
      float val[kPerThread];
      const float4 v0 = *reinterpret_cast<const float4*>(pend_val + lane * kPerThread);
      const float4 v1 = *reinterpret_cast<const float4*>(pend_val + lane * kPerThread + 4);
      val[0] = v0.x; val[1] = v0.y; val[2] = v0.z; val[3] = v0.w;
      val[4] = v1.x; val[5] = v1.y; val[6] = v1.z; val[7] = v1.w;
      const int p0 = pend_p0[lane];
      uint32_t take_mask = 0;
      if (have) {
#pragma unroll
        for (int u = 0; u < kPerThread; ++u)
          if (to_key(val[u]) >= floor_key && (unsigned)(p0 + u) < (unsigned)e) take_mask |= 1u << u;
      }
      const int mine = __popc(take_mask);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const int total = __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
      for (int u = 0; u < kPerThread; ++u)
        if (take_mask & (1u << u)) atomicAdd(&top_hist[top_word(to_key(val[u]) >> (32 - kTopBits))], 1u);
      if (cnt + total > kWarpCap) filter_list();
      if (cnt + total > kWarpCap) { warp_refloor(); filter_list(); }   // my list alone is too long: fresher floor
      if (cnt + total <= kWarpCap) {
        int at = cnt + incl - mine;
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) {
          if (take_mask & (1u << u)) {
            ck[at] = to_key(val[u]);
            ci[at] = p0 + u;
            ++at;
          }
        }
        cnt += total;
      } else if (lane == 0) {
        *overflow = 1;                                       // the list is lost: the unit takes the generic path
      }
      n_pend = 0;
      __syncwarp();
    };

    // One step of my warp: the pooled values of positions p0 .. p0 + 7 of every lane.
    auto process = [&](const float (&val)[kPerThread], int p0, int st) {
      const float vmax = fmax3(fmax3(val[0], val[1], val[2]), fmax3(val[3], val[4], val[5]), fmaxf(val[6], val[7]));
      const bool hot = p0 + kPerThread > 0 && p0 < e && to_key(vmax) >= floor_key;
      const uint32_t hot_lanes = __ballot_sync(0xffffffffu, hot);
      if (hot_lanes) {
        const int n_hot = __popc(hot_lanes);
        if (n_pend + n_hot > 32) expand();
        if (hot) {
          const int slot = n_pend + __popc(hot_lanes & lt_mask);
          *reinterpret_cast<float4*>(pend_val + slot * kPerThread) = make_float4(val[0], val[1], val[2], val[3]);
          *reinterpret_cast<float4*>(pend_val + slot * kPerThread + 4) = make_float4(val[4], val[5], val[6], val[7]);
          pend_p0[slot] = p0;
        }
        n_pend += n_hot;
        __syncwarp();
      }
      // Floor updates after steps 0, 3, 15, 63, then every 64th; none after the last step, the
      // final selection follows it anyway.
      const bool refloor = ((((st + 1) & st) == 0 && (__popc(st) & 1) == 0) || (st & 63) == 63) && st + 1 < g.n_steps;
      if (refloor) expand();                                 // the histogram must be complete for the floor
      if (refloor) {
        // While only a fraction f of the unit has been seen, the floor is taken at rank 2 f take + 64
        // of the keys seen instead of rank take: about f take of them are expected above the final
        // threshold, so this bin is below it unless the large keys crowd into the part seen first.
        // That case leaves fewer than `take` candidates at the end, which the final selection
        // detects and hands to the generic path; the result is exact either way.
        int fb, ab;
        const long long seen = (long long)(st + 1) * (kWarpStep * kSelWarps);
        const int need = seen >= e ? take : min(take, (int)(2 * ((long long)take * seen / e)) + 64);
        if (locate_bin(top_hist + top_word(tid * (kTopBins / kSelThreads)), kTopBins / kSelThreads, need, wsum, out2, fb, ab)) {
          floor_key = max(floor_key, (uint32_t)fb << (32 - kTopBits));
          early_floor = max(early_floor, (uint32_t)fb << (32 - kTopBits));    // the same in every thread of the CTA
        }
      }
    };

    if (max7) {
      // Every lane loads its own eight scores of a step (two 16-byte loads, kAhead steps in
      // flight); the three scores on either side come from the neighbouring lanes by shuffle.
      // Lane 0 takes them from lane 31 of the warp's previous step (kept in `carry`; before the
      // first step they are loaded), lane 31 loads the four scores that follow its own.
      constexpr int kAhead = 2;                            // steps in flight (three or four spill under the 64-register cap)
      float4 w[kAhead][2];
#pragma unroll
      for (int sidx = 0; sidx < kAhead; ++sidx) {
        if (sidx < g.n_steps) {
          const int pf = x_warp + sidx * kWarpStep - g.mis;
          w[sidx][0] = load4(g, pf);
          w[sidx][1] = load4(g, pf + 4);
        }
      }
      float carry[3];
      {
        const int pb = warp * g.span - g.mis - 3;            // the three positions before my warp's range
#pragma unroll
        for (int q = 0; q < 3; ++q) carry[q] = (pb + q >= 0 && pb + q < e) ? __ldg(src + pb + q) : -INFINITY;
      }
      for (int st = 0; st < g.n_steps; st += kAhead) {
#pragma unroll
        for (int sidx = 0; sidx < kAhead; ++sidx) {
          if (st + sidx < g.n_steps) {                       // warp-uniform
            const int pf = x_warp + (st + sidx) * kWarpStep - g.mis;    // my first position
            const float4 (&cur)[2] = w[sidx];
            float4 after = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lane == 31) after = load4(g, pf + 8);
            float l[3], r[3];
            l[0] = __shfl_up_sync(0xffffffffu, cur[1].y, 1);
            l[1] = __shfl_up_sync(0xffffffffu, cur[1].z, 1);
            l[2] = __shfl_up_sync(0xffffffffu, cur[1].w, 1);
            r[0] = __shfl_down_sync(0xffffffffu, cur[0].x, 1);
            r[1] = __shfl_down_sync(0xffffffffu, cur[0].y, 1);
            r[2] = __shfl_down_sync(0xffffffffu, cur[0].z, 1);
            if (lane == 0) { l[0] = carry[0]; l[1] = carry[1]; l[2] = carry[2]; }
            if (lane == 31) { r[0] = after.x; r[1] = after.y; r[2] = after.z; }
            carry[0] = __shfl_sync(0xffffffffu, cur[1].y, 31);
            carry[1] = __shfl_sync(0xffffffffu, cur[1].z, 31);
            carry[2] = __shfl_sync(0xffffffffu, cur[1].w, 31);
            float val[kPerThread];
            pool_max7_halo(l, cur, r, val);
            if (st + sidx + kAhead < g.n_steps) {
              const int pn = pf + kAhead * kWarpStep;
              w[sidx][0] = load4(g, pn);
              w[sidx][1] = load4(g, pn + 4);
            }
            process(val, pf, st + sidx);
          }
        }
      }
    } else {
      // any other pooling: windows read element by element (L1 serves the overlap)
      for (int st = 0; st < g.n_steps; ++st) {
        const int p0 = x_warp + st * kWarpStep - g.mis;
        float val[kPerThread];
#pragma unroll
        for (int u = 0; u < kPerThread; ++u)
          val[u] = (unsigned)(p0 + u) < (unsigned)e ? pooled_at(src, e, p0 + u, g.pool, g.k) : 0.f;
        process(val, p0, st);
      }
    }
    expand();
    if (lane == 0) wcnt[warp] = cnt;
    int b1 = 0, above = 0;
    bool fits = locate_bin(top_hist + top_word(tid * (kTopBins / kSelThreads)), kTopBins / kSelThreads, take, wsum, out2, b1, above);   // fails on NaN scores or when an early floor was too high
    // Below an early floor the histogram and the lists are incomplete: a threshold bin found there
    // means that floor was too high.
    fits = fits && *overflow == 0 && ((uint32_t)b1 << (32 - kTopBits)) >= early_floor;
    if (fits) {
      // ---- remaining bits on the candidates only (every warp walks its own list)
      int known = kTopBits;
      uint32_t prefix = (uint32_t)b1 << (32 - kTopBits);
      uint32_t mask = ~((1u << (32 - kTopBits)) - 1u);
      int remaining = take - above;
      while (known < 32) {
        const int w = min(10, 32 - known), shift = 32 - known - w;
        for (int i = tid; i < kFinBins; i += kSelThreads) fin_hist[i] = 0;
        __syncthreads();
        for (int i = lane; i < cnt; i += 32) {
          const uint32_t kk = ck[i];
          if ((kk & mask) == prefix) atomicAdd(&fin_hist[(kk >> shift) & ((1u << w) - 1u)], 1u);
        }
        int dg, ab;
        locate_bin(fin_hist + tid * (kFinBins / kSelThreads), kFinBins / kSelThreads, remaining, wsum, out2, dg, ab);
        remaining -= ab;
        prefix |= (uint32_t)dg << shift;
        mask |= ((1u << w) - 1u) << shift;
        known += w;
      }
      // ---- ordered emission: key > T, or key == T among the first `remaining` equal keys
      const uint32_t T = prefix;
      const int need_eq = remaining;
      int gt = 0, eq = 0;
      for (int i = lane; i < cnt; i += 32) { const uint32_t kk = ck[i]; gt += kk > T; eq += kk == T; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, o);
        eq += __shfl_xor_sync(0xffffffffu, eq, o);
      }
      __syncthreads();                                     // wcnt no longer needed: reuse it for (gt, eq) per warp
      if (lane == 0) wcnt[warp] = gt | (eq << 16);         // a list holds at most kWarpCap < 2^16 entries
      __syncthreads();
      int pre_gt = 0, pre_eq = 0;
      for (int w = 0; w < warp; ++w) { const int x = wcnt[w]; pre_gt += x & 0xffff; pre_eq += x >> 16; }
      for (int r = 0; r < cnt; r += 32) {
        const int i = r + lane;
        const uint32_t kk = i < cnt ? ck[i] : 0u;
        const bool is_gt = i < cnt && kk > T, is_eq = i < cnt && kk == T;
        const uint32_t bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
        const int my_gt = pre_gt + __popc(bg & lt_mask), my_eq = pre_eq + __popc(be & lt_mask);
        if (is_gt) idx[my_gt + min(my_eq, need_eq)] = ci[i];
        else if (is_eq && my_eq < need_eq) idx[my_gt + my_eq] = ci[i];
        pre_gt += __popc(bg);
        pre_eq += __popc(be);
      }
    } else {
      // ---- candidates lost or too many keys share the leading bits: generic selection
      __syncthreads();
      SelectScratch sc;
      sc.hist = cand_key;                                  // 16 KB + a few words of the 64 KB of the candidate lists
      sc.misc = reinterpret_cast<int*>(sc.hist + kSelWarps * 256);
      KeySource key;
      key.scores = src;
      key.e = e; key.pool = p.pool; key.k = p.pool_k;
      key.keys = nullptr;
      uint32_t T;
      int need_eq;
      radix_select(key, e, take, sc, T, need_eq);
      ordered_emit(key, e, T, need_eq, sc, [&](int rank, int j) { idx[rank] = j; });
    }
  } else {
    for (int c = tid; c < take; c += kSelThreads) idx[c] = c;      // every eligible position is kept
  }
  for (int c = take + tid; c < p.c_max; c += kSelThreads) idx[c] = (c - take < forced) ? e + (c - take) : -1;
  if (p.count_out && tid == 0) p.count_out[unit] = take + forced;
}


// ---------------------------------------------------------------------- SpecPC ------

// Token score: reduction over all layers and KV heads, in (layer, head) order.
__global__ void __launch_bounds__(256) token_reduce_kernel(const float* __restrict__ scores, float* __restrict__ tok,
                                                           int64_t T, int n_vec, int reduce) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const float* src = scores + t;
  float acc = reduce == SPEC_REDUCE_SUM ? 0.f : -INFINITY;
  int i = 0;
  for (; i + 8 <= n_vec; i += 8) {
    float x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) x[u] = __ldg(src + (int64_t)(i + u) * T);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc = reduce == SPEC_REDUCE_SUM ? acc + x[u] : fmaxf(acc, x[u]);
  }
  for (; i < n_vec; ++i) {
    const float x = __ldg(src + (int64_t)i * T);
    acc = reduce == SPEC_REDUCE_SUM ? acc + x : fmaxf(acc, x);
  }
  tok[t] = acc;
}

// First stage of Algorithm 2 lines 8-9 in the printed order: the average pool of the token
// scores over each sequence's eligible range, written to a second vector.
__global__ void __launch_bounds__(256) token_avgpool_kernel(const float* __restrict__ tok, float* __restrict__ out,
                                                            const int32_t* __restrict__ cu, int n_in, int n_seq,
                                                            int n_forced, int k) {
  const int s = blockIdx.y;
  int begin, n;
  seq_range(cu, n_in, s, begin, n);
  const int e = n - min(n_forced, n);
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < e; j += gridDim.x * blockDim.x)
    out[begin + j] = pooled_at(tok + begin, e, j, SPEC_POOL_AVG, k);
}

struct KeepParams {
  const float* tok;
  const int32_t* cu;
  int32_t* keep_out;
  int32_t* n_keep_out;
  int n_in, pool, pool_k, c_max, n_neighbor, n_forced, keep_capacity, cap, bitmap_words;
  int32_t* status;
};

__global__ void __launch_bounds__(kSelThreads) specpc_keep_kernel(KeepParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  SelectScratch sc;
  sc.hist = reinterpret_cast<uint32_t*>(smem_raw);
  sc.misc = reinterpret_cast<int*>(sc.hist + kSelWarps * 256);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(sc.misc + 2 * kSelWarps + 8);
  uint32_t* keys = bitmap + p.bitmap_words;

  const int s = blockIdx.x;
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int forced = min(p.n_forced, n);
  const int e = n - forced;
  const int take = min(p.c_max, e);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int32_t* keep = p.keep_out + (int64_t)s * p.keep_capacity;
  const int n_words = (n + 31) >> 5;

  for (int w = tid; w < n_words; w += kSelThreads) bitmap[w] = 0;
  __syncthreads();

  auto mark = [&](int lo, int hi) {                       // set bits lo..hi (inclusive)
    for (int w = lo >> 5; w <= (hi >> 5); ++w) {
      const int b0 = max(lo, w << 5) & 31, b1 = min(hi, (w << 5) + 31) & 31;
      const uint32_t m = (0xffffffffu >> (31 - b1)) & (0xffffffffu << b0);
      atomicOr(&bitmap[w], m);
    }
  };

  if (take > 0 && take < e) {
    KeySource key;
    key.scores = p.tok + begin;
    key.e = e; key.pool = p.pool; key.k = p.pool_k;
    key.keys = nullptr;
    if (e <= p.cap) {
      if (p.pool == SPEC_POOL_MAX && p.pool_k == 7) {
        // width-7 maximum with the loads of eight positions per thread in flight at once;
        // positions outside [0, e) read as -infinity
        const float* src = p.tok + begin;
        for (int j0 = tid; j0 < e; j0 += 8 * kSelThreads) {
          float w[8][7];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int t = 0; t < 7; ++t) {
              const int q = j0 + u * kSelThreads + t - 3;
              w[u][t] = (q >= 0 && q < e) ? __ldg(src + q) : -INFINITY;
            }
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * kSelThreads;
            if (j < e) keys[j] = to_key(fmax3(fmax3(w[u][0], w[u][1], w[u][2]), fmax3(w[u][3], w[u][4], w[u][5]), w[u][6]));
          }
        }
      } else {
        for (int j = tid; j < e; j += kSelThreads) keys[j] = key(j);
      }
      key.keys = keys;
      __syncthreads();
    }
    const int nb = p.n_neighbor;
    if (key.keys) {
      // Resident keys: three radix passes (11, 11, 10 bits) find the key T of the take-th largest
      // position.  Thread t looks at positions t, t + 512, ..., so the lanes of a warp hold
      // consecutive positions and the runs of equal digits that pooling produces are merged into
      // one histogram update by ballot.  Marking needs no order for keys above T; of the keys
      // equal to T the first need_eq by position are found with a scan over the warps' ballots.
      uint32_t* hist = sc.hist;
      int* out2 = sc.misc;
      int* wsum = sc.misc + 8;
      const uint32_t lt_mask = (1u << lane) - 1u;
      const int rows = (e + kSelThreads - 1) / kSelThreads;
      uint32_t prefix = 0, mask = 0;
      int remaining = take;
#pragma unroll 1
      for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
        const int bins = pass == 2 ? 1024 : 2048;
        for (int b = tid; b < bins; b += kSelThreads) hist[b] = 0;
        __syncthreads();
        for (int i = 0; i < rows; ++i) {
          const int j = i * kSelThreads + tid;
          const uint32_t kk = j < e ? keys[j] : 0u;
          const bool in = j < e && (kk & mask) == prefix;
          const uint32_t dg = (kk >> shift) & (uint32_t)(bins - 1);
          const uint32_t dg_prev = __shfl_up_sync(0xffffffffu, dg, 1);
          const uint32_t ins = __ballot_sync(0xffffffffu, in);
          const bool head = in && (lane == 0 || !((ins >> (lane - 1)) & 1u) || dg_prev != dg);
          const uint32_t heads = __ballot_sync(0xffffffffu, head);
          if (head) {
            const uint32_t stop = (heads | ~ins) & ~(lt_mask | (1u << lane));   // next run, or a lane that is out
            atomicAdd(&hist[dg], (uint32_t)((stop ? __ffs(stop) - 1 : 32) - lane));
          }
        }
        int dg, ab;
        locate_bin(hist + tid * (bins / kSelThreads), bins / kSelThreads, remaining, wsum, out2, dg, ab);
        remaining -= ab;
        prefix |= (uint32_t)dg << shift;
        mask |= (uint32_t)(bins - 1) << shift;
      }
      const uint32_t T = prefix;
      const int need_eq = remaining;
      uint32_t* eqm = sc.hist;                               // [rows][kSelWarps] ballots of the keys equal to T
      for (int i = 0; i < rows; ++i) {
        const int j = i * kSelThreads + tid;
        const uint32_t kk = j < e ? keys[j] : 0u;
        if (j < e && kk > T) mark(max(j - nb, 0), min(j + nb, e - 1));
        const uint32_t be = __ballot_sync(0xffffffffu, j < e && kk == T);
        if (lane == 0) eqm[i * kSelWarps + warp] = be;
      }
      __syncthreads();
      const int n_ent = rows * kSelWarps;
      const int ept = (n_ent + kSelThreads - 1) / kSelThreads;
      const int e0 = tid * ept, e1 = min(e0 + ept, n_ent);
      int mine = 0;
      for (int en = e0; en < e1; ++en) mine += __popc(eqm[en]);
      int total_eq;
      int before = block_exclusive_scan(mine, wsum + kSelWarps, total_eq);
      for (int en = e0; en < e1 && before < need_eq; ++en) {
        uint32_t bits = eqm[en];
        const int base = (en / kSelWarps) * kSelThreads + (en % kSelWarps) * 32;
        while (bits && before < need_eq) {
          const int j = base + __ffs(bits) - 1;
          bits &= bits - 1;
          mark(max(j - nb, 0), min(j + nb, e - 1));
          ++before;
        }
      }
    } else {
      uint32_t T;
      int need_eq;
      radix_select(key, e, take, sc, T, need_eq);
      ordered_emit(key, e, T, need_eq, sc, [&](int, int j) { mark(max(j - nb, 0), min(j + nb, e - 1)); });
    }
  } else if (take > 0) {
    for (int w = tid; w < ((e + 31) >> 5); w += kSelThreads) {
      const int hi = min(e - 1, (w << 5) + 31);
      mark(w << 5, hi);
    }
  }
  __syncthreads();
  if (forced > 0) {
    for (int j = e + tid; j < n; j += kSelThreads) mark(j, j);
    __syncthreads();
  }

  // Ordered extraction of the set bits: every thread owns a run of consecutive words.
  const int wpt = (n_words + kSelThreads - 1) / kSelThreads;
  const int w0 = tid * wpt, w1 = min(w0 + wpt, n_words);
  int cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
  int sc_incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, sc_incl, o);
    if (lane >= o) sc_incl += a;
  }
  int* wt = sc.misc + 8;
  if (lane == 31) wt[warp] = sc_incl;
  __syncthreads();
  int pos = sc_incl - cnt, total = 0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) {
    if (w < warp) pos += wt[w];
    total += wt[w];
  }
  for (int w = w0; w < w1; ++w) {
    uint32_t bits = bitmap[w];
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if (pos < p.keep_capacity) keep[pos] = (w << 5) + b;
      ++pos;
    }
  }
  if (total > p.keep_capacity && tid == 0) report(p.status, SPEC_ERR_BAD_ARG);
  const int kept = min(total, p.keep_capacity);
  for (int c = kept + tid; c < p.keep_capacity; c += kSelThreads) keep[c] = -1;
  if (tid == 0) p.n_keep_out[s] = kept;
}

static int select_smem_bytes(int max_len, int bitmap_words, int* cap_out) {
  const int fixed = kSelWarps * 256 * 4 + (2 * kSelWarps + 8) * 4 + bitmap_words * 4;
  int cap = (kSmemLimit - fixed) / 4;
  cap &= ~3;
  if (cap < 0) cap = 0;
  int want = max_len <= cap ? max_len : 0;                 // longer units stream from global memory
  *cap_out = want;
  return fixed + want * 4;
}

static int check_pool_args(int pool, int pool_k, int c_max, int n_forced_tail, bool two_stage_ok = false) {
  if (pool != SPEC_POOL_MAX && pool != SPEC_POOL_AVG && !(two_stage_ok && pool == SPEC_POOL_AVG_THEN_MAX))
    return fail(SPEC_ERR_BAD_ARG, "pool=%d is not a spec_pool value this call accepts", pool);
  if (pool_k < 1 || pool_k > 255) return fail(SPEC_ERR_BAD_ARG, "pool_k=%d outside [1, 255]", pool_k);
  if (c_max < 1) return fail(SPEC_ERR_BAD_ARG, "c_max=%d must be >= 1", c_max);
  if (n_forced_tail < 0) return fail(SPEC_ERR_BAD_ARG, "n_forced_tail=%d is negative", n_forced_tail);
  return SPEC_OK;
}

}  // namespace spec

SPEC_EXPORT int32_t spec_pool_topk(const spec_problem* pr, const float* scores, int32_t pool, int32_t pool_k,
                                   int32_t c_max, int32_t n_forced_tail, int32_t* idx_out, int32_t* count_out,
                                   void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  using namespace spec;
  (void)workspace; (void)workspace_bytes; (void)status_word;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !idx_out) return fail(SPEC_ERR_BAD_ARG, "scores and idx_out must not be NULL");
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail);
  if (rc != SPEC_OK) return rc;
  if (n_forced_tail > c_max) return fail(SPEC_ERR_BAD_ARG, "n_forced_tail=%d exceeds c_max=%d", n_forced_tail, c_max);
  rc = check_device();
  if (rc != SPEC_OK) return rc;

  TopkParams p;
  p.scores = scores; p.cu = pr->cu_seqlens; p.idx_out = idx_out; p.count_out = count_out;
  p.T = pr->total_tokens; p.n_in = pr->n_in; p.L = pr->n_layers; p.H = pr->n_kv_heads;
  p.pool = pool; p.pool_k = pool_k; p.c_max = c_max; p.n_forced = n_forced_tail;
  p.cap = 0;
  const int smem = kTopkSmemBytes;
  SPEC_CUDA_OK(cudaFuncSetAttribute(pool_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  const unsigned n_units = (unsigned)(pr->n_seq * pr->n_layers * pr->n_kv_heads);
  pool_topk_kernel<<<n_units, kSelThreads, smem, static_cast<cudaStream_t>(stream)>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}

SPEC_EXPORT int32_t specpc_token_select(const spec_problem* pr, const float* scores, int32_t layer_head_reduce,
                                        int32_t pool, int32_t pool_k, int32_t c_max, int32_t n_neighbor,
                                        int32_t n_forced_tail, int32_t* keep_out, int32_t keep_capacity,
                                        int32_t* n_keep_out, void* workspace, size_t workspace_bytes,
                                        int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !keep_out || !n_keep_out) return fail(SPEC_ERR_BAD_ARG, "scores, keep_out and n_keep_out must not be NULL");
  if (layer_head_reduce != SPEC_REDUCE_SUM && layer_head_reduce != SPEC_REDUCE_MAX)
    return fail(SPEC_ERR_BAD_ARG, "layer_head_reduce=%d is not a spec_reduce value", layer_head_reduce);
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail, true);
  if (rc != SPEC_OK) return rc;
  if (n_neighbor < 0) return fail(SPEC_ERR_BAD_ARG, "n_neighbor=%d is negative", n_neighbor);
  const int max_len = max_seq_len(pr);
  const bool two_stage = pool == SPEC_POOL_AVG_THEN_MAX;
  if (two_stage && n_neighbor > 255) return fail(SPEC_ERR_BAD_ARG, "n_neighbor=%d as a pooling width exceeds 255", n_neighbor);
  const int64_t worst = two_stage ? (int64_t)c_max + n_forced_tail : (int64_t)c_max * (2 * (int64_t)n_neighbor + 1) + n_forced_tail;
  const int64_t need_cap = worst < max_len ? worst : max_len;
  if (keep_capacity < need_cap)
    return fail(SPEC_ERR_BAD_ARG, "keep_capacity=%d is below the worst case %lld", keep_capacity, (long long)need_cap);
  const WorkspacePlan wp = plan_workspace(pr);
  if (!workspace || workspace_bytes < wp.total)
    return fail(SPEC_ERR_WORKSPACE, "workspace of %zu bytes given, %zu needed", workspace_bytes, wp.total);
  const int bitmap_words = (max_len + 31) / 32 + 1;
  if ((int64_t)bitmap_words * 4 > 160 * 1024)
    return fail(SPEC_ERR_UNSUPPORTED, "sequences longer than %d tokens are not supported by specpc_token_select", 160 * 1024 * 8);
  rc = check_device();
  if (rc != SPEC_OK) return rc;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* tok = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + wp.token_off);
  const int64_t T = pr->total_tokens;
  if (T > 0) {
    token_reduce_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(scores, tok, T, pr->n_layers * pr->n_kv_heads,
                                                                     layer_head_reduce);
    SPEC_CUDA_OK(cudaGetLastError());
  }
  if (two_stage && T > 0) {
    // Algorithm 2 lines 8-9 as printed: average pool, then the keep kernel max-pools with width
    // n_neighbor before it selects, and widens nothing
    float* tok2 = tok + T;
    const dim3 grid((unsigned)((max_len + 255) / 256 > 0 ? (max_len + 255) / 256 : 1), (unsigned)pr->n_seq);
    token_avgpool_kernel<<<grid, 256, 0, st>>>(tok, tok2, pr->cu_seqlens, pr->n_in, pr->n_seq, n_forced_tail, pool_k);
    SPEC_CUDA_OK(cudaGetLastError());
    tok = tok2;
    pool = SPEC_POOL_MAX;
    pool_k = n_neighbor > 1 ? n_neighbor : 1;
    n_neighbor = 0;
  }
  KeepParams p;
  p.tok = tok; p.cu = pr->cu_seqlens; p.keep_out = keep_out; p.n_keep_out = n_keep_out;
  p.n_in = pr->n_in; p.pool = pool; p.pool_k = pool_k; p.c_max = c_max; p.n_neighbor = n_neighbor;
  p.n_forced = n_forced_tail; p.keep_capacity = keep_capacity; p.bitmap_words = bitmap_words;
  p.status = status_word;
  const int smem = select_smem_bytes(max_len, bitmap_words, &p.cap);
  SPEC_CUDA_OK(cudaFuncSetAttribute(specpc_keep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  specpc_keep_kernel<<<(unsigned)pr->n_seq, kSelThreads, smem, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}

// ------------------------------------------------- entry point without allocations ---
//
// Some callers cannot hand the library a workspace because they cannot allocate device
// memory at the point of the call: code running inside a serving engine whose allocator
// has already claimed (or is profiling) the whole device, or a plugin that is only given
// the tensors of the request.  For them the token-score vector of the SpecPC selection
// lives in a fixed array that is part of the library image.

namespace spec {

// The scratch of specpc_token_select_static: one fp32 token score per packed token.  Every
// device that loads the library holds these SPEC_STATIC_MAX_TOKENS * 4 bytes until the
// process exits.  In host code this name is only a handle for cudaGetSymbolAddress; it is
// not a device address and must never be passed to a kernel.
static __device__ __align__(256) float g_static_token_scores[SPEC_STATIC_MAX_TOKENS];

constexpr int kMaxDevices = 64;

// Device address of the array on the current device, looked up once per device.
static int static_scratch(float** out) {
  static float* cached[kMaxDevices] = {nullptr};
  int dev = 0;
  SPEC_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(SPEC_ERR_UNSUPPORTED, "device ordinal %d is not supported", dev);
  float* ptr = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
  if (!ptr) {
    const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_token_scores);
    if (e != cudaSuccess || !ptr)
      return fail(SPEC_ERR_CUDA, "cudaGetSymbolAddress(static token scratch): %s", cudaGetErrorString(e));
    __atomic_store_n(&cached[dev], ptr, __ATOMIC_RELEASE);
  }
  *out = ptr;
  return SPEC_OK;
}

}  // namespace spec

SPEC_EXPORT int32_t specpc_token_select_static(const spec_problem* pr, const float* scores, int32_t layer_head_reduce,
                                               int32_t pool, int32_t pool_k, int32_t c_max, int32_t n_neighbor,
                                               int32_t n_forced_tail, int32_t* keep_out, int32_t keep_capacity,
                                               int32_t* n_keep_out, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !keep_out || !n_keep_out) return fail(SPEC_ERR_BAD_ARG, "scores, keep_out and n_keep_out must not be NULL");
  if (layer_head_reduce != SPEC_REDUCE_SUM && layer_head_reduce != SPEC_REDUCE_MAX)
    return fail(SPEC_ERR_BAD_ARG, "layer_head_reduce=%d is not a spec_reduce value", layer_head_reduce);
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail);   // SPEC_POOL_AVG_THEN_MAX needs a second vector: not offered here
  if (rc != SPEC_OK) return rc;
  if (n_neighbor < 0) return fail(SPEC_ERR_BAD_ARG, "n_neighbor=%d is negative", n_neighbor);
  if (pr->total_tokens > SPEC_STATIC_MAX_TOKENS)
    return fail(SPEC_ERR_UNSUPPORTED, "total_tokens=%d exceeds the built-in scratch of %d tokens; use specpc_token_select with a workspace",
                pr->total_tokens, SPEC_STATIC_MAX_TOKENS);
  const int max_len = max_seq_len(pr);
  const int64_t worst = (int64_t)c_max * (2 * (int64_t)n_neighbor + 1) + n_forced_tail;
  const int64_t need_cap = worst < max_len ? worst : max_len;
  if (keep_capacity < need_cap)
    return fail(SPEC_ERR_BAD_ARG, "keep_capacity=%d is below the worst case %lld", keep_capacity, (long long)need_cap);
  const int bitmap_words = (max_len + 31) / 32 + 1;
  rc = check_device();
  if (rc != SPEC_OK) return rc;
  float* tok = nullptr;
  rc = static_scratch(&tok);                 // first call on a device: looks the array's address up
  if (rc != SPEC_OK) return rc;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t T = pr->total_tokens;
  if (T > 0) {
    // Writes every token score the selection reads, so nothing of an earlier call survives.
    token_reduce_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(scores, tok, T, pr->n_layers * pr->n_kv_heads,
                                                                     layer_head_reduce);
    SPEC_CUDA_OK(cudaGetLastError());
  }
  KeepParams p;
  p.tok = tok; p.cu = pr->cu_seqlens; p.keep_out = keep_out; p.n_keep_out = n_keep_out;
  p.n_in = pr->n_in; p.pool = pool; p.pool_k = pool_k; p.c_max = c_max; p.n_neighbor = n_neighbor;
  p.n_forced = n_forced_tail; p.keep_capacity = keep_capacity; p.bitmap_words = bitmap_words;
  p.status = status_word;
  const int smem = select_smem_bytes(max_len, bitmap_words, &p.cap);
  SPEC_CUDA_OK(cudaFuncSetAttribute(specpc_keep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  specpc_keep_kernel<<<(unsigned)pr->n_seq, kSelThreads, smem, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}
