// Device helpers shared by the selection kernels: order-preserving keys, block scans, histogram
// search, and the generic radix selection that recomputes pooled keys from global memory.
// Not part of the public interface.
#pragma once

#include "common.cuh"

namespace spec {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelVec = 4;                       // consecutive positions per thread in the ordered pass of the generic path
constexpr int kSmemLimit = 227 * 1024;

// Monotone map float -> uint32 (larger float <=> larger key), valid for any sign.
__device__ __forceinline__ uint32_t to_key(float v) {
  const uint32_t b = __float_as_uint(v + 0.0f);            // -0.0 + 0.0 = +0.0: the two zeros tie, as they compare equal
  return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);   // negative: all bits flipped; else: sign bit set
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Block-wide exclusive scan of one int per thread; total returned to every thread.
// wsum: kSelWarps ints of shared memory that no thread touches again before the CTA's next
// synchronisation after this call.  One __syncthreads.
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

// Finds the bin holding the need-th largest element of a histogram whose bins are spread
// over the threads, bins_per_thread consecutive bins each starting at my_bins (need >= 1).
// Returns the bin and the number of elements in higher bins to every thread; false (outputs
// untouched) when the histogram holds fewer than `need` elements.
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
__device__ inline void radix_select(const KeySource& key, int e, int need, const SelectScratch& sc,
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
__device__ inline int ordered_emit(const KeySource& key, int e, uint32_t T, int need_eq, const SelectScratch& sc, Emit emit) {
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

// Launches the streaming selection (select_stream.cu) for width-7 max pooling when the caller gave
// a workspace.  Returns SPEC_OK with *done = false when the problem is outside what that path serves.
SPEC_HIDDEN int run_stream_topk(const spec_problem* pr, const float* scores, int c_max, int n_forced_tail, int32_t* idx_out,
                                int32_t* count_out, int n_vert, int32_t* vert_out, int32_t* vert_count_out, void* workspace,
                                size_t workspace_bytes, int32_t* status_word, cudaStream_t st, bool* done);

}  // namespace spec
