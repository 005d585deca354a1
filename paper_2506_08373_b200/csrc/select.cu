// Pooling + exact top-C selection (Algorithm 1 lines 10, 11 and 13) and the SpecPC keep set
// (Algorithm 2 lines 7-10).
//
// A (sequence, layer, KV head) unit (SpecPC: a sequence) is owned by a thread-block cluster.
// Every CTA of the cluster copies its contiguous share of the unit's scores into shared memory
// with one bulk asynchronous copy (no registers are tied up while the bytes are in flight),
// pools them there and turns the pooled values into order-preserving 32-bit keys that stay
// resident.  The C-th largest key of the whole unit is then found by an MSB-first radix select
// (11 + 11 + 10 bits): every CTA counts its own keys in a shared-memory histogram, adds the
// non-empty bins into the merged histogram of every CTA of the cluster through distributed
// shared memory, and after one cluster barrier per pass every CTA locates the digit by itself.
// A first histogram over a 1-in-32 sample of the keys gives a floor under the threshold, so
// that the first full pass only counts the few keys at or above it (if the floor turns out
// too high the pass is repeated without it: the result is exact either way, and the cost does
// not depend on where in the unit the large scores sit).  Winners are written in ascending
// position: the CTAs exchange their counts, and each one emits its own winners behind those
// of the CTAs before it; ties at the threshold go to the lower position.  The scores are read
// from global memory once, whatever the number of budgets selected from them.
//
// Units too long for a cluster's shared memory take a generic path: one CTA per unit, keys
// recomputed from global memory in every radix pass.
#include "select_common.cuh"

#include <algorithm>

namespace spec {

// ------------------------------------------------------------- cluster primitives ----

__device__ __forceinline__ uint32_t shared_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
  cluster_arrive();
  cluster_wait();
}
// Address of this CTA's shared-memory location `saddr` in the CTA of the given rank.
__device__ __forceinline__ uint32_t in_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void remote_add(uint32_t caddr, uint32_t v) {
  asm volatile("red.relaxed.cluster.shared::cluster.add.u32 [%0], %1;" ::"r"(caddr), "r"(v) : "memory");
}
__device__ __forceinline__ void remote_or(uint32_t caddr, uint32_t v) {
  asm volatile("red.relaxed.cluster.shared::cluster.or.b32 [%0], %1;" ::"r"(caddr), "r"(v) : "memory");
}
__device__ __forceinline__ void remote_store(uint32_t caddr, int v) {
  asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(caddr), "r"(v) : "memory");
}

// ------------------------------------------------------------------ pooling ----------

// Pooling of any width from shared memory.  win[j .. j + k - 1] is the window of output j
// (positions outside the eligible range hold -infinity for MAX, 0 for AVG).  A thread owns a
// run of P consecutive outputs, P odd (lanes then hit distinct banks) and at most k, so that
// the P windows share a core, reduced once; the P - 1 values on either side of the core enter
// through a backward scan (parked in tmp[j], the run's own slots) and a forward scan.  Per
// output that is about (k + 3P) / P shared-memory accesses instead of k.  AVG adds in a fixed
// order without subtractions and divides by k.  win must be readable up to index
// n_out + k + 15, tmp up to n_out + 15.
constexpr int kPoolRun = 17;

template <bool AVG, class Store>
__device__ __forceinline__ void pool_runs(const float* win, float* tmp, int n_out, int k, Store store) {
  int P = (k & 1) ? k : k - 1;
  if (P > kPoolRun) P = kPoolRun;
  if (P < 1) P = 1;
  const int n_runs = (n_out + P - 1) / P;
  const float ident = AVG ? 0.f : -INFINITY;
  for (int r = threadIdx.x; r < n_runs; r += blockDim.x) {
    const int j0 = r * P;
    const float* a = win + j0;
    float core = ident;
    for (int t = P - 1; t < k; ++t) core = AVG ? core + a[t] : fmaxf(core, a[t]);
    float suf = ident;
    for (int u = P - 2; u >= 0; --u) {
      suf = AVG ? suf + a[u] : fmaxf(suf, a[u]);
      tmp[j0 + u] = suf;
    }
    float pre = ident;
    for (int u = 0; u < P; ++u) {
      const float left = u <= P - 2 ? tmp[j0 + u] : ident;
      const float o = AVG ? (left + core) + pre : fmax3(left, core, pre);
      if (j0 + u < n_out) store(j0 + u, AVG ? o / (float)k : o);
      if (u < P - 1) pre = AVG ? pre + a[k + u] : fmaxf(pre, a[k + u]);
    }
  }
}

// ---------------------------------------------------- cluster-resident selection -----

constexpr int kBins = 2048;                      // 11-bit digits (the last pass uses 1024 of them)
constexpr int kClMiscInts = 128;
constexpr int kClusterUse = 8;                   // largest cluster the host asks for

struct ClusterSelParams {
  const float* scores;        // [L, H, T]; keep set: the token scores [T] with L = H = 1
  const int32_t* cu;
  int64_t T;
  int n_in, L, H;
  int pool, pool_k, n_forced;
  int cap;                    // positions a CTA can hold (multiple of 4)
  int halo_l, halo_r;         // padding of the staged scores on either side (multiples of 4)
  int inplace;                // width-7 maximum, pooled in place
  int mode;                   // 0: top-C index lists, 1: keep set
  int c_max;
  int32_t* idx_out;
  int32_t* count_out;
  int n_vert;                 // second budget over the same pooled scores (0: none)
  int32_t* vert_out;
  int32_t* vert_count_out;
  int n_neighbor, keep_capacity;
  int32_t* keep_out;
  int32_t* n_keep_out;
  int32_t* status;
};

// Shared memory of a CTA: local histogram, two merged histograms, bookkeeping, (keep set) the
// bitmap of its positions, the staged scores with their halos and, unless pooling is in
// place, the keys.
__host__ __device__ inline int cluster_cap_pad(int cap) { return (cap + 127) & ~127; }
__host__ __device__ inline int cluster_bitmap_words(int cap, int mode) { return mode == 1 ? cluster_cap_pad(cap) / 32 + 4 : 0; }
__host__ __device__ inline size_t cluster_smem_bytes(int cap, int halo_l, int halo_r, int inplace, int mode) {
  const size_t raw = (size_t)halo_l + cluster_cap_pad(cap) + halo_r + 32;
  const size_t keys = inplace ? 0 : (size_t)cluster_cap_pad(cap) + 32;
  return (size_t)(3 * kBins + kClMiscInts + cluster_bitmap_words(cap, mode)) * 4 + (raw + keys) * 4;
}

struct ClusterCtx {
  uint32_t* local_hist;
  uint32_t* merged;           // [2][kBins]
  int* wsum;
  int* out2;
  int* r_a;                   // [16] per-rank counts, first kind
  int* r_b;                   // [16] per-rank counts, second kind
  const uint32_t* keys;
  int j_lo, j_hi;             // valid local positions
  uint32_t rank, cs;
  int stage;                  // merged-histogram uses so far
};

// Adds the non-empty bins of the local histogram into merged[stage & 1] of every CTA.
__device__ __forceinline__ void merge_hist(const ClusterCtx& c) {
  const uint32_t dst = shared_u32(c.merged + (c.stage & 1) * kBins);
  for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
    const uint32_t v = c.local_hist[b];
    if (v) {
      for (uint32_t r = 0; r < c.cs; ++r) remote_add(in_rank(dst + 4u * b, r), v);
    }
  }
}

// Clears the local histogram and the merged histogram of the NEXT stage (no CTA adds to it
// before the cluster barrier of the current stage).
__device__ __forceinline__ void clear_hists(const ClusterCtx& c) {
  uint32_t* next = c.merged + ((c.stage + 1) & 1) * kBins;
  for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
    c.local_hist[b] = 0;
    next[b] = 0;
  }
}

// Counts digit dg of the warp's keys that are `in`; neighbouring lanes with equal digits (the
// runs that pooling produces) are merged into one update.
__device__ __forceinline__ void hist_update(uint32_t* hist, bool in, uint32_t dg, int lane) {
  const uint32_t ins = __ballot_sync(0xffffffffu, in);
  if (ins == 0) return;                                    // warp-uniform
  if (__popc(ins) <= 4) {
    if (in) atomicAdd(&hist[dg], 1u);
    return;
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
  const uint32_t dg_prev = __shfl_up_sync(0xffffffffu, dg, 1);
  const bool head = in && (lane == 0 || !((ins >> (lane - 1)) & 1u) || dg_prev != dg);
  const uint32_t heads = __ballot_sync(0xffffffffu, head);
  if (head) {
    const uint32_t stop = (heads | ~ins) & ~(lt_mask | (1u << lane));   // next run, or a lane that is out
    atomicAdd(&hist[dg], (uint32_t)((stop ? __ffs(stop) - 1 : 32) - lane));
  }
}

// The key T of the take-th largest position of the unit (1 <= take < eligible positions) and
// how many positions with key == T belong to the selection.  floor_key: keys below it are
// known (or believed) to be out; a floor that was too high is detected and dropped.  Every
// thread of every CTA of the cluster calls this with the same arguments.
__device__ void cluster_threshold(ClusterCtx& c, int take, uint32_t floor_key, uint32_t& T_out, int& need_eq_out) {
  const int tid = threadIdx.x, lane = tid & 31;
  uint32_t prefix = 0, mask = 0;
  int remaining = take;
  int pass = 0;
  while (pass < 3) {
    const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
    const uint32_t dmask = pass == 2 ? 1023u : 2047u;
    clear_hists(c);
    __syncthreads();
    for (int jb = c.j_lo; jb < c.j_hi; jb += kSelThreads) {
      const int j = jb + tid;
      const bool valid = j < c.j_hi;
      const uint32_t kk = valid ? c.keys[j] : 0u;
      const bool in = valid && (pass == 0 ? kk >= floor_key : (kk & mask) == prefix);
      hist_update(c.local_hist, in, (kk >> shift) & dmask, lane);
    }
    __syncthreads();
    merge_hist(c);
    cluster_sync_all();
    const uint32_t* mg = c.merged + (c.stage & 1) * kBins;
    ++c.stage;
    int dg, ab;
    if (!locate_bin(mg + tid * (kBins / kSelThreads), kBins / kSelThreads, remaining, c.wsum, c.out2, dg, ab)) {
      floor_key = 0;                                       // fewer than `take` keys above the floor: count them all
      continue;
    }
    remaining -= ab;
    prefix |= (uint32_t)dg << shift;
    mask |= dmask << shift;
    ++pass;
  }
  T_out = prefix;
  need_eq_out = remaining;
}

// Per-CTA counts of keys above and equal to T, and the same per warp slab (a warp owns `slab`
// consecutive local positions).  Returns (gt, eq) of the CTA; w_gt / w_eq are this warp's
// exclusive prefixes within the CTA.
__device__ void count_winners(const ClusterCtx& c, uint32_t T, int slab, int& cta_gt, int& cta_eq, int& w_gt, int& w_eq,
                              int* sh_gt, int* sh_eq) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = max(warp * slab, c.j_lo), e = min((warp + 1) * slab, c.j_hi);
  int gt = 0, eq = 0;
  for (int jb = b; jb < e; jb += 32) {
    const int j = jb + lane;
    const uint32_t kk = j < e ? c.keys[j] : 0u;
    gt += __popc(__ballot_sync(0xffffffffu, j < e && kk > T));
    eq += __popc(__ballot_sync(0xffffffffu, j < e && kk == T));
  }
  __syncthreads();
  if (lane == 0) { sh_gt[warp] = gt; sh_eq[warp] = eq; }
  __syncthreads();
  cta_gt = cta_eq = w_gt = w_eq = 0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) {
    const int a = sh_gt[w], q = sh_eq[w];
    if (w < warp) { w_gt += a; w_eq += q; }
    cta_gt += a;
    cta_eq += q;
  }
}

// Publishes two counts of this CTA to every CTA of the cluster (slot = my rank); after the
// barrier returns the sums over the lower ranks and over all ranks.
__device__ void exchange_counts(const ClusterCtx& c, int a, int b, int& a_before, int& b_before, int& a_total, int& b_total) {
  if (threadIdx.x < c.cs) {
    remote_store(in_rank(shared_u32(c.r_a + c.rank), threadIdx.x), a);
    remote_store(in_rank(shared_u32(c.r_b + c.rank), threadIdx.x), b);
  }
  cluster_sync_all();
  a_before = b_before = a_total = b_total = 0;
  for (uint32_t r = 0; r < c.cs; ++r) {
    const int x = c.r_a[r], y = c.r_b[r];
    if (r < c.rank) { a_before += x; b_before += y; }
    a_total += x;
    b_total += y;
  }
}

__global__ void __launch_bounds__(kSelThreads, 2) cluster_select_kernel(const ClusterSelParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  ClusterCtx c;
  c.local_hist = reinterpret_cast<uint32_t*>(smem_raw);
  c.merged = c.local_hist + kBins;
  int* misc = reinterpret_cast<int*>(c.merged + 2 * kBins);
  c.wsum = misc;                                           // 32
  c.out2 = misc + 32;                                      // 4
  c.r_a = misc + 40;                                       // 16
  c.r_b = misc + 56;                                       // 16
  int* sh_gt = misc + 72;                                  // 16
  int* sh_eq = misc + 88;                                  // 16
  int* timed_out = misc + 104;
  uint64_t* mbar = reinterpret_cast<uint64_t*>(misc + 106);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(misc + kClMiscInts);
  const int cap_pad = cluster_cap_pad(p.cap);
  float* raw = reinterpret_cast<float*>(bitmap + cluster_bitmap_words(p.cap, p.mode));
  uint32_t* keys_w = p.inplace ? reinterpret_cast<uint32_t*>(raw + p.halo_l)
                               : reinterpret_cast<uint32_t*>(raw + p.halo_l + cap_pad + p.halo_r + 32);
  c.keys = keys_w;
  c.rank = cluster_rank();
  c.cs = cluster_size();
  c.stage = 0;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const int unit = blockIdx.x / c.cs;
  const int h = unit % p.H, l = (unit / p.H) % p.L, s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  int forced = min(p.n_forced, n);
  int e = n - forced;
  const float* src = p.scores + ((int64_t)l * p.H + h) * p.T + begin;
  const int mis = (int)((reinterpret_cast<uintptr_t>(src) >> 2) & 3u);
  // Positions are shifted by the misalignment of the unit's first score, x = position + mis, so
  // that every multiple of four in x is a 16-byte boundary of global memory.
  int X = e + mis;
  int CL = (((X + (int)c.cs - 1) / (int)c.cs) + 3) & ~3;   // positions per CTA
  if (CL > p.cap) {                                        // a sequence longer than the bound the host sized for
    if (tid == 0 && c.rank == 0) report(p.status, SPEC_ERR_BAD_ARG);
    e = 0; forced = 0; X = mis; CL = 0;                    // nothing is selected; the lists come out empty
  }
  const int x0 = (int)c.rank * CL;
  const int x1 = min(x0 + CL, X);
  c.j_lo = min(max(mis - x0, 0), max(x1 - x0, 0));
  c.j_hi = max(x1 - x0, 0);

  // budgets
  const int n_budgets = p.mode == 0 && p.n_vert > 0 ? 2 : 1;
  int take[2];
  take[0] = p.mode == 0 ? min(p.c_max - forced, e) : min(p.c_max, e);
  take[1] = min(p.n_vert, e);
  bool selects = false;
  for (int b = 0; b < n_budgets; ++b) selects = selects || (take[b] > 0 && take[b] < e);

  // ---- clear what other CTAs will add to, then let them know this CTA is up
  for (int b = tid; b < kBins; b += kSelThreads) c.merged[b] = 0;
  if (p.mode == 1)
    for (int w = tid; w < cluster_bitmap_words(p.cap, 1); w += kSelThreads) bitmap[w] = 0;
  if (tid == 0) {
    *timed_out = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(shared_u32(mbar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();

  if (selects) {
    // ---- stage my share of the scores: [x0 - halo_l, x0 + n_steps * 128 + halo_r) in x
    const int n_steps = (CL + 127) >> 7;
    const int xa = x0 - p.halo_l;
    const int total = p.halo_l + n_steps * 128 + p.halo_r;
    int bx0 = max(xa, mis ? 4 : 0), bx1 = min(xa + total, X & ~3);
    const bool bulk = bx1 > bx0;
    if (!bulk) bx0 = bx1 = xa + total;
    if (bulk && tid == 0) {
      const uint32_t bytes = (uint32_t)(bx1 - bx0) * 4u;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(shared_u32(mbar)), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(shared_u32(raw + (bx0 - xa))), "l"(src + (bx0 - mis)), "r"(bytes), "r"(shared_u32(mbar)) : "memory");
    }
    const float pad = p.pool == SPEC_POOL_MAX ? -INFINITY : 0.f;
    for (int i = tid; i < total; i += kSelThreads) {
      const int x = xa + i;
      if (x >= bx0 && x < bx1) { i += ((bx1 - x - 1) / kSelThreads) * kSelThreads; continue; }   // skip the bulk-copied part
      const int pp = x - mis;
      raw[i] = (pp >= 0 && pp < e) ? __ldg(src + pp) : pad;
    }
    if (bulk) {
      uint32_t ok = 0;
      for (uint32_t it = 0; it < (1u << 20) && !ok; ++it)
        asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\nselp.u32 %0, 1, 0, q;\n}"
                     : "=r"(ok) : "r"(shared_u32(mbar)) : "memory");
      if (!ok) *timed_out = 1;                             // the copy never landed: the result is reported as undefined
    }
    __syncthreads();

    // ---- pooled keys
    if (p.inplace) {
      // Width-7 maximum in place.  A warp owns consecutive 128-position steps; every lane holds
      // four scores of a step and takes the three on either side from its neighbours by
      // shuffle, lane 0 from the previous step (carried in registers), lane 31 from the next
      // step (not yet overwritten).  The values just outside a warp's steps are read before any
      // warp writes.
      float* base = raw + p.halo_l;
      const int spw = (n_steps + kSelWarps - 1) / kSelWarps;
      const int s0 = warp * spw, s1 = min(s0 + spw, n_steps);
      float carry[3] = {0.f, 0.f, 0.f}, rh[3] = {0.f, 0.f, 0.f};
      if (s0 < s1) {
#pragma unroll
        for (int q = 0; q < 3; ++q) { carry[q] = base[s0 * 128 - 3 + q]; rh[q] = base[s1 * 128 + q]; }
      }
      __syncthreads();
      for (int st = s0; st < s1; ++st) {
        float4* slot = reinterpret_cast<float4*>(base + st * 128) + lane;
        const float4 v = *slot;
        float4 nx = make_float4(rh[0], rh[1], rh[2], 0.f);
        if (lane == 31 && st + 1 < s1) nx = *reinterpret_cast<const float4*>(base + (st + 1) * 128);
        float x[10];
        x[0] = __shfl_up_sync(0xffffffffu, v.y, 1);
        x[1] = __shfl_up_sync(0xffffffffu, v.z, 1);
        x[2] = __shfl_up_sync(0xffffffffu, v.w, 1);
        x[7] = __shfl_down_sync(0xffffffffu, v.x, 1);
        x[8] = __shfl_down_sync(0xffffffffu, v.y, 1);
        x[9] = __shfl_down_sync(0xffffffffu, v.z, 1);
        if (lane == 0) { x[0] = carry[0]; x[1] = carry[1]; x[2] = carry[2]; }
        if (lane == 31) { x[7] = nx.x; x[8] = nx.y; x[9] = nx.z; }
        carry[0] = __shfl_sync(0xffffffffu, v.y, 31);
        carry[1] = __shfl_sync(0xffffffffu, v.z, 31);
        carry[2] = __shfl_sync(0xffffffffu, v.w, 31);
        x[3] = v.x; x[4] = v.y; x[5] = v.z; x[6] = v.w;
        float t3[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t3[i] = fmax3(x[i], x[i + 1], x[i + 2]);
        uint4 kq;
        kq.x = to_key(fmax3(t3[0], t3[3], x[6]));
        kq.y = to_key(fmax3(t3[1], t3[4], x[7]));
        kq.z = to_key(fmax3(t3[2], t3[5], x[8]));
        kq.w = to_key(fmax3(t3[3], t3[6], x[9]));
        *reinterpret_cast<uint4*>(slot) = kq;
        __syncwarp();
      }
    } else {
      const float* win = raw + p.halo_l - (p.pool_k >> 1);          // window of local position j starts at win[j]
      float* tmp = reinterpret_cast<float*>(keys_w);
      const int n_out = c.j_hi;
      auto store = [&](int j, float v) { keys_w[j] = to_key(v); };
      if (p.pool == SPEC_POOL_MAX) pool_runs<false>(win, tmp, n_out, p.pool_k, store);
      else pool_runs<true>(win, tmp, n_out, p.pool_k, store);
    }
    __syncthreads();
  }
  cluster_wait();                                          // every CTA of the cluster has cleared its shared memory

  // ---- a floor under the thresholds from a 1-in-32 sample of the keys
  uint32_t floor_key[2] = {0u, 0u};
  bool sample = false;
  for (int b = 0; b < n_budgets; ++b) sample = sample || (take[b] > 0 && take[b] < e && (int64_t)take[b] * 4 <= e && e >= 4096);
  if (sample) {
    clear_hists(c);
    __syncthreads();
    const int n_blocks = (CL + 31) >> 5;
    for (int b = tid; b < n_blocks; b += kSelThreads) {
      uint32_t hsh = ((uint32_t)unit * 0x9E3779B1u) ^ ((uint32_t)((x0 >> 5) + b) * 0x85EBCA6Bu);
      hsh ^= hsh >> 15; hsh *= 0x2C1B3C6Du; hsh ^= hsh >> 12;
      const int j = b * 32 + (int)(hsh & 31u);
      if (j >= c.j_lo && j < c.j_hi) atomicAdd(&c.local_hist[c.keys[j] >> 21], 1u);
    }
    __syncthreads();
    merge_hist(c);
    cluster_sync_all();
    const uint32_t* mg = c.merged + (c.stage & 1) * kBins;
    ++c.stage;
    for (int b = 0; b < n_budgets; ++b) {
      if (!(take[b] > 0 && take[b] < e && (int64_t)take[b] * 4 <= e)) continue;
      // About take/32 of the samples lie above the threshold; the floor is taken four standard
      // deviations further down the sample.
      const float m = (float)take[b] * (1.f / 32.f);
      const int rho = (int)(m + 4.f * sqrtf(m) + 8.f);
      int fb, ab;
      if (locate_bin(mg + tid * (kBins / kSelThreads), kBins / kSelThreads, rho, c.wsum, c.out2, fb, ab))
        floor_key[b] = (uint32_t)fb << 21;
    }
  }

  const int slab = ((CL + kSelThreads - 1) / kSelThreads) * 32;    // local positions per warp in the ordered sweeps

  if (p.mode == 0) {
    for (int b = 0; b < n_budgets; ++b) {
      int32_t* idx = (b == 0 ? p.idx_out + (int64_t)unit * p.c_max : p.vert_out + (int64_t)unit * p.n_vert);
      int32_t* cnt = b == 0 ? p.count_out : p.vert_count_out;
      const int width = b == 0 ? p.c_max : p.n_vert;
      const int tail = b == 0 ? forced : 0;
      const int tk = take[b];
      if (tk > 0 && tk < e) {
        uint32_t T;
        int need_eq;
        cluster_threshold(c, tk, floor_key[b], T, need_eq);
        int cta_gt, cta_eq, w_gt, w_eq;
        count_winners(c, T, slab, cta_gt, cta_eq, w_gt, w_eq, sh_gt, sh_eq);
        int gt_before, eq_before, gt_total, eq_total;
        exchange_counts(c, cta_gt, cta_eq, gt_before, eq_before, gt_total, eq_total);
        // ordered emission of my winners behind those of the lower ranks
        const int jb0 = max(warp * slab, c.j_lo), je = min((warp + 1) * slab, c.j_hi);
        int pre_gt = gt_before + w_gt, pre_eq = eq_before + w_eq;
        for (int jb = jb0; jb < je; jb += 32) {
          const int j = jb + lane;
          const uint32_t kk = j < je ? c.keys[j] : 0u;
          const bool is_gt = j < je && kk > T, is_eq = j < je && kk == T;
          const uint32_t bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
          const int my_gt = pre_gt + __popc(bg & lt_mask), my_eq = pre_eq + __popc(be & lt_mask);
          if (is_gt) idx[my_gt + min(my_eq, need_eq)] = x0 + j - mis;
          else if (is_eq && my_eq < need_eq) idx[my_gt + my_eq] = x0 + j - mis;
          pre_gt += __popc(bg);
          pre_eq += __popc(be);
        }
      } else if (tk > 0) {
        for (int j = c.j_lo + tid; j < c.j_hi; j += kSelThreads) idx[x0 + j - mis] = x0 + j - mis;   // every eligible position is kept
      }
      if (c.rank == 0) {
        const int tk0 = max(tk, 0);
        for (int q = tk0 + tid; q < width; q += kSelThreads) idx[q] = (q - tk0 < tail) ? e + (q - tk0) : -1;
        if (cnt && tid == 0) cnt[unit] = tk0 + tail;
      }
    }
  } else {
    // ---- keep set: winners and their neighbourhoods into the distributed bitmap
    const int tk = take[0];
    const int nb = p.n_neighbor;
    auto mark = [&](int xlo, int xhi) {                    // x range, inclusive, inside [mis, X)
      for (int r = xlo / CL; r <= xhi / CL; ++r) {
        const int a = max(xlo, r * CL) - r * CL, z = min(xhi, r * CL + CL - 1) - r * CL;
        for (int w = a >> 5; w <= (z >> 5); ++w) {
          const int b0 = max(a, w << 5) & 31, b1 = min(z, (w << 5) + 31) & 31;
          remote_or(in_rank(shared_u32(bitmap + w), (uint32_t)r), (0xffffffffu >> (31 - b1)) & (0xffffffffu << b0));
        }
      }
    };
    if (tk > 0 && tk < e) {
      uint32_t T;
      int need_eq;
      cluster_threshold(c, tk, floor_key[0], T, need_eq);
      int cta_gt, cta_eq, w_gt, w_eq;
      count_winners(c, T, slab, cta_gt, cta_eq, w_gt, w_eq, sh_gt, sh_eq);
      int gt_before, eq_before, gt_total, eq_total;
      exchange_counts(c, cta_gt, cta_eq, gt_before, eq_before, gt_total, eq_total);
      const int jb0 = max(warp * slab, c.j_lo), je = min((warp + 1) * slab, c.j_hi);
      int pre_eq = eq_before + w_eq;
      for (int jb = jb0; jb < je; jb += 32) {
        const int j = jb + lane;
        const uint32_t kk = j < je ? c.keys[j] : 0u;
        const bool is_eq = j < je && kk == T;
        const uint32_t be = __ballot_sync(0xffffffffu, is_eq);
        const bool win = j < je && (kk > T || (is_eq && pre_eq + __popc(be & lt_mask) < need_eq));
        if (win) mark(max(x0 + j - nb, mis), min(x0 + j + nb, X - 1));
        pre_eq += __popc(be);
      }
    } else if (tk > 0) {
      for (int w = tid; w * 32 < c.j_hi; w += kSelThreads) {
        const int a = max(w << 5, c.j_lo), z = min((w << 5) + 31, c.j_hi - 1);
        if (a <= z) atomicOr(&bitmap[w], (0xffffffffu >> (31 - (z & 31))) & (0xffffffffu << (a & 31)));
      }
    }
    cluster_sync_all();                                    // all marks have landed
    // ---- ordered extraction: every thread owns a run of consecutive bitmap words
    const int n_words = (CL + 31) >> 5;
    const int wpt = (n_words + kSelThreads - 1) / kSelThreads;
    const int w0 = tid * wpt, w1 = min(w0 + wpt, n_words);
    int mine = 0;
    for (int w = w0; w < w1; ++w) mine += __popc(bitmap[w]);
    int cta_total;
    const int before = block_exclusive_scan(mine, c.wsum, cta_total);
    int tot_before, dummy_b, total, dummy_t;
    exchange_counts(c, cta_total, 0, tot_before, dummy_b, total, dummy_t);
    int32_t* keep = p.keep_out + (int64_t)s * p.keep_capacity;
    int pos = tot_before + before;
    for (int w = w0; w < w1; ++w) {
      uint32_t bits = bitmap[w];
      while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        if (pos < p.keep_capacity) keep[pos] = x0 + (w << 5) + b - mis;
        ++pos;
      }
    }
    if (c.rank == 0) {
      // the forced tail (the always-kept window) follows the selected positions
      for (int q = tid; q < forced; q += kSelThreads)
        if (total + q < p.keep_capacity) keep[total + q] = e + q;
      const int kept = min(total + forced, p.keep_capacity);
      for (int q = kept + tid; q < p.keep_capacity; q += kSelThreads) keep[q] = -1;
      if (tid == 0) {
        if (total + forced > p.keep_capacity) report(p.status, SPEC_ERR_BAD_ARG);
        p.n_keep_out[s] = kept;
      }
    }
  }
  if (*timed_out && tid == 0) report(p.status, SPEC_ERR_TIMEOUT);
  // No CTA leaves while another may still write to its shared memory.
  cluster_sync_all();
}

// ------------------------------------------------------------- generic selection -----
//
// One CTA per unit, any length: pooled keys are recomputed from global memory in each of the
// four 8-bit radix passes and in the ordered emission.  Only units that do not fit a cluster's
// shared memory come here.

struct TopkParams {
  const float* scores;
  const int32_t* cu;
  int32_t* idx_out;
  int32_t* count_out;
  int64_t T;
  int n_in, L, H, pool, pool_k, c_max, n_forced;
  int no_tail;                // the budget is taken over the eligible range only and the forced tail is not appended
};

__global__ void __launch_bounds__(kSelThreads) pool_topk_generic_kernel(TopkParams p) {
  __shared__ uint32_t hist[kSelWarps * 256];
  __shared__ int misc[2 * kSelWarps + 8];
  const int unit = blockIdx.x;
  const int h = unit % p.H, l = (unit / p.H) % p.L, s = unit / (p.H * p.L);
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int forced = min(p.n_forced, n);
  const int e = n - forced;
  const int tail = p.no_tail ? 0 : forced;
  const int take = max(min(p.c_max - tail, e), 0);
  int32_t* idx = p.idx_out + (int64_t)unit * p.c_max;
  const int tid = threadIdx.x;
  const float* src = p.scores + ((int64_t)l * p.H + h) * p.T + begin;
  if (take > 0 && take < e) {
    SelectScratch sc;
    sc.hist = hist;
    sc.misc = misc;
    KeySource key;
    key.scores = src;
    key.e = e; key.pool = p.pool; key.k = p.pool_k;
    key.keys = nullptr;
    uint32_t T;
    int need_eq;
    radix_select(key, e, take, sc, T, need_eq);
    ordered_emit(key, e, T, need_eq, sc, [&](int rank, int j) { idx[rank] = j; });
  } else {
    for (int q = tid; q < take; q += kSelThreads) idx[q] = q;      // every eligible position is kept
  }
  for (int q = take + tid; q < p.c_max; q += kSelThreads) idx[q] = (q - take < tail) ? e + (q - take) : -1;
  if (p.count_out && tid == 0) p.count_out[unit] = take + tail;
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
// scores over each sequence's eligible range, written to a second vector.  A CTA stages a tile
// of kAvgTile outputs with its window margins in shared memory and pools it there.
constexpr int kAvgTile = 4096;
constexpr int kAvgThreads = 256;

__global__ void __launch_bounds__(kAvgThreads) token_avgpool_kernel(const float* __restrict__ tok, float* __restrict__ out,
                                                                    const int32_t* __restrict__ cu, int n_in, int n_forced, int k) {
  __shared__ float win[kAvgTile + 256 + 32];
  __shared__ float tmp[kAvgTile + 32];
  const int s = blockIdx.y;
  int begin, n;
  seq_range(cu, n_in, s, begin, n);
  const int e = n - min(n_forced, n);
  const int lo = k >> 1;
  for (int t0 = blockIdx.x * kAvgTile; t0 < e; t0 += gridDim.x * kAvgTile) {
    const int n_out = min(kAvgTile, e - t0);
    __syncthreads();
    for (int i = threadIdx.x; i < n_out + k + 16; i += kAvgThreads) {
      const int j = t0 - lo + i;
      win[i] = (j >= 0 && j < e) ? __ldg(tok + begin + j) : 0.f;
    }
    __syncthreads();
    float* dst = out + begin + t0;
    pool_runs<true>(win, tmp, n_out, k, [&](int j, float v) { dst[j] = v; });
  }
}

struct KeepParams {
  const float* tok;
  const int32_t* cu;
  int32_t* keep_out;
  int32_t* n_keep_out;
  int n_in, pool, pool_k, c_max, n_neighbor, n_forced, keep_capacity, bitmap_words;
  int32_t* status;
};

// Keep set of a sequence too long for a cluster: one CTA, keys recomputed from global memory
// in every radix pass, the bitmap of the whole sequence in its shared memory.
__global__ void __launch_bounds__(kSelThreads) specpc_keep_generic_kernel(KeepParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  SelectScratch sc;
  sc.hist = reinterpret_cast<uint32_t*>(smem_raw);
  sc.misc = reinterpret_cast<int*>(sc.hist + kSelWarps * 256);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(sc.misc + 2 * kSelWarps + 8);

  const int s = blockIdx.x;
  int begin, n;
  seq_range(p.cu, p.n_in, s, begin, n);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int32_t* keep = p.keep_out + (int64_t)s * p.keep_capacity;
  if (((n + 31) >> 5) > p.bitmap_words) {                  // a sequence longer than the bound the host sized for
    if (tid == 0) {
      report(p.status, SPEC_ERR_BAD_ARG);
      p.n_keep_out[s] = 0;
    }
    for (int q = tid; q < p.keep_capacity; q += kSelThreads) keep[q] = -1;
    return;
  }
  const int forced = min(p.n_forced, n);
  const int e = n - forced;
  const int take = min(p.c_max, e);
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
    const int nb = p.n_neighbor;
    uint32_t T;
    int need_eq;
    radix_select(key, e, take, sc, T, need_eq);
    ordered_emit(key, e, T, need_eq, sc, [&](int, int j) { mark(max(j - nb, 0), min(j + nb, e - 1)); });
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
  for (int q = kept + tid; q < p.keep_capacity; q += kSelThreads) keep[q] = -1;
  if (tid == 0) p.n_keep_out[s] = kept;
}

// ------------------------------------------------------------------ host side ---------

constexpr int kChunkTarget = 8192;               // positions per CTA the cluster size is chosen for
constexpr int kMaxDevices = 64;

struct ClusterPlan {
  bool fits;
  int cs, cap, halo_l, halo_r, inplace;
  size_t smem;
};

static ClusterPlan plan_cluster(int max_len, int pool, int pool_k, int mode, int max_cs) {
  ClusterPlan pl;
  pl.inplace = pool == SPEC_POOL_MAX && pool_k == 7;
  if (pl.inplace) {
    pl.halo_l = pl.halo_r = 4;
  } else {
    pl.halo_l = ((pool_k >> 1) + 3) & ~3;
    pl.halo_r = ((pool_k - 1 - (pool_k >> 1)) + kPoolRun + 3) & ~3;
  }
  const int64_t x_max = (int64_t)max_len + 3;
  int cs = 1;
  while (cs < max_cs && (x_max + cs - 1) / cs > kChunkTarget) cs <<= 1;
  pl.cs = cs;
  pl.cap = (int)((((x_max + cs - 1) / cs) + 3) & ~(int64_t)3);
  pl.smem = cluster_smem_bytes(pl.cap, pl.halo_l, pl.halo_r, pl.inplace, mode);
  pl.fits = pl.smem <= (size_t)kSmemLimit;
  return pl;
}

// One-time function attributes of the cluster kernel on the current device.
static int prepare_cluster_kernel(int* max_cs_out) {
  static int state[kMaxDevices] = {0};                     // 0: not set, 8 / 16: largest cluster size usable
  int dev = 0;
  SPEC_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(SPEC_ERR_UNSUPPORTED, "device ordinal %d is not supported", dev);
  int st = __atomic_load_n(&state[dev], __ATOMIC_ACQUIRE);
  if (!st) {
    SPEC_CUDA_OK(cudaFuncSetAttribute(cluster_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
    st = 8;
    if (kClusterUse > 8) {
      if (cudaFuncSetAttribute(cluster_select_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) st = kClusterUse;
      else cudaGetLastError();
    }
    __atomic_store_n(&state[dev], st, __ATOMIC_RELEASE);
  }
  *max_cs_out = st;
  return SPEC_OK;
}

static int launch_cluster(const ClusterSelParams& p, int64_t n_units, const ClusterPlan& pl, cudaStream_t st) {
  if (n_units * pl.cs > 0x7fffffffLL) return fail(SPEC_ERR_UNSUPPORTED, "too many units for one launch");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_units * pl.cs));
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)pl.cs;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  SPEC_CUDA_OK(cudaLaunchKernelEx(&cfg, cluster_select_kernel, p));
  return SPEC_OK;
}

// two_stage: 0 = SPEC_POOL_AVG_THEN_MAX is not a value of this call, 1 = accepted, 2 = known but not offered.
static int check_pool_args(int pool, int pool_k, int c_max, int n_forced_tail, int two_stage = 0) {
  if (pool == SPEC_POOL_AVG_THEN_MAX && two_stage == 2)
    return fail(SPEC_ERR_UNSUPPORTED, "SPEC_POOL_AVG_THEN_MAX is not offered by this entry point (it needs a second scratch vector); "
                                      "use specpc_token_select with a workspace");
  if (pool != SPEC_POOL_MAX && pool != SPEC_POOL_AVG && !(two_stage == 1 && pool == SPEC_POOL_AVG_THEN_MAX))
    return fail(SPEC_ERR_BAD_ARG, "pool=%d is not a spec_pool value this call accepts", pool);
  if (pool_k < 1 || pool_k > 255) return fail(SPEC_ERR_BAD_ARG, "pool_k=%d outside [1, 255]", pool_k);
  if (c_max < 1) return fail(SPEC_ERR_BAD_ARG, "c_max=%d must be >= 1", c_max);
  if (n_forced_tail < 0) return fail(SPEC_ERR_BAD_ARG, "n_forced_tail=%d is negative", n_forced_tail);
  return SPEC_OK;
}

// Top-C lists (and optionally the vertical lists) of every unit.
static int run_pool_topk(const spec_problem* pr, const float* scores, int pool, int pool_k, int c_max, int n_forced_tail,
                         int32_t* idx_out, int32_t* count_out, int n_vert, int32_t* vert_out, int32_t* vert_count_out,
                         void* workspace, size_t workspace_bytes, int32_t* status_word, cudaStream_t st) {
  // The default pooling with a budget that is a modest share of the sequence streams through the
  // workspace; everything else (and every call without a workspace) stays resident in a cluster.
  if (pool == SPEC_POOL_MAX && pool_k == 7 && (int64_t)std::max(c_max, n_vert) * 6 <= max_seq_len(pr)) {
    bool done = false;
    const int rc = run_stream_topk(pr, scores, c_max, n_forced_tail, idx_out, count_out, n_vert, vert_out, vert_count_out,
                                   workspace, workspace_bytes, status_word, st, &done);
    if (rc != SPEC_OK || done) return rc;
  }
  int max_cs = 8;
  int rc = prepare_cluster_kernel(&max_cs);
  if (rc != SPEC_OK) return rc;
  const int64_t n_units = (int64_t)pr->n_seq * pr->n_layers * pr->n_kv_heads;
  const ClusterPlan pl = plan_cluster(max_seq_len(pr), pool, pool_k, 0, max_cs);
  if (pl.fits) {
    ClusterSelParams p = {};
    p.scores = scores; p.cu = pr->cu_seqlens; p.T = pr->total_tokens; p.n_in = pr->n_in;
    p.L = pr->n_layers; p.H = pr->n_kv_heads; p.pool = pool; p.pool_k = pool_k; p.n_forced = n_forced_tail;
    p.cap = pl.cap; p.halo_l = pl.halo_l; p.halo_r = pl.halo_r; p.inplace = pl.inplace; p.mode = 0;
    p.c_max = c_max; p.idx_out = idx_out; p.count_out = count_out;
    p.n_vert = n_vert; p.vert_out = vert_out; p.vert_count_out = vert_count_out;
    p.status = status_word;
    return launch_cluster(p, n_units, pl, st);
  }
  TopkParams p;
  p.scores = scores; p.cu = pr->cu_seqlens; p.idx_out = idx_out; p.count_out = count_out;
  p.T = pr->total_tokens; p.n_in = pr->n_in; p.L = pr->n_layers; p.H = pr->n_kv_heads;
  p.pool = pool; p.pool_k = pool_k; p.c_max = c_max; p.n_forced = n_forced_tail;
  p.no_tail = 0;
  pool_topk_generic_kernel<<<(unsigned)n_units, kSelThreads, 0, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  if (n_vert > 0) {                                        // a second sweep: this path keeps nothing resident
    p.idx_out = vert_out; p.count_out = vert_count_out; p.c_max = n_vert;
    p.no_tail = 1;
    pool_topk_generic_kernel<<<(unsigned)n_units, kSelThreads, 0, st>>>(p);
    SPEC_CUDA_OK(cudaGetLastError());
  }
  return SPEC_OK;
}

// Keep lists from token scores `tok` (already reduced over layers and heads).
static int run_keep(const spec_problem* pr, const float* tok, int pool, int pool_k, int c_max, int n_neighbor,
                    int n_forced_tail, int32_t* keep_out, int keep_capacity, int32_t* n_keep_out, int32_t* status_word,
                    cudaStream_t st) {
  int max_cs = 8;
  int rc = prepare_cluster_kernel(&max_cs);
  if (rc != SPEC_OK) return rc;
  const int max_len = max_seq_len(pr);
  const ClusterPlan pl = plan_cluster(max_len, pool, pool_k, 1, max_cs);
  if (pl.fits) {
    ClusterSelParams p = {};
    p.scores = tok; p.cu = pr->cu_seqlens; p.T = pr->total_tokens; p.n_in = pr->n_in;
    p.L = 1; p.H = 1; p.pool = pool; p.pool_k = pool_k; p.n_forced = n_forced_tail;
    p.cap = pl.cap; p.halo_l = pl.halo_l; p.halo_r = pl.halo_r; p.inplace = pl.inplace; p.mode = 1;
    p.c_max = c_max; p.n_neighbor = n_neighbor; p.keep_capacity = keep_capacity;
    p.keep_out = keep_out; p.n_keep_out = n_keep_out; p.status = status_word;
    return launch_cluster(p, pr->n_seq, pl, st);
  }
  const int bitmap_words = (max_len + 31) / 32 + 1;
  const int smem = kSelWarps * 256 * 4 + (2 * kSelWarps + 8) * 4 + bitmap_words * 4;
  if (smem > kSmemLimit)
    return fail(SPEC_ERR_UNSUPPORTED, "sequences longer than %d tokens are not supported by specpc_token_select", (kSmemLimit - 20000) * 8);
  static int set[kMaxDevices] = {0};
  int dev = 0;
  SPEC_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 0 && dev < kMaxDevices && !__atomic_load_n(&set[dev], __ATOMIC_ACQUIRE)) {
    SPEC_CUDA_OK(cudaFuncSetAttribute(specpc_keep_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
    __atomic_store_n(&set[dev], 1, __ATOMIC_RELEASE);
  }
  KeepParams p;
  p.tok = tok; p.cu = pr->cu_seqlens; p.keep_out = keep_out; p.n_keep_out = n_keep_out;
  p.n_in = pr->n_in; p.pool = pool; p.pool_k = pool_k; p.c_max = c_max; p.n_neighbor = n_neighbor;
  p.n_forced = n_forced_tail; p.keep_capacity = keep_capacity; p.bitmap_words = bitmap_words;
  p.status = status_word;
  specpc_keep_generic_kernel<<<(unsigned)pr->n_seq, kSelThreads, smem, st>>>(p);
  SPEC_CUDA_OK(cudaGetLastError());
  return SPEC_OK;
}

}  // namespace spec

SPEC_EXPORT int32_t spec_pool_topk(const spec_problem* pr, const float* scores, int32_t pool, int32_t pool_k,
                                   int32_t c_max, int32_t n_forced_tail, int32_t* idx_out, int32_t* count_out,
                                   void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !idx_out) return fail(SPEC_ERR_BAD_ARG, "scores and idx_out must not be NULL");
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail);
  if (rc != SPEC_OK) return rc;
  if (n_forced_tail > c_max) return fail(SPEC_ERR_BAD_ARG, "n_forced_tail=%d exceeds c_max=%d", n_forced_tail, c_max);
  rc = check_device();
  if (rc != SPEC_OK) return rc;
  return run_pool_topk(pr, scores, pool, pool_k, c_max, n_forced_tail, idx_out, count_out, 0, nullptr, nullptr, workspace,
                       workspace_bytes, status_word, static_cast<cudaStream_t>(stream));
}

SPEC_EXPORT int32_t spec_pool_topk_vert(const spec_problem* pr, const float* scores, int32_t pool, int32_t pool_k,
                                        int32_t c_max, int32_t n_forced_tail, int32_t* idx_out, int32_t* count_out,
                                        int32_t n_vert, int32_t* vert_idx_out, int32_t* vert_count_out,
                                        void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !idx_out || !vert_idx_out) return fail(SPEC_ERR_BAD_ARG, "scores, idx_out and vert_idx_out must not be NULL");
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail);
  if (rc != SPEC_OK) return rc;
  if (n_forced_tail > c_max) return fail(SPEC_ERR_BAD_ARG, "n_forced_tail=%d exceeds c_max=%d", n_forced_tail, c_max);
  if (n_vert < 1) return fail(SPEC_ERR_BAD_ARG, "n_vert=%d must be >= 1", n_vert);
  rc = check_device();
  if (rc != SPEC_OK) return rc;
  return run_pool_topk(pr, scores, pool, pool_k, c_max, n_forced_tail, idx_out, count_out, n_vert, vert_idx_out,
                       vert_count_out, workspace, workspace_bytes, status_word, static_cast<cudaStream_t>(stream));
}

namespace spec {

// Argument checks shared by the two keep-set entry points; max_len and the pooling actually
// run by the keep kernel come back through the references.
static int check_keep_args(const spec_problem* pr, const float* scores, int layer_head_reduce, int pool, int pool_k, int c_max,
                           int n_neighbor, int n_forced_tail, const int32_t* keep_out, int keep_capacity,
                           const int32_t* n_keep_out, int two_stage_ok) {
  int rc = check_problem(pr);
  if (rc != SPEC_OK) return rc;
  if (!scores || !keep_out || !n_keep_out) return fail(SPEC_ERR_BAD_ARG, "scores, keep_out and n_keep_out must not be NULL");
  if (layer_head_reduce != SPEC_REDUCE_SUM && layer_head_reduce != SPEC_REDUCE_MAX)
    return fail(SPEC_ERR_BAD_ARG, "layer_head_reduce=%d is not a spec_reduce value", layer_head_reduce);
  rc = check_pool_args(pool, pool_k, c_max, n_forced_tail, two_stage_ok);
  if (rc != SPEC_OK) return rc;
  if (n_neighbor < 0) return fail(SPEC_ERR_BAD_ARG, "n_neighbor=%d is negative", n_neighbor);
  const bool two_stage = pool == SPEC_POOL_AVG_THEN_MAX;
  if (two_stage && n_neighbor > 255) return fail(SPEC_ERR_BAD_ARG, "n_neighbor=%d as a pooling width exceeds 255", n_neighbor);
  const int max_len = max_seq_len(pr);
  const int64_t worst = two_stage ? (int64_t)c_max + n_forced_tail : (int64_t)c_max * (2 * (int64_t)n_neighbor + 1) + n_forced_tail;
  const int64_t need_cap = worst < max_len ? worst : max_len;
  if (keep_capacity < need_cap)
    return fail(SPEC_ERR_BAD_ARG, "keep_capacity=%d is below the worst case %lld", keep_capacity, (long long)need_cap);
  return SPEC_OK;
}

}  // namespace spec

SPEC_EXPORT int32_t specpc_token_select(const spec_problem* pr, const float* scores, int32_t layer_head_reduce,
                                        int32_t pool, int32_t pool_k, int32_t c_max, int32_t n_neighbor,
                                        int32_t n_forced_tail, int32_t* keep_out, int32_t keep_capacity,
                                        int32_t* n_keep_out, void* workspace, size_t workspace_bytes,
                                        int32_t* status_word, void* stream) {
  using namespace spec;
  int rc = check_keep_args(pr, scores, layer_head_reduce, pool, pool_k, c_max, n_neighbor, n_forced_tail, keep_out,
                           keep_capacity, n_keep_out, 1);
  if (rc != SPEC_OK) return rc;
  const WorkspacePlan wp = plan_workspace(pr);
  if (!workspace || workspace_bytes < wp.total)
    return fail(SPEC_ERR_WORKSPACE, "workspace of %zu bytes given, %zu needed", workspace_bytes, wp.total);
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
  if (pool == SPEC_POOL_AVG_THEN_MAX && T > 0) {
    // Algorithm 2 lines 8-9 as printed: average pool, then the keep kernel max-pools with width
    // n_neighbor before it selects, and widens nothing
    float* tok2 = tok + T;
    const int max_len = max_seq_len(pr);
    const int tiles = (max_len + kAvgTile - 1) / kAvgTile;
    const dim3 grid((unsigned)(tiles > 0 ? tiles : 1), (unsigned)pr->n_seq);
    token_avgpool_kernel<<<grid, kAvgThreads, 0, st>>>(tok, tok2, pr->cu_seqlens, pr->n_in, n_forced_tail, pool_k);
    SPEC_CUDA_OK(cudaGetLastError());
    tok = tok2;
    pool = SPEC_POOL_MAX;
    pool_k = n_neighbor > 1 ? n_neighbor : 1;
    n_neighbor = 0;
  }
  return run_keep(pr, tok, pool, pool_k, c_max, n_neighbor, n_forced_tail, keep_out, keep_capacity, n_keep_out, status_word, st);
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
  // SPEC_POOL_AVG_THEN_MAX needs a second vector: not offered here
  int rc = check_keep_args(pr, scores, layer_head_reduce, pool, pool_k, c_max, n_neighbor, n_forced_tail, keep_out,
                           keep_capacity, n_keep_out, 2);
  if (rc != SPEC_OK) return rc;
  if (pr->total_tokens > SPEC_STATIC_MAX_TOKENS)
    return fail(SPEC_ERR_UNSUPPORTED, "total_tokens=%d exceeds the built-in scratch of %d tokens; use specpc_token_select with a workspace",
                pr->total_tokens, SPEC_STATIC_MAX_TOKENS);
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
  return run_keep(pr, tok, pool, pool_k, c_max, n_neighbor, n_forced_tail, keep_out, keep_capacity, n_keep_out, status_word, st);
}
