// Selection steps of the compressor, one thread block per unit:
//   top-t of C (Eq. 14) and the semantic vector v' = sum_{j in I} C[j] V[j,:] (Eq. 15);
//   the k middle activations: top-k of the average-pooled scores over the
//   intermediate positions [s1, N - s2) (Sec. IV-B, pooling of Sec. V-D), written
//   with the sinks and the recent window as the unit's ascending index list.
// Both selections find the exact k-th largest order-preserving 32-bit key by bisection
// over the key bits, followed by an ordered compaction; of equal scores the lower
// position wins.  Up to 32768 positions the keys live in the registers of one block
// (select_fast_kernel), up to 262144 in those of a thread-block cluster
// (select_cluster_kernel); longer units, or other pooling kernels, stream them from L2
// once per bisection step until few enough survive to be collected in shared memory
// (select_kernel).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace taskkv {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ uint32_t ordered_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k) {   // inverse of ordered_key
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

struct ScoreKey {          // key of C[j]
  const float* C;
  __device__ __forceinline__ uint32_t operator()(int j) const { return ordered_key(C[j]); }
};

struct SelectSmem {
  int cnt[2][kWarps];
  int cnt3[2][3][kWarps];
  uint32_t mn[kWarps], mx[kWarps];
  long long scan[kWarps];
  int list_n;
  uint32_t list_thr;
};

// #(key(j) >= cand), j in [lo, hi), over the whole block: one coalesced pass over the keys.
template <class KeyFn>
__device__ int stream_count_ge(int lo, int hi, const KeyFn& key, uint32_t cand, int* slot) {
  int c = 0;
#pragma unroll 8    // several loads in flight per thread: the pass is bound by L2 latency otherwise
  for (int j = lo + (int)threadIdx.x; j < hi; j += kThreads) c += key(j) >= cand;
  c = __reduce_add_sync(0xffffffffu, c);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) slot[warp] = c;
  __syncthreads();
  return __reduce_add_sync(0xffffffffu, slot[lane]);
}

// Finds the key `thr` of the `want`-th largest element of key(j), j in [lo, hi)
// (1 <= want <= hi - lo), and how many elements equal to thr belong to the top
// `want` (need_eq); elements with key > thr number want - need_eq.
// Bisection over the key bits, one pass over the keys per step, which also tells how many keys still lie in
// the undecided range [t, t + 2^(bit+1)); once they fit into `list` (shared memory, `cap` entries) they are
// collected there and one warp settles the remaining bits.
template <class KeyFn>
__device__ void block_stream_select(SelectSmem& sm, int lo, int hi, int want, const KeyFn& key, uint32_t* list,
                                    int cap, uint32_t& thr, int& need_eq) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll 8
  for (int j = lo + tid; j < hi; j += kThreads) {
    const uint32_t kx = key(j);
    kmin = min(kmin, kx);
    kmax = max(kmax, kx);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { sm.mn[warp] = kmin; sm.mx[warp] = kmax; }
  if (tid == 0) sm.list_n = 0;
  __syncthreads();
  kmin = __reduce_min_sync(0xffffffffu, sm.mn[lane]);
  kmax = __reduce_max_sync(0xffffffffu, sm.mx[lane]);
  // bits above the highest bit in which the keys differ are common to the answer
  const uint32_t diff = kmin ^ kmax;
  int bit = diff ? 31 - __clz(diff) : -1;
  uint32_t t = diff ? (kmax & ~((2u << bit) - 1u)) : kmax;
  int par = 0;
  int above = 0;             // keys >= t + 2^(bit+1): the last count that fell short of `want`
  int at_least = hi - lo;    // keys >= t: all of them at the start, then the last count that reached `want`
  // two bits per pass over the keys (the pass is bound by the L2 stream, three compares per key are free)
  for (; bit >= 1 && at_least - above > cap; bit -= 2) {
    const uint32_t c10 = t | (2u << (bit - 1)), c11 = t | (3u << (bit - 1)), c01 = t | (1u << (bit - 1));
    int n10 = 0, n11 = 0, n01 = 0;
#pragma unroll 8
    for (int j = lo + tid; j < hi; j += kThreads) {
      const uint32_t kx = key(j);
      n10 += kx >= c10;
      n11 += kx >= c11;
      n01 += kx >= c01;
    }
    n10 = __reduce_add_sync(0xffffffffu, n10);
    n11 = __reduce_add_sync(0xffffffffu, n11);
    n01 = __reduce_add_sync(0xffffffffu, n01);
    if (lane == 0) { sm.cnt3[par][0][warp] = n10; sm.cnt3[par][1][warp] = n11; sm.cnt3[par][2][warp] = n01; }
    __syncthreads();
    n10 = __reduce_add_sync(0xffffffffu, sm.cnt3[par][0][lane]);
    n11 = __reduce_add_sync(0xffffffffu, sm.cnt3[par][1][lane]);
    n01 = __reduce_add_sync(0xffffffffu, sm.cnt3[par][2][lane]);
    par ^= 1;
    if (n10 >= want) {
      if (n11 >= want) { t = c11; at_least = n11; } else { t = c10; at_least = n10; above = n11; }
    } else {
      if (n01 >= want) { t = c01; at_least = n01; above = n10; } else above = n01;
    }
  }
  for (; bit >= 0 && at_least - above > cap; --bit) {   // an odd bit left over
    const uint32_t cand = t | (1u << bit);
    const int c = stream_count_ge(lo, hi, key, cand, sm.cnt[par]);
    if (c >= want) { t = cand; at_least = c; } else above = c;
    par ^= 1;
  }
  if (bit >= 0) {
    const uint32_t top = t + (2u << bit);            // end of the undecided range (0 if it wraps: no upper bound)
    const int alive = at_least - above;
#pragma unroll 8
    for (int j = lo + tid; j < hi; j += kThreads) {
      const uint32_t kx = key(j);
      if (kx >= t && (top == 0u || kx < top)) list[atomicAdd(&sm.list_n, 1)] = kx;
    }
    __syncthreads();
    if (warp == 0) {
      const int want2 = want - above;                 // rank inside the collected keys
      for (; bit >= 0; --bit) {
        const uint32_t cand = t | (1u << bit);
        int c = 0;
        for (int i = lane; i < alive; i += 32) c += list[i] >= cand;
        c = __reduce_add_sync(0xffffffffu, c);
        if (c >= want2) t = cand;
      }
      if (lane == 0) sm.list_thr = t;
    }
    __syncthreads();
    t = sm.list_thr;
  }
  const int n_gt = (t == 0xffffffffu) ? 0 : stream_count_ge(lo, hi, key, t + 1u, sm.cnt[par]);
  thr = t;
  need_eq = want - n_gt;
  __syncthreads();
}

// Writes, ascending, every j in [lo, hi) with key > thr plus the first need_eq
// with key == thr.  emit(pos, j) receives the output slot.  Every warp owns a contiguous stretch of positions
// and walks it 32 at a time (coalesced): one pass counts, one block scan places the stretches, one pass
// ranks by ballot and writes.
template <class KeyFn, class Emit>
__device__ void block_compact(SelectSmem& sm, int lo, int hi, uint32_t thr, int need_eq, const KeyFn& key,
                              const Emit& emit) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int stretch = ((hi - lo + kWarps - 1) / kWarps + 31) & ~31;
  const int j0 = min(hi, lo + warp * stretch), j1 = min(hi, j0 + stretch);
  int gt = 0, eq = 0;
#pragma unroll 4
  for (int j = j0 + lane; j < j1; j += 32) {
    const uint32_t kx = key(j);
    gt += kx > thr;
    eq += kx == thr;
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  eq = __reduce_add_sync(0xffffffffu, eq);
  if (lane == 0) sm.scan[warp] = (long long)gt | ((long long)eq << 32);
  __syncthreads();
  const long long wp = sm.scan[lane];
  long long wi = wp;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long y = __shfl_up_sync(0xffffffffu, wi, o);
    if (lane >= o) wi += y;
  }
  const long long wexcl = __shfl_sync(0xffffffffu, wi - wp, warp);
  int gt_before = (int)(wexcl & 0xffffffffll), eq_before = (int)(wexcl >> 32);
  const unsigned lt = (1u << lane) - 1u;
  for (int jb = j0; jb < j1; jb += 32) {              // warp-uniform trip count
    const int j = jb + lane;
    bool g = false, q = false;
    if (j < j1) {
      const uint32_t kx = key(j);
      g = kx > thr;
      q = kx == thr;
    }
    const unsigned gm = __ballot_sync(0xffffffffu, g), qm = __ballot_sync(0xffffffffu, q);
    const int my_gt = gt_before + __popc(gm & lt), my_eq = eq_before + __popc(qm & lt);
    if (g || (q && my_eq < need_eq)) emit(my_gt + min(my_eq, need_eq), j);
    gt_before += __popc(gm);
    eq_before += __popc(qm);
  }
  __syncthreads();
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) select_kernel(DeviceProblem p, UnitRange ur) {
  __shared__ SelectSmem sm;
  __shared__ int sel[TASKKV_MAX_TOP_T];
  __shared__ float red[kWarps][D];

  const int u = ur.unit(blockIdx.x);
  const int N = p.unit_N[u];
  const float* C = p.C + p.c_off[u];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- Eq. 14: I = top-min(t, N) of C
  const int t = min(p.top_t, N);
  uint32_t thr;
  int need_eq;
  const ScoreKey skey{C};
  uint32_t* scratch = reinterpret_cast<uint32_t*>(&red[0][0]);   // free until the semantic vector is summed
  block_stream_select(sm, 0, N, t, skey, scratch, kWarps * D, thr, need_eq);
  int* topt = p.topt + (size_t)u * p.top_t;
  block_compact(sm, 0, N, thr, need_eq, skey, [&](int pos, int j) {
    sel[pos] = j;
    topt[pos] = j;
  });
  for (int i = t + tid; i < p.top_t; i += kThreads) topt[i] = -1;
  __syncthreads();

  // ---- Eq. 15: v' = sum_{j in I} C[j] V[j,:], fixed summation order
  constexpr int EPL = D / 32;   // elements per lane
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  const T* V = static_cast<const T*>(p.v_ptr[u]);
  for (int i = warp; i < t; i += kWarps) {
    const int j = sel[i];
    const float c = C[j];
    const T* row = V + (size_t)j * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(c, to_float(row[e]), acc[e]);
  }
#pragma unroll
  for (int e = 0; e < EPL; ++e) red[warp][lane * EPL + e] = acc[e];
  __syncthreads();
  if (tid < D) {
    float s = 0.f;
    for (int w = 0; w < kWarps; ++w) s += red[w][tid];
    p.sem[(size_t)u * D + tid] = s;
  }

  // ---- Sec. IV-B: sinks, middle activations (top-k of the pooled scores), recent window
  const int s1 = p.sink, s2 = p.recent;
  if (N <= s1 + s2) return;                       // the unit keeps everything
  const int lo = s1, hi = N - s2;
  const int kmid = min(p.unit_mid[u], hi - lo);
  if (kmid >= hi - lo) return;                    // budget covers the whole middle: keeps everything
  int* idx = p.idx + (size_t)u * p.idx_stride;
  for (int i = tid; i < s1; i += kThreads) idx[i] = i;
  for (int i = tid; i < s2; i += kThreads) idx[s1 + kmid + i] = N - s2 + i;
  if (p.mid_policy != TASKKV_MID_SELECT) {
    // Sec. V-G variants: the budget extends the recent window, or names the first position of each of the
    // kmid contiguous groups whose mean becomes a compensation row (written after the gather)
    for (int i = tid; i < kmid; i += kThreads)
      idx[s1 + i] = p.mid_policy == TASKKV_MID_RECENT ? hi - kmid + i
                                                     : lo + (int)(((int64_t)i * (hi - lo)) / kmid);
    return;
  }
  if (kmid > 0) {
    // the pooling-window sums once, into the unit's scratch row, then selected like plain scores
    const int half = (p.pool_w - 1) / 2;
    float* P = p.pooled + p.c_off[u];
#pragma unroll 2
    for (int j = tid; j < N; j += kThreads) {
      float sum = 0.f;                      // added in ascending position, zeros outside [0, N)
      if (j >= half && j + half < N) {
        if (half == 3) {
          sum = C[j - 3]; sum += C[j - 2]; sum += C[j - 1]; sum += C[j]; sum += C[j + 1]; sum += C[j + 2]; sum += C[j + 3];
        } else {
          for (int o = -half; o <= half; ++o) sum += C[j + o];
        }
      } else {
        for (int o = -half; o <= half; ++o) {
          const int q = j + o;
          sum += (q >= 0 && q < N) ? C[q] : 0.f;
        }
      }
      P[j] = sum;
    }
    __syncthreads();
    const ScoreKey qkey{P};
    block_stream_select(sm, lo, hi, kmid, qkey, scratch, kWarps * D, thr, need_eq);
    block_compact(sm, lo, hi, thr, need_eq, qkey, [&](int pos, int j) { idx[s1 + pos] = j; });
  }
}


// ---------------------------------------------------------------------------
// Register-resident variant for N <= 32768 (and pooling kernel 1 or 7): every
// thread keeps 32 consecutive scores in registers, so a selection is a bisection
// over the 32 key bits -- each step is 32 compares per thread plus one block-wide
// count -- and the ordered compaction is a single block scan.  Same results as
// the radix path: exact k-th key, lower position first among equal keys, pooled
// sums added in ascending position.
constexpr int kEpt = 32;

struct FastSmem {
  int cnt[2][kWarps];
  uint32_t mn[kWarps], mx[kWarps];
  int scan[kWarps];
  int scan_tot;
  int list_n;          // keys collected for the narrow phase of the bisection
  uint32_t list_thr;   // its result
};
constexpr int kNarrow = 1023;  // the bisection runs over all keys until at most this many lie in the undecided range

__device__ __forceinline__ int block_count_ge(const uint32_t (&key)[kEpt], uint32_t cand, int* slot) {
  int c = 0;
#pragma unroll
  for (int e = 0; e < kEpt; ++e) c += (key[e] >= cand) ? 1 : 0;
  c = __reduce_add_sync(0xffffffffu, c);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) slot[warp] = c;
  __syncthreads();
  return __reduce_add_sync(0xffffffffu, slot[lane]);
}

// k-th largest key (1 <= want <= number of non-zero keys) and how many keys equal to it belong to the top `want`.
// Every step over all keys also tells how many keys still lie in the undecided range [t, t + 2^(bit+1)); once
// they are few, they are collected into `list` (shared memory, `cap` entries, any order) and one warp settles
// the remaining bits on them.  With many near-equal scores that moment may never come and the bisection simply
// stays on all keys.  The result is the same key either way.
__device__ void block_bisect(FastSmem& fs, const uint32_t (&key)[kEpt], int want, uint32_t* list, int cap,
                             uint32_t& thr, int& need_eq) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // bits above the highest bit in which the non-zero keys differ are common to the answer
  uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll
  for (int e = 0; e < kEpt; ++e)
    if (key[e]) { lo = min(lo, key[e]); hi = max(hi, key[e]); }
  lo = __reduce_min_sync(0xffffffffu, lo);
  hi = __reduce_max_sync(0xffffffffu, hi);
  if (lane == 0) { fs.mn[warp] = lo; fs.mx[warp] = hi; }
  if (threadIdx.x == 0) fs.list_n = 0;
  __syncthreads();
  lo = __reduce_min_sync(0xffffffffu, fs.mn[lane]);
  hi = __reduce_max_sync(0xffffffffu, fs.mx[lane]);
  const uint32_t diff = lo ^ hi;
  int bit = diff ? 31 - __clz(diff) : -1;
  uint32_t t = diff ? (hi & ~((2u << bit) - 1u)) : hi;
  int par = 0;
  int above = 0;           // keys >= t + 2^(bit+1): the last count that fell short of `want`
  int at_least = 1 << 30;  // keys >= t: the last count that reached `want` (unknown before the first one)
  const int narrow = min(cap, kNarrow);
  for (; bit >= 0 && at_least - above > narrow; --bit) {
    const uint32_t cand = t | (1u << bit);
    const int c = block_count_ge(key, cand, fs.cnt[par]);
    if (c >= want) { t = cand; at_least = c; } else above = c;
    par ^= 1;
  }
  if (bit >= 0) {
    const uint32_t top = t + (2u << bit);            // end of the undecided range (0 if it wraps: no upper bound)
    const int alive = at_least - above;
    {
#pragma unroll
      for (int e = 0; e < kEpt; ++e)
        if (key[e] >= t && (top == 0u || key[e] < top)) list[atomicAdd(&fs.list_n, 1)] = key[e];
      __syncthreads();
      // every thread takes one collected key (there are at most as many as threads); two bits per step: the
      // counts above the three thresholds travel packed in one word (10 bits each hold a count <= 1023)
      static_assert(kNarrow <= kThreads && kNarrow < (1 << 10), "one key per thread, three counts per word");
      const uint32_t mine = (int)threadIdx.x < alive ? list[threadIdx.x] : 0u;
      const int want2 = want - above;                 // rank inside the collected keys
      while (bit >= 0) {
        const uint32_t b_hi = 1u << bit, b_lo = bit > 0 ? 1u << (bit - 1) : 0u;
        const uint32_t c10 = t | b_hi, c11 = c10 | b_lo, c01 = t | b_lo;
        int v = (int)(mine >= c10) | ((int)(mine >= c11) << 10) | ((int)(b_lo != 0u && mine >= c01) << 20);
        v = __reduce_add_sync(0xffffffffu, v);
        if (lane == 0) fs.cnt[par][warp] = v;
        __syncthreads();
        v = __reduce_add_sync(0xffffffffu, fs.cnt[par][lane]);
        par ^= 1;
        const int n10 = v & 0x3ff, n11 = (v >> 10) & 0x3ff, n01 = (v >> 20) & 0x3ff;
        if (b_lo != 0u && n11 >= want2) t = c11;
        else if (n10 >= want2) t = c10;
        else if (b_lo != 0u && n01 >= want2) t = c01;
        bit -= 2;
      }
    }
  }
  const int n_gt = (t == 0xffffffffu) ? 0 : block_count_ge(key, t + 1u, fs.cnt[par]);
  thr = t;
  need_eq = want - n_gt;
  __syncthreads();
}

// Ordered compaction of this thread's 32 consecutive positions [base, base + 32): emit(rank, position) for every
// key above thr and for the first need_eq keys equal to it (lower position first).  The comparisons are made once,
// into two bit masks; the selected keys are few per thread, so the emitting loop walks set bits only.
template <class Emit>
__device__ void block_compact_regs(FastSmem& fs, const uint32_t (&key)[kEpt], int base, uint32_t thr, int need_eq,
                                   const Emit& emit) {
  static_assert(kEpt == 32, "one mask bit per key");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t m_gt = 0u, m_ge = 0u;
#pragma unroll
  for (int e = 0; e < kEpt; ++e) {
    m_gt |= (uint32_t)(key[e] > thr) << e;
    m_ge |= (uint32_t)(key[e] >= thr) << e;
  }
  const int gt = __popc(m_gt), eq = __popc(m_ge) - gt;
  const int packed = gt | (eq << 16);
  int incl = packed;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) fs.scan[warp] = incl;
  __syncthreads();
  int wp = fs.scan[lane];
  int wi = wp;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, wi, o);
    if (lane >= o) wi += y;
  }
  const int wexcl = __shfl_sync(0xffffffffu, wi - wp, warp);
  const int excl = incl - packed + wexcl;
  int gt_before = excl & 0xffff, eq_before = excl >> 16;
  for (uint32_t m = m_ge; m != 0u; m &= m - 1u) {
    const int e = __ffs((int)m) - 1;
    const bool g = (m_gt >> e) & 1u;
    if (g || eq_before < need_eq) emit(gt_before + min(eq_before, need_eq), base + e);
    gt_before += g;
    eq_before += !g;
  }
  __syncthreads();
}

template <typename T, int D, int POOL_HALF>
__global__ void __launch_bounds__(kThreads, 1) select_fast_kernel(DeviceProblem p, UnitRange ur) {
  __shared__ FastSmem fs;
  __shared__ int sel[TASKKV_MAX_TOP_T];
  __shared__ float selw[TASKKV_MAX_TOP_T];
  __shared__ float red[kWarps][D];

  const int u = ur.unit(blockIdx.x);
  const int N = p.unit_N[u];
  const float* C = p.C + p.c_off[u];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = tid * kEpt;

  // only the keys are kept (a key maps back to its score exactly); key 0 marks "no element"
  uint32_t key[kEpt];
  if (base + kEpt <= N && ((reinterpret_cast<uintptr_t>(C + base) & 15) == 0)) {
#pragma unroll
    for (int e = 0; e < kEpt; e += 4) {
      const float4 v = *reinterpret_cast<const float4*>(C + base + e);
      key[e] = ordered_key(v.x); key[e + 1] = ordered_key(v.y);
      key[e + 2] = ordered_key(v.z); key[e + 3] = ordered_key(v.w);
    }
  } else {
#pragma unroll
    for (int e = 0; e < kEpt; ++e) key[e] = (base + e < N) ? ordered_key(C[base + e]) : 0u;
  }

  // ---- Eq. 14: I = top-min(t, N) of C
  const int t = min(p.top_t, N);
  uint32_t thr;
  int need_eq;
  uint32_t* scratch = reinterpret_cast<uint32_t*>(&red[0][0]);   // free until the semantic vector is summed
  block_bisect(fs, key, t, scratch, kWarps * D, thr, need_eq);
  int* topt = p.topt + (size_t)u * p.top_t;
  block_compact_regs(fs, key, base, thr, need_eq, [&](int pos, int j) {
    sel[pos] = j;
    selw[pos] = C[j];
    topt[pos] = j;
  });
  for (int i = t + tid; i < p.top_t; i += kThreads) topt[i] = -1;

  // ---- Eq. 15: v' = sum_{j in I} C[j] V[j,:], fixed summation order
  constexpr int EPL = D / 32;
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  const T* V = static_cast<const T*>(p.v_ptr[u]);
  for (int i = warp; i < t; i += kWarps) {
    const float w = selw[i];
    const T* row = V + (size_t)sel[i] * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(w, to_float(row[e]), acc[e]);
  }
#pragma unroll
  for (int e = 0; e < EPL; ++e) red[warp][lane * EPL + e] = acc[e];
  __syncthreads();
  if (tid < D) {
    float s = 0.f;
    for (int w = 0; w < kWarps; ++w) s += red[w][tid];
    p.sem[(size_t)u * D + tid] = s;
  }

  // ---- Sec. IV-B: sinks, middle activations (top-k of the pooled scores), recent window
  const int s1 = p.sink, s2 = p.recent;
  if (N <= s1 + s2) return;
  const int lo = s1, hi = N - s2;
  const int kmid = min(p.unit_mid[u], hi - lo);
  if (kmid >= hi - lo) return;
  int* idx = p.idx + (size_t)u * p.idx_stride;
  for (int i = tid; i < s1; i += kThreads) idx[i] = i;
  for (int i = tid; i < s2; i += kThreads) idx[s1 + kmid + i] = N - s2 + i;
  if (p.mid_policy != TASKKV_MID_SELECT) {
    // Sec. V-G variants: the budget extends the recent window, or names the first position of each of the
    // kmid contiguous groups whose mean becomes a compensation row (written after the gather)
    for (int i = tid; i < kmid; i += kThreads)
      idx[s1 + i] = p.mid_policy == TASKKV_MID_RECENT ? hi - kmid + i
                                                     : lo + (int)(((int64_t)i * (hi - lo)) / kmid);
    return;
  }
  if (kmid == 0) return;

  // pooled window sums in ascending position: ext = [3 left neighbours][32 own][3 right neighbours]
  if (POOL_HALF > 0) {
    float ext[kEpt + 2 * POOL_HALF];
#pragma unroll
    for (int h = 0; h < POOL_HALF; ++h) {
      const int jl = base - POOL_HALF + h, jr = base + kEpt + h;
      ext[h] = (jl >= 0 && jl < N) ? C[jl] : 0.f;
      ext[POOL_HALF + kEpt + h] = (jr < N) ? C[jr] : 0.f;
    }
#pragma unroll
    for (int e = 0; e < kEpt; ++e) ext[POOL_HALF + e] = (base + e < N) ? key_score(key[e]) : 0.f;
#pragma unroll
    for (int e = 0; e < kEpt; ++e) {
      float sum = 0.f;
#pragma unroll
      for (int o = 0; o <= 2 * POOL_HALF; ++o) sum += ext[e + o];
      const int j = base + e;
      key[e] = (j >= lo && j < hi) ? ordered_key(sum) : 0u;
    }
  } else {
#pragma unroll
    for (int e = 0; e < kEpt; ++e) {
      const int j = base + e;
      if (!(j >= lo && j < hi)) key[e] = 0u;
    }
  }
  __syncthreads();
  block_bisect(fs, key, kmid, scratch, kWarps * D, thr, need_eq);
  block_compact_regs(fs, key, base, thr, need_eq, [&](int pos, int j) { idx[s1 + pos] = j; });
}

// ---------------------------------------------------------------------------
// Cluster variant for 32768 < N <= 262144 (and pooling kernel 1 or 7): a thread-block cluster of 2, 4 or 8 CTAs
// owns a unit, CTA c keeps positions [32768 c, 32768 (c + 1)) in registers exactly as select_fast_kernel does, and
// every block-wide count becomes a cluster-wide one: each warp leaves its count in a slot of every CTA's shared
// memory (distributed shared memory), one cluster barrier, and every thread adds up all slots.  The slots are
// double-buffered by step parity: a slot is rewritten two barriers after it was read.  Same results as the other
// two kernels: exact k-th key, lower position first among equal keys, pooled sums added in ascending position.
constexpr int kMaxCS = 8;

struct ClusterSmem {
  int cnt[2][kMaxCS][kWarps];
  int loc[2][kWarps];        // block-local counts of the narrow phase (peers never write here)
  uint32_t mn[kMaxCS][kWarps], mx[kMaxCS][kWarps];
  int tot[2][kMaxCS][2];     // per compaction and CTA: keys above the threshold, keys equal to it
  int scan[kWarps];
  int list_n;                // survivors received from all CTAs
  int loc_n;                 // this CTA's own survivors
  int base[kMaxCS];          // where they go in each CTA's list
};

// Sum over the whole cluster of one int per warp (v: this warp's value, already reduced over the warp).
__device__ __forceinline__ int cluster_sum(cg::cluster_group& cl, ClusterSmem& cs, int cs_n, int rank, int par, int v) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane < cs_n) cl.map_shared_rank(&cs.cnt[par][rank][warp], lane)[0] = v;
  cl.sync();
  int acc = 0;
  for (int r = 0; r < cs_n; ++r) acc += cs.cnt[par][r][lane];
  return __reduce_add_sync(0xffffffffu, acc);
}

__device__ __forceinline__ int cluster_count_ge(cg::cluster_group& cl, ClusterSmem& cs, int cs_n, int rank, int par,
                                                const uint32_t (&key)[kEpt], uint32_t cand) {
  int c = 0;
#pragma unroll
  for (int e = 0; e < kEpt; ++e) c += (key[e] >= cand) ? 1 : 0;
  c = __reduce_add_sync(0xffffffffu, c);
  return cluster_sum(cl, cs, cs_n, rank, par, c);
}

// block_bisect over the keys of the whole cluster.  For the narrow phase every CTA sends its surviving keys to all
// CTAs (at most kNarrow in the whole cluster, so at most one per thread), and each settles the rest on its own copy.
// `list` must hold 2 (kNarrow + 1) words.
__device__ void cluster_bisect(cg::cluster_group& cl, ClusterSmem& cs, int cs_n, int rank, const uint32_t (&key)[kEpt],
                               int want, uint32_t* list, int cap, uint32_t& thr, int& need_eq) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll
  for (int e = 0; e < kEpt; ++e)
    if (key[e]) { lo = min(lo, key[e]); hi = max(hi, key[e]); }
  lo = __reduce_min_sync(0xffffffffu, lo);
  hi = __reduce_max_sync(0xffffffffu, hi);
  if (lane < cs_n) {
    cl.map_shared_rank(&cs.mn[rank][warp], lane)[0] = lo;
    cl.map_shared_rank(&cs.mx[rank][warp], lane)[0] = hi;
  }
  if (threadIdx.x == 0) { cs.list_n = 0; cs.loc_n = 0; }
  cl.sync();
  lo = 0xffffffffu; hi = 0u;
  for (int r = 0; r < cs_n; ++r) { lo = min(lo, cs.mn[r][lane]); hi = max(hi, cs.mx[r][lane]); }
  lo = __reduce_min_sync(0xffffffffu, lo);
  hi = __reduce_max_sync(0xffffffffu, hi);
  const uint32_t diff = lo ^ hi;
  int bit = diff ? 31 - __clz(diff) : -1;
  uint32_t t = diff ? (hi & ~((2u << bit) - 1u)) : hi;
  int par = 0;
  int above = 0;
  int at_least = 1 << 30;
  const int narrow = min(cap - (kNarrow + 1), kNarrow);   // lower half of `list`: the cluster's survivors; upper half: staging
  for (; bit >= 0 && at_least - above > narrow; --bit) {
    const uint32_t cand = t | (1u << bit);
    const int c = cluster_count_ge(cl, cs, cs_n, rank, par, key, cand);
    if (c >= want) { t = cand; at_least = c; } else above = c;
    par ^= 1;
  }
  if (bit >= 0) {
    const uint32_t top = t + (2u << bit);            // end of the undecided range (0 if it wraps: no upper bound)
    const int alive = at_least - above;              // survivors in the whole cluster: at most one per thread
    // this CTA's survivors are staged in the upper half of `list`, then copied into every CTA's lower half at an
    // offset reserved with one remote atomic per CTA (any order: only counts matter)
    uint32_t* stage = list + kNarrow + 1;
#pragma unroll
    for (int e = 0; e < kEpt; ++e)
      if (key[e] >= t && (top == 0u || key[e] < top)) stage[atomicAdd(&cs.loc_n, 1)] = key[e];
    __syncthreads();
    const int n_loc = cs.loc_n;
    if ((int)threadIdx.x < cs_n) cs.base[threadIdx.x] = atomicAdd(cl.map_shared_rank(&cs.list_n, threadIdx.x), n_loc);
    __syncthreads();
    for (int r = 0; r < cs_n; ++r) {
      uint32_t* dst = cl.map_shared_rank(list, r) + cs.base[r];
      for (int i = threadIdx.x; i < n_loc; i += kThreads) dst[i] = stage[i];
    }
    cl.sync();
    // from here on every CTA settles the remaining bits on its own copy, with block barriers only
    const uint32_t mine = (int)threadIdx.x < alive ? list[threadIdx.x] : 0u;
    const int want2 = want - above;                  // rank inside the collected keys
    int lpar = 0;
    while (bit >= 0) {
      const uint32_t b_hi = 1u << bit, b_lo = bit > 0 ? 1u << (bit - 1) : 0u;
      const uint32_t c10 = t | b_hi, c11 = c10 | b_lo, c01 = t | b_lo;
      int v = (int)(mine >= c10) | ((int)(mine >= c11) << 10) | ((int)(b_lo != 0u && mine >= c01) << 20);
      v = __reduce_add_sync(0xffffffffu, v);
      if (lane == 0) cs.loc[lpar][warp] = v;
      __syncthreads();
      v = __reduce_add_sync(0xffffffffu, cs.loc[lpar][lane]);
      lpar ^= 1;
      const int n10 = v & 0x3ff, n11 = (v >> 10) & 0x3ff, n01 = (v >> 20) & 0x3ff;
      if (b_lo != 0u && n11 >= want2) t = c11;
      else if (n10 >= want2) t = c10;
      else if (b_lo != 0u && n01 >= want2) t = c01;
      bit -= 2;
    }
    // keys above the threshold: those above the undecided range plus the survivors above it (no pass over all keys)
    int g = __reduce_add_sync(0xffffffffu, (int)(mine > t));
    if (lane == 0) cs.loc[lpar][warp] = g;
    __syncthreads();
    g = __reduce_add_sync(0xffffffffu, cs.loc[lpar][lane]);
    thr = t;
    need_eq = want - (above + g);
    __syncthreads();
    return;
  }
  const int n_gt = (t == 0xffffffffu) ? 0 : cluster_count_ge(cl, cs, cs_n, rank, par, key, t + 1u);
  thr = t;
  need_eq = want - n_gt;
  __syncthreads();
}

// block_compact_regs with the ranks continued across the CTAs of the cluster (`which` names the totals' slot).
template <class Emit>
__device__ void cluster_compact_regs(cg::cluster_group& cl, ClusterSmem& cs, int cs_n, int rank, int which,
                                     const uint32_t (&key)[kEpt], int base, uint32_t thr, int need_eq,
                                     const Emit& emit) {
  static_assert(kEpt == 32, "one mask bit per key");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t m_gt = 0u, m_ge = 0u;
#pragma unroll
  for (int e = 0; e < kEpt; ++e) {
    m_gt |= (uint32_t)(key[e] > thr) << e;
    m_ge |= (uint32_t)(key[e] >= thr) << e;
  }
  const int gt = __popc(m_gt), eq = __popc(m_ge) - gt;
  const int packed = gt | (eq << 16);                 // a CTA holds 32768 keys: both fields stay below 2^16
  int incl = packed;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) cs.scan[warp] = incl;
  __syncthreads();
  int wp = cs.scan[lane];
  int wi = wp;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, wi, o);
    if (lane >= o) wi += y;
  }
  const int wexcl = __shfl_sync(0xffffffffu, wi - wp, warp);
  const int excl = incl - packed + wexcl;
  const int total = __shfl_sync(0xffffffffu, wi, 31);   // this CTA's totals
  if (warp == 0 && lane < cs_n) {
    int* dst = cl.map_shared_rank(&cs.tot[which][rank][0], lane);
    dst[0] = total & 0xffff;
    dst[1] = (int)((uint32_t)total >> 16);            // 32768 equal keys fill the sign bit of the packed word
  }
  cl.sync();
  int gt_before = excl & 0xffff, eq_before = excl >> 16;
  for (int r = 0; r < rank; ++r) { gt_before += cs.tot[which][r][0]; eq_before += cs.tot[which][r][1]; }
  for (uint32_t m = m_ge; m != 0u; m &= m - 1u) {
    const int e = __ffs((int)m) - 1;
    const bool g = (m_gt >> e) & 1u;
    if (g || eq_before < need_eq) emit(gt_before + min(eq_before, need_eq), base + e);
    gt_before += g;
    eq_before += !g;
  }
  __syncthreads();
}

template <typename T, int D, int POOL_HALF>
__global__ void __launch_bounds__(kThreads, 1) select_cluster_kernel(DeviceProblem p, UnitRange ur) {
  __shared__ ClusterSmem cs;
  __shared__ int sel[TASKKV_MAX_TOP_T];
  __shared__ float selw[TASKKV_MAX_TOP_T];
  __shared__ float red[kWarps][D];
  __shared__ float vpart[kMaxCS][D];

  cg::cluster_group cl = cg::this_cluster();
  const int cs_n = (int)cl.num_blocks();
  const int rank = (int)cl.block_rank();
  const int u = ur.unit(blockIdx.x / cs_n);
  const int N = p.unit_N[u];
  const float* C = p.C + p.c_off[u];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = (rank * kThreads + tid) * kEpt;

  uint32_t key[kEpt];
  if (base + kEpt <= N && ((reinterpret_cast<uintptr_t>(C + base) & 15) == 0)) {
#pragma unroll
    for (int e = 0; e < kEpt; e += 4) {
      const float4 v = *reinterpret_cast<const float4*>(C + base + e);
      key[e] = ordered_key(v.x); key[e + 1] = ordered_key(v.y);
      key[e + 2] = ordered_key(v.z); key[e + 3] = ordered_key(v.w);
    }
  } else {
#pragma unroll
    for (int e = 0; e < kEpt; ++e) key[e] = (base + e < N) ? ordered_key(C[base + e]) : 0u;
  }

  // ---- Eq. 14: I = top-min(t, N) of C; every CTA receives the whole list
  const int t = min(p.top_t, N);
  uint32_t thr;
  int need_eq;
  uint32_t* scratch = reinterpret_cast<uint32_t*>(&red[0][0]);   // free until the semantic vector is summed
  cluster_bisect(cl, cs, cs_n, rank, key, t, scratch, kWarps * D, thr, need_eq);
  int* topt = p.topt + (size_t)u * p.top_t;
  cluster_compact_regs(cl, cs, cs_n, rank, 0, key, base, thr, need_eq, [&](int pos, int j) {
    const float w = C[j];
    for (int r = 0; r < cs_n; ++r) {
      cl.map_shared_rank(&sel[pos], r)[0] = j;
      cl.map_shared_rank(&selw[pos], r)[0] = w;
    }
    topt[pos] = j;
  });
  if (rank == 0)
    for (int i = t + tid; i < p.top_t; i += kThreads) topt[i] = -1;
  cl.sync();

  // ---- Eq. 15: v' = sum_{j in I} C[j] V[j,:]: the CTAs share the t rows, fixed summation order
  constexpr int EPL = D / 32;
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  const T* V = static_cast<const T*>(p.v_ptr[u]);
  for (int i = rank * kWarps + warp; i < t; i += cs_n * kWarps) {
    const float w = selw[i];
    const T* row = V + (size_t)sel[i] * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(w, to_float(row[e]), acc[e]);
  }
#pragma unroll
  for (int e = 0; e < EPL; ++e) red[warp][lane * EPL + e] = acc[e];
  __syncthreads();
  if (tid < D) {
    float s = 0.f;
    for (int w = 0; w < kWarps; ++w) s += red[w][tid];
    cl.map_shared_rank(&vpart[rank][tid], 0)[0] = s;
  }
  cl.sync();
  if (rank == 0 && tid < D) {
    float s = 0.f;
    for (int r = 0; r < cs_n; ++r) s += vpart[r][tid];
    p.sem[(size_t)u * D + tid] = s;
  }

  // ---- Sec. IV-B: sinks, middle activations (top-k of the pooled scores), recent window
  // (every condition below depends on the unit alone, so the CTAs of a cluster leave together)
  const int s1 = p.sink, s2 = p.recent;
  if (N <= s1 + s2) return;
  const int lo = s1, hi = N - s2;
  const int kmid = min(p.unit_mid[u], hi - lo);
  if (kmid >= hi - lo) return;
  int* idx = p.idx + (size_t)u * p.idx_stride;
  const int ctid = rank * kThreads + tid, cthreads = cs_n * kThreads;
  for (int i = ctid; i < s1; i += cthreads) idx[i] = i;
  for (int i = ctid; i < s2; i += cthreads) idx[s1 + kmid + i] = N - s2 + i;
  if (p.mid_policy != TASKKV_MID_SELECT) {
    for (int i = ctid; i < kmid; i += cthreads)
      idx[s1 + i] = p.mid_policy == TASKKV_MID_RECENT ? hi - kmid + i
                                                     : lo + (int)(((int64_t)i * (hi - lo)) / kmid);
    return;
  }
  if (kmid == 0) return;

  if (POOL_HALF > 0) {
    float ext[kEpt + 2 * POOL_HALF];
#pragma unroll
    for (int h = 0; h < POOL_HALF; ++h) {
      const int jl = base - POOL_HALF + h, jr = base + kEpt + h;
      ext[h] = (jl >= 0 && jl < N) ? C[jl] : 0.f;
      ext[POOL_HALF + kEpt + h] = (jr < N) ? C[jr] : 0.f;
    }
#pragma unroll
    for (int e = 0; e < kEpt; ++e) ext[POOL_HALF + e] = (base + e < N) ? key_score(key[e]) : 0.f;
#pragma unroll
    for (int e = 0; e < kEpt; ++e) {
      float sum = 0.f;
#pragma unroll
      for (int o = 0; o <= 2 * POOL_HALF; ++o) sum += ext[e + o];
      const int j = base + e;
      key[e] = (j >= lo && j < hi) ? ordered_key(sum) : 0u;
    }
  } else {
#pragma unroll
    for (int e = 0; e < kEpt; ++e) {
      const int j = base + e;
      if (!(j >= lo && j < hi)) key[e] = 0u;
    }
  }
  __syncthreads();
  cluster_bisect(cl, cs, cs_n, rank, key, kmid, scratch, kWarps * D, thr, need_eq);
  cluster_compact_regs(cl, cs, cs_n, rank, 1, key, base, thr, need_eq, [&](int pos, int j) { idx[s1 + pos] = j; });
}

template <typename T, int D, int POOL_HALF>
cudaError_t launch_cluster_k(const DeviceProblem& p, const UnitRange& ur, int cs_n, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(ur.blocks * cs_n), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = (unsigned)cs_n;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, select_cluster_kernel<T, D, POOL_HALF>, p, ur);
}

// Whether the device can co-schedule at least one cluster of cs_n such CTAs (asked once per cluster size).
template <typename T, int D, int POOL_HALF>
bool cluster_fits(int cs_n) {
  static int cached[kMaxCS + 1] = {0};      // 0 unknown, 1 yes, -1 no
  if (cached[cs_n] == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cs_n, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = (unsigned)cs_n;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, select_cluster_kernel<T, D, POOL_HALF>, &cfg) != cudaSuccess) n = 0;
    cudaGetLastError();
    cached[cs_n] = n > 0 ? 1 : -1;
  }
  return cached[cs_n] > 0;
}

template <typename T, int D>
bool cluster_supported(const DeviceProblem& p, int cs_n) {
  return p.pool_w == 7 ? cluster_fits<T, D, 3>(cs_n) : cluster_fits<T, D, 0>(cs_n);
}

template <typename T, int D>
cudaError_t launch_cluster(const DeviceProblem& p, const UnitRange& ur, int cs_n, cudaStream_t s) {
  return p.pool_w == 7 ? launch_cluster_k<T, D, 3>(p, ur, cs_n, s) : launch_cluster_k<T, D, 0>(p, ur, cs_n, s);
}

template <typename T, int D>
void launch_fast(const DeviceProblem& p, const UnitRange& ur, cudaStream_t s) {
  if (p.pool_w == 7) select_fast_kernel<T, D, 3><<<ur.blocks, kThreads, 0, s>>>(p, ur);
  else select_fast_kernel<T, D, 0><<<ur.blocks, kThreads, 0, s>>>(p, ur);
}

}  // namespace

cudaError_t launch_select(const DeviceProblem& p, int dtype, int max_N, cudaStream_t s, const UnitRange* range) {
  LaunchScope ls(K_SELECT, s);
  const UnitRange ur = range ? *range : UnitRange{0, p.U, p.U, p.U};
  if (ur.blocks <= 0) return cudaSuccess;
  if (max_N <= kThreads * kEpt && (p.pool_w == 7 || p.pool_w == 1)) {
    if (dtype == TASKKV_F32) {
      if (p.d == 64) launch_fast<float, 64>(p, ur, s); else launch_fast<float, 128>(p, ur, s);
    } else {
      if (p.d == 64) launch_fast<__nv_bfloat16, 64>(p, ur, s); else launch_fast<__nv_bfloat16, 128>(p, ur, s);
    }
    return cudaGetLastError();
  }
  if (max_N <= kMaxCS * kThreads * kEpt && (p.pool_w == 7 || p.pool_w == 1)) {
    int cs_n = 2;
    while (cs_n * kThreads * kEpt < max_N) cs_n *= 2;
    const bool fits = dtype == TASKKV_F32
                          ? (p.d == 64 ? cluster_supported<float, 64>(p, cs_n) : cluster_supported<float, 128>(p, cs_n))
                          : (p.d == 64 ? cluster_supported<__nv_bfloat16, 64>(p, cs_n)
                                       : cluster_supported<__nv_bfloat16, 128>(p, cs_n));
    if (fits) {
      if (dtype == TASKKV_F32)
        return p.d == 64 ? launch_cluster<float, 64>(p, ur, cs_n, s) : launch_cluster<float, 128>(p, ur, cs_n, s);
      return p.d == 64 ? launch_cluster<__nv_bfloat16, 64>(p, ur, cs_n, s)
                       : launch_cluster<__nv_bfloat16, 128>(p, ur, cs_n, s);
    }
    // a device that cannot place such a cluster streams the keys instead (below)
  }
  if (dtype == TASKKV_F32) {
    if (p.d == 64) select_kernel<float, 64><<<ur.blocks, kThreads, 0, s>>>(p, ur);
    else select_kernel<float, 128><<<ur.blocks, kThreads, 0, s>>>(p, ur);
  } else {
    if (p.d == 64) select_kernel<__nv_bfloat16, 64><<<ur.blocks, kThreads, 0, s>>>(p, ur);
    else select_kernel<__nv_bfloat16, 128><<<ur.blocks, kThreads, 0, s>>>(p, ur);
  }
  return cudaGetLastError();
}

}  // namespace taskkv
