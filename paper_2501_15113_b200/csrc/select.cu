// Selection steps of the compressor, one thread block per unit:
//   top-t of C (Eq. 14) and the semantic vector v' = sum_{j in I} C[j] V[j,:] (Eq. 15);
//   the k middle activations: top-k of the average-pooled scores over the
//   intermediate positions [s1, N - s2) (Sec. IV-B, pooling of Sec. V-D), written
//   with the sinks and the recent window as the unit's ascending index list.
// Both selections are an exact block-level radix select on order-preserving
// 32-bit keys (4 passes of 8 bits) followed by an ordered compaction; of equal
// scores the lower position wins.
#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ uint32_t ordered_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct ScoreKey {          // key of C[j]
  const float* C;
  __device__ __forceinline__ uint32_t operator()(int j) const { return ordered_key(C[j]); }
};

struct PooledKey {         // key of the pooling-window sum around j (zeros outside [0, N))
  const float* C;
  int N, half;
  __device__ __forceinline__ uint32_t operator()(int j) const {
    float s = 0.f;
    for (int o = -half; o <= half; ++o) {
      const int q = j + o;
      s += (q >= 0 && q < N) ? C[q] : 0.f;
    }
    return ordered_key(s);
  }
};

struct SelectSmem {
  int hist[256];
  int warp_tot[kWarps];
  uint32_t prefix;
  int remaining;
  int run_gt, run_eq, tile_tot;
};

// Finds the key `thr` of the `want`-th largest element of key(j), j in [lo, hi)
// (1 <= want <= hi - lo), and how many elements equal to thr belong to the top
// `want` (need_eq); elements with key > thr number want - need_eq.
template <class KeyFn>
__device__ void block_radix_select(SelectSmem& sm, int lo, int hi, int want, const KeyFn& key,
                                   uint32_t& thr, int& need_eq) {
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) { sm.prefix = 0u; sm.remaining = want; }
  uint32_t mask = 0u;
  const int trips = (hi - lo + kThreads - 1) / kThreads;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += kThreads) sm.hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = sm.prefix;
    for (int it = 0; it < trips; ++it) {
      const int j = lo + it * kThreads + tid;
      int digit = 256;                       // lanes without a candidate element
      if (j < hi) {
        const uint32_t kx = key(j);
        if ((kx & mask) == prefix) digit = (kx >> shift) & 255;
      }
      // warp-aggregated histogram: one atomic per distinct digit per warp
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      if (digit < 256 && lane == (__ffs(peers) - 1)) atomicAdd(&sm.hist[digit], __popc(peers));
    }
    __syncthreads();
    if (tid < 32) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin holding the `remaining`-th largest
      const int remaining = sm.remaining;
      int local[8], tot = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) { local[b] = sm.hist[255 - 8 * lane - b]; tot += local[b]; }
      int incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      int above = incl - tot;   // elements in bins owned by lower lanes (= larger digits)
      if (above < remaining && remaining <= incl) {
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          if (above < remaining && remaining <= above + local[b]) {
            sm.prefix = prefix | ((uint32_t)(255 - 8 * lane - b) << shift);
            sm.remaining = remaining - above;
          }
          above += local[b];
        }
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  thr = sm.prefix;
  need_eq = sm.remaining;
  __syncthreads();
}

// Writes, ascending, every j in [lo, hi) with key > thr plus the first need_eq
// with key == thr.  emit(pos, j) receives the output slot.
template <class KeyFn, class Emit>
__device__ void block_compact(SelectSmem& sm, int lo, int hi, uint32_t thr, int need_eq, const KeyFn& key,
                              const Emit& emit) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { sm.run_gt = 0; sm.run_eq = 0; }
  __syncthreads();
  const int trips = (hi - lo + kThreads - 1) / kThreads;
  for (int it = 0; it < trips; ++it) {
    const int j = lo + it * kThreads + tid;
    int gt = 0, eq = 0;
    if (j < hi) {
      const uint32_t kx = key(j);
      gt = kx > thr;
      eq = kx == thr;
    }
    // block exclusive scan of the packed pair (gt in the low half, eq in the high half)
    const int packed = gt | (eq << 16);
    int incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) sm.warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int w = sm.warp_tot[lane];
      int wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += y;
      }
      sm.warp_tot[lane] = wi - w;   // exclusive prefix of the warp totals
      if (lane == 31) sm.tile_tot = wi;
    }
    __syncthreads();
    const int excl = incl - packed + sm.warp_tot[warp];
    const int gt_before = sm.run_gt + (excl & 0xffff);
    const int eq_before = sm.run_eq + (excl >> 16);
    if (gt || (eq && eq_before < need_eq)) emit(gt_before + min(eq_before, need_eq), j);
    __syncthreads();
    if (tid == 0) {
      sm.run_gt += sm.tile_tot & 0xffff;
      sm.run_eq += sm.tile_tot >> 16;
    }
    __syncthreads();
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) select_kernel(DeviceProblem p) {
  __shared__ SelectSmem sm;
  __shared__ int sel[TASKKV_MAX_TOP_T];
  __shared__ float red[kWarps][D];

  const int u = blockIdx.x;
  const int N = p.unit_N[u];
  const float* C = p.C + p.c_off[u];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- Eq. 14: I = top-min(t, N) of C
  const int t = min(p.top_t, N);
  uint32_t thr;
  int need_eq;
  const ScoreKey skey{C};
  block_radix_select(sm, 0, N, t, skey, thr, need_eq);
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
  if (kmid > 0) {
    const PooledKey pkey{C, N, (p.pool_w - 1) / 2};
    __syncthreads();
    block_radix_select(sm, lo, hi, kmid, pkey, thr, need_eq);
    block_compact(sm, lo, hi, thr, need_eq, pkey, [&](int pos, int j) { idx[s1 + pos] = j; });
  }
}

}  // namespace

cudaError_t launch_select(const DeviceProblem& p, int dtype, cudaStream_t s) {
  LaunchScope ls(K_SELECT, s);
  if (dtype == TASKKV_F32) {
    if (p.d == 64) select_kernel<float, 64><<<p.U, kThreads, 0, s>>>(p);
    else select_kernel<float, 128><<<p.U, kThreads, 0, s>>>(p);
  } else {
    if (p.d == 64) select_kernel<__nv_bfloat16, 64><<<p.U, kThreads, 0, s>>>(p);
    else select_kernel<__nv_bfloat16, 128><<<p.U, kThreads, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace taskkv
