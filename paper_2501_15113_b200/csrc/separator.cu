// Semantic separator (Sec. IV-A) and cache planning.
//   separator: per (sequence, layer) the center is the mean of the layer's
//     semantic vectors (Eq. 8), each head's distance is the L2 norm of its offset
//     from the center (Eq. 7), heads are ranked far -> near, the first f are
//     heterogeneous (class 1) and the closest of the rest is promoted (class 2).
//     n_kv * d values: done in double precision by one small block.
//   plan: per unit the retained length (N for classes 1/2, sinks + recent +
//     middle budget otherwise), the capacity, and exclusive scans that place the
//     segments in the pools and number the gather / decode work items.
#include "common.cuh"

namespace taskkv {

namespace {

__global__ void __launch_bounds__(128) separator_kernel(DeviceProblem p) {
  grid_dependency_wait();
  __shared__ double center[128];
  __shared__ double dist[TASKKV_MAX_KV_HEADS];
  __shared__ int cls[TASKKV_MAX_KV_HEADS];
  const int br = blockIdx.x;               // b * R + r
  const int n = p.n_kv, d = p.d;
  const int tid = threadIdx.x;
  const float* sem = p.sem + (size_t)br * n * d;

  if (tid < d) {
    double s = 0.0;
    for (int h = 0; h < n; ++h) s += (double)sem[h * d + tid];
    center[tid] = s / (double)n;
  }
  __syncthreads();
  if (tid < n) {
    double s = 0.0;
    for (int x = 0; x < d; ++x) {
      const double o = (double)sem[tid * d + x] - center[x];
      s += o * o;
    }
    dist[tid] = sqrt(s);
  }
  __syncthreads();

  int f = p.nhet[br];
  bool promote = p.promote_center != 0;
  if (p.force_class == 1) f = n;
  if (p.force_class == 0) { f = 0; promote = false; }
  f = max(0, min(f, n));

  if (tid < n) {
    // rank among all heads, farthest first, lower index first on equal distance
    const double me = dist[tid];
    int rank = 0;
    for (int h = 0; h < n; ++h) rank += (dist[h] > me) || (dist[h] == me && h < tid);
    cls[tid] = rank < f ? TASKKV_CLASS_HETERO : TASKKV_CLASS_NON_HETERO;
  }
  __syncthreads();
  if (tid < n) {
    int c = cls[tid];
    if (promote && c == TASKKV_CLASS_NON_HETERO) {
      const double me = dist[tid];
      int nearer = 0;
      for (int h = 0; h < n; ++h)
        if (cls[h] == TASKKV_CLASS_NON_HETERO) nearer += (dist[h] < me) || (dist[h] == me && h < tid);
      if (nearer == 0) c = TASKKV_CLASS_CENTER;
    }
    p.cls[(size_t)br * n + tid] = c;
    p.dist[(size_t)br * n + tid] = (float)dist[tid];
  }
}

constexpr int kPlanThreads = 1024;

// Block-wide exclusive scan of one int64 per thread; the block total is left in
// *total (shared) until the next call.
__device__ int64_t block_excl_scan(int64_t v, int64_t* warp_tot, int64_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int64_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int64_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();                 // readers of the previous call's warp_tot / total are done
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int64_t w = warp_tot[lane];
    int64_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int64_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    warp_tot[lane] = wi - w;
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return incl - v + warp_tot[warp];
}

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(DeviceProblem p) {
  grid_dependency_wait();
  __shared__ int64_t warp_tot[32];
  __shared__ int64_t total;
  int64_t run_rows = 0, run_gather = 0;
  const int tid = threadIdx.x;
  for (int base = 0; base < p.U; base += kPlanThreads) {
    const int u = base + tid;
    int len = 0, cap = 0;
    if (u < p.U) {
      const int N = p.unit_N[u];
      len = N;
      if (p.cls[u] == TASKKV_CLASS_NON_HETERO && N > p.sink + p.recent)
        len = p.sink + p.recent + min(p.unit_mid[u], N - p.sink - p.recent);
      cap = len + p.max_new;
      p.len[u] = len;
      p.cap[u] = cap;
    }
    const int64_t ro = block_excl_scan(cap, warp_tot, &total);
    const int64_t tot_rows = total;
    const int64_t go = block_excl_scan((len + kGatherRows - 1) / kGatherRows, warp_tot, &total);
    const int64_t tot_gather = total;
    if (u < p.U) {
      p.seg_off[u] = run_rows + ro;
      p.gather_off[u] = (int32_t)(run_gather + go);
    }
    run_rows += tot_rows;
    run_gather += tot_gather;
  }
  if (tid == 0) {
    p.seg_off[p.U] = run_rows;
    p.gather_off[p.U] = (int32_t)run_gather;
    if (run_rows > p.pool_rows) set_status(p.status, TASKKV_ESTATE);
  }
  // decode work items: ceil(capacity / kDecodeChunk) per unit, numbered in layer-major order
  __syncthreads();
  int64_t run_items = 0;
  for (int base = 0; base < p.U; base += kPlanThreads) {
    const int w = base + tid;
    const int items = (w < p.U) ? (p.cap[lm_unit(p, w).u] + kDecodeChunk - 1) / kDecodeChunk : 0;
    const int64_t o = block_excl_scan(items, warp_tot, &total);
    if (w < p.U) p.dec_off[w] = (int32_t)(run_items + o);
    run_items += total;
  }
  if (tid == 0) {
    p.dec_off[p.U] = (int32_t)min(run_items, p.max_items);
    if (run_items > p.max_items) set_status(p.status, TASKKV_ESTATE);
  }
}

}  // namespace

cudaError_t launch_separator_plan(const DeviceProblem& p, int n_br, cudaStream_t s) {
  cudaError_t e;
  {
    LaunchScope ls(K_SEPARATOR, s);
    e = launch_dependent(separator_kernel, (unsigned)n_br, 128u, s, p);
  }
  if (e != cudaSuccess) return e;
  {
    LaunchScope ls(K_PLAN, s);
    e = launch_dependent(plan_kernel, 1u, (unsigned)kPlanThreads, s, p);
  }
  return e;
}

}  // namespace taskkv
