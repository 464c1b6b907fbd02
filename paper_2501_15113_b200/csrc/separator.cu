// Semantic separator (Sec. IV-A) and cache planning.
//   separator: per (sequence, layer) the center is the mean of the layer's
//     semantic vectors (Eq. 8), each head's distance is the L2 norm of its offset
//     from the center (Eq. 7), heads are ranked far -> near, the first f are
//     heterogeneous (class 1) and the closest of the rest is promoted (class 2).
//     n_kv * d values: done in double precision by one small block.
//   plan: the same block then gives every unit of its (sequence, layer) the
//     retained length (N for classes 1/2, sinks + recent + middle budget
//     otherwise), the capacity, its place in the pools and its gather / decode
//     work items.  Where the block starts in each of these is known on the host
//     (Eq. 16 fixes how many heads keep everything), so blocks are independent:
//     a layer is planned as soon as its own semantic vectors exist.
#include "common.cuh"

namespace taskkv {

namespace {

__global__ void __launch_bounds__(128) separator_plan_kernel(DeviceProblem p, int layer0, int n_layers) {
  grid_dependency_wait();
  __shared__ double center[128];
  __shared__ double dist[TASKKV_MAX_KV_HEADS];
  __shared__ int cls[TASKKV_MAX_KV_HEADS];
  const int b_seq = blockIdx.x / n_layers, r_lay = layer0 + blockIdx.x % n_layers;
  const int br = b_seq * p.R + r_lay;
  const int nl = p.n_kv, d = p.d;          // heads of this problem (a shard holds nl of the model's n)
  const int n = p.n_kv_model, h0 = p.kv_first;
  const int tid = threadIdx.x;
  const float* sem = p.sem_all ? p.sem_all + (size_t)br * n * d : p.sem + (size_t)br * nl * d;

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
  int c = TASKKV_CLASS_NON_HETERO;
  if (tid < n) {
    c = cls[tid];
    if (promote && c == TASKKV_CLASS_NON_HETERO) {
      const double me = dist[tid];
      int nearer = 0;
      for (int h = 0; h < n; ++h)
        if (cls[h] == TASKKV_CLASS_NON_HETERO) nearer += (dist[h] < me) || (dist[h] == me && h < tid);
      if (nearer == 0) c = TASKKV_CLASS_CENTER;
    }
    if (tid >= h0 && tid < h0 + nl) {      // this problem's own heads
      p.cls[(size_t)br * nl + tid - h0] = c;
      p.dist[(size_t)br * nl + tid - h0] = (float)dist[tid];
    }
  }
  __syncthreads();                 // every thread has read the far / not-far marks
  if (tid < n) cls[tid] = c;
  __syncthreads();

  // ---- plan of this block's units (the problem's own heads)
  __shared__ int s_cap[TASKKV_MAX_KV_HEADS], s_git[TASKKV_MAX_KV_HEADS], s_dit[TASKKV_MAX_KV_HEADS];
  const int B = lm_batch(p);
  const int lm_block = r_lay * B + b_seq;
  int len = 0;
  if (tid < nl) {
    const int u = br * nl + tid;
    const int N = p.unit_N[u];
    len = N;
    if (cls[h0 + tid] == TASKKV_CLASS_NON_HETERO && N > p.sink + p.recent)
      len = p.sink + p.recent + min(p.unit_mid[u], N - p.sink - p.recent);
    const int cap = len + p.max_new;
    p.len[u] = len;
    p.cap[u] = cap;
    s_cap[tid] = cap;
    s_git[tid] = (len + kGatherRows - 1) / kGatherRows;
    s_dit[tid] = (cap + kDecodeChunk - 1) / kDecodeChunk;
  }
  __syncthreads();
  if (tid < nl) {
    int64_t rows_before = 0;
    int git_before = 0, dit_before = 0;
    for (int h = 0; h < tid; ++h) { rows_before += s_cap[h]; git_before += s_git[h]; dit_before += s_dit[h]; }
    const int u = br * nl + tid, w = lm_block * nl + tid;
    p.seg_off[u] = p.seg_base[br] + rows_before;
    p.gather_off[w] = p.gather_base[lm_block] + git_before;
    p.dec_off[w] = p.dec_base[lm_block] + dit_before;
    if (tid == nl - 1) {
      // The block must end exactly where the host placed the next one.  (A shard cannot know how many of the layer's
      // full-cache heads it will hold, so its blocks are sized for the most it can get and may end early: rows and
      // work items between a block's end and the next block's start stay unused, and the kernels skip such items.)
      const int64_t end_rows = p.seg_base[br] + rows_before + s_cap[tid];
      const int end_git = p.gather_base[lm_block] + git_before + s_git[tid];
      const int end_dit = p.dec_base[lm_block] + dit_before + s_dit[tid];
      const bool sharded = n != nl;
      const bool fits = sharded ? (end_rows <= p.seg_base[br + 1] && end_git <= p.gather_base[lm_block + 1] &&
                                   end_dit <= p.dec_base[lm_block + 1])
                                : (end_rows == p.seg_base[br + 1] && end_git == p.gather_base[lm_block + 1] &&
                                   end_dit == p.dec_base[lm_block + 1]);
      if (!fits) set_status(p.status, TASKKV_ESTATE);
      if (br == B * p.R - 1) p.seg_off[p.U] = p.seg_base[br + 1];
      if (lm_block == B * p.R - 1) {
        p.gather_off[p.U] = p.gather_base[lm_block + 1];
        p.dec_off[p.U] = p.dec_base[lm_block + 1];
      }
    }
  }
  // ---- paged cache: the block takes the pages of its units' retained rows off the pool in one step (growth takes
  // pages later, one at a time) and deals them out in unit order
  if (p.page_rows > 0) {
    __shared__ int s_pages[TASKKV_MAX_KV_HEADS];
    __shared__ int s_base;
    if (tid < nl) s_pages[tid] = (len + p.page_rows - 1) / p.page_rows;
    __syncthreads();
    if (tid == 0) {
      int total = 0;
      for (int h = 0; h < nl; ++h) total += s_pages[h];
      s_base = total > 0 ? pool_pop(p, total) : 0;
    }
    __syncthreads();
    if (tid < nl && s_base >= 0) {
      int before = 0;
      for (int h = 0; h < tid; ++h) before += s_pages[h];
      int32_t* tab = p.page_tab + (size_t)(br * nl + tid) * p.page_stride;
      for (int i = 0; i < s_pages[tid]; ++i) tab[i] = p.pool_free[s_base + before + i];
    }
    // an empty pool (ESTATE is set): the block's units hold nothing, so that gather and decode pass them by
    if (tid < nl && s_base < 0) p.len[br * nl + tid] = 0;
  }
}

// Gives every page of the cache's units back to the pool (a paged cache is being destroyed).
__global__ void __launch_bounds__(128) release_pages_kernel(DeviceProblem p) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= p.U) return;
  const int pages = min((p.len[u] + p.page_rows - 1) / p.page_rows, p.page_stride);
  if (pages <= 0) return;
  const int pos = atomicAdd(p.pool_top, pages);
  const int32_t* tab = p.page_tab + (size_t)u * p.page_stride;
  // (a cache left inconsistent by an earlier ESTATE -- a pop from an empty pool -- must not write outside the stack
  // or put a number on it that is no page)
  bool ok = pos >= 0 && pos + pages <= p.pool_pages;
  for (int i = 0; ok && i < pages; ++i) ok = tab[i] >= 0 && tab[i] < p.pool_pages;
  if (ok) {
    for (int i = 0; i < pages; ++i) p.pool_free[pos + i] = tab[i];
  } else {
    atomicSub(p.pool_top, pages);
    set_status(p.status, TASKKV_ESTATE);
  }
  p.len[u] = 0;
}

// Eq. 17 with the budget given as a fraction of the full cache: k = floor((B - N h) / (n - h)) - s1 - s2 with
// B = fraction * n * N token-heads and h the heads of the block that keep everything (Eq. 16's f plus the promoted
// one), clamped to [0, N - s1 - s2].  Every operation is rounded on its own (no fused multiply-add), so the host's
// plan, which sizes the pools from the same formula, gets the same integer.
__global__ void __launch_bounds__(128) budget_kernel(DeviceProblem p, UnitRange ur) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= ur.blocks) return;
  const int u = ur.unit(i);
  const int n = p.n_kv_model, br = u / p.n_kv;      // Eq. 16 and Eq. 17 count over the model's heads
  const int N = p.unit_N[u];
  int f = max(0, min(p.nhet[br], n));
  int h = min(n, f + ((p.promote_center && f < n) ? 1 : 0));
  if (p.force_class == 1) h = n;
  if (p.force_class == 0) h = 0;
  int k = 0;
  if (n > h) {
    const double budget = __dmul_rn(__dmul_rn((double)p.budget_frac, (double)n), (double)N);
    const double per_head = floor(__ddiv_rn(__dsub_rn(budget, __dmul_rn((double)N, (double)h)), (double)(n - h)));
    double kk = per_head - (double)p.sink - (double)p.recent;
    const double room = (double)max(0, N - p.sink - p.recent);
    kk = kk < 0.0 ? 0.0 : kk;
    kk = kk > room ? room : kk;
    k = (int)kk;
  }
  p.unit_mid[u] = k;
}

// The input pointers of one layer's units, from the layer's per-sequence base pointers (passed by value, up to
// kPtrSeqs sequences per launch): only this layer's entries of the tables are written, so calls for different
// layers never touch the same words.
constexpr int kPtrSeqs = 64;
struct LayerBases {
  const void* q[kPtrSeqs];
  const void* k[kPtrSeqs];
  const void* v[kPtrSeqs];
};
__global__ void __launch_bounds__(128) set_layer_pointers_kernel(DeviceProblem p, const __grid_constant__ LayerBases bases,
                                                                 int b0, int nb, int layer, int elem_size) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nb * p.n_kv) return;
  const int bi = i / p.n_kv, h = i % p.n_kv;
  const size_t u = ((size_t)(b0 + bi) * p.R + layer) * p.n_kv + h;
  const size_t N = (size_t)p.unit_N[u], row = (size_t)p.d * elem_size;
  p.q_ptr[u] = static_cast<const unsigned char*>(bases.q[bi]) + (size_t)h * p.rows * row;
  p.k_ptr[u] = static_cast<const unsigned char*>(bases.k[bi]) + (size_t)h * N * row;
  p.v_ptr[u] = static_cast<const unsigned char*>(bases.v[bi]) + (size_t)h * N * row;
}

}  // namespace

cudaError_t launch_set_layer_pointers(const DeviceProblem& p, int batch, int layer, int elem_size, const void* const* q_win,
                                      const void* const* k, const void* const* v, cudaStream_t s) {
  for (int b0 = 0; b0 < batch; b0 += kPtrSeqs) {
    const int nb = batch - b0 < kPtrSeqs ? batch - b0 : kPtrSeqs;
    LayerBases bases = {};
    for (int i = 0; i < nb; ++i) { bases.q[i] = q_win[b0 + i]; bases.k[i] = k[b0 + i]; bases.v[i] = v[b0 + i]; }
    LaunchScope ls(K_PLAN, s);
    set_layer_pointers_kernel<<<(nb * p.n_kv + 127) / 128, 128, 0, s>>>(p, bases, b0, nb, layer, elem_size);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_release_pages(const DeviceProblem& p, cudaStream_t s) {
  if (p.page_rows <= 0 || p.U <= 0) return cudaSuccess;
  LaunchScope ls(K_PLAN, s);
  release_pages_kernel<<<(p.U + 127) / 128, 128, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_budget(const DeviceProblem& p, int batch, int layer0, int n_layers, cudaStream_t s) {
  if (!(p.budget_frac > 0.f)) return cudaSuccess;
  if (n_layers < 0) { layer0 = 0; n_layers = p.R; }
  const UnitRange ur = layer_range(p, batch, layer0, n_layers);
  if (ur.blocks <= 0) return cudaSuccess;
  LaunchScope ls(K_PLAN, s);
  budget_kernel<<<(ur.blocks + 127) / 128, 128, 0, s>>>(p, ur);
  return cudaGetLastError();
}

cudaError_t launch_separator_plan(const DeviceProblem& p, int batch, int layer0, int n_layers, cudaStream_t s) {
  if (n_layers < 0) { layer0 = 0; n_layers = p.R; }
  LaunchScope ls(K_SEPARATOR, s);
  return launch_dependent(separator_plan_kernel, (unsigned)(batch * n_layers), 128u, s, p, layer0, n_layers);
}

}  // namespace taskkv
