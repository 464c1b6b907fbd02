// Shared declarations of the Task-KV CUDA library (internal; the public
// boundary is include/taskkv.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "taskkv.h"

namespace taskkv {

constexpr int kDecodeChunk = 512;                 // rows of one split-K decode item
constexpr int kGatherRows = 64;                   // rows of one gather item
constexpr int kScoreChunk = 1024;                 // keys of one window-score work item (CUDA-core path)
constexpr int kTcChunk = 2048;                    // fewest keys of one window-score work item (tensor-core path)
constexpr int kTcParts = 8;                       // partial-statistic slots per work item (one per epilogue warp)
constexpr float kLog2e = 1.4426950408889634f;

// kernel ids for launch counting / timing
enum KernelId : int32_t {
  K_WINDOW_STATS = 0,
  K_WINDOW_REDUCE,
  K_WINDOW_SCORES,
  K_SELECT,
  K_SEPARATOR,
  K_PLAN,
  K_GATHER,
  K_APPEND,
  K_DECODE_ATTN,
  K_DECODE_COMBINE,
  K_WINDOW_TC,
  K_COMPENSATE,
  K_EXACT_SUM,
  K_SELFTEST,
  K_COUNT
};

// Device-side description of one compression / decode problem.  All pointers
// are device pointers into the cache memory or the workspace.
struct DeviceProblem {
  int32_t U;            // units
  int32_t R, n_heads, n_kv, G, d;
  int32_t L;            // window
  int32_t rows;         // G * L
  int32_t rows_pad;     // rows rounded up to 16
  int32_t top_t, pool_w;
  int32_t sink, recent;
  int32_t promote_center, force_class;
  int32_t mid_policy;   // TASKKV_MID_*
  int32_t max_mid;      // largest middle budget of any layer
  // Append and decode address a range of layers of every sequence ("view"): view unit v = (b * view_nl + r') *
  // n_kv + h stands for layer view_l0 + r'.  q, k_new, v_new, out and `lengths` are indexed by view unit.
  int32_t view_l0, view_nl, view_U;
  int32_t max_new;
  float budget_frac;    // > 0: the middle budget follows Eq. 17 from this fraction of the full cache
  // Head sharding: this problem holds KV heads [kv_first, kv_first + n_kv) of a model with n_kv_model per layer.
  // Eq. 8 / Eq. 16 / Eq. 17 count over the model's heads; the separator then reads every head's semantic vector
  // from sem_all ([B*R][n_kv_model][d], gathered from all shards).  Unsharded: n_kv_model = n_kv, kv_first = 0,
  // sem_all = nullptr (the cache's own vectors).
  int32_t n_kv_model, kv_first;
  const float* sem_all;
  int32_t idx_stride;   // ints per unit in idx
  int32_t chunks_max;   // partial-statistic slots per unit (longest sequence)
  int64_t pool_rows;
  int64_t max_items;    // decode work items the scratch can hold
  // per unit tables
  const int32_t* unit_N;      // [U] sequence length
  int32_t* unit_mid;          // [U] middle budget k of the unit's (sequence, layer): from the host's table, or
                              // written by budget_kernel when the budget is given as a fraction (Eq. 17)
  const int32_t* nhet;        // [B*R] far heads per (sequence, layer)
  const int64_t* c_off;       // [U+1] offset of the unit's scores in C
  // Where each (sequence, layer) block of n_kv units starts.  The number of full-cache heads of a block is fixed by
  // Eq. 16 (only which heads is data dependent), so these are known on the host before any kernel runs, and a
  // layer can be planned and gathered without the layers before it.
  const int64_t* seg_base;    // [B*R+1] first pool row of block b * R + r
  const int32_t* gather_base; // [R*B+1] first gather work item of block r * B + b (layer-major)
  const int32_t* dec_base;    // [R*B+1] first decode work item of block r * B + b (layer-major)
  const void** q_ptr;         // [U] -> [rows][d]
  const void** k_ptr;         // [U] -> [N][d]
  const void** v_ptr;         // [U] -> [N][d]
  // results
  int32_t* status;            // sticky status word
  int32_t* len;               // [U]
  int32_t* cap;               // [U]
  int64_t* seg_off;           // [U+1] first pool row
  int32_t* cls;               // [U]
  float* dist;                // [U]
  float* sem;                 // [U][d]
  int32_t* idx;               // [U][idx_stride]
  int32_t* gather_off;        // [U+1] gather work items, indexed layer-major like dec_off
  int32_t* dec_off;           // [U+1] decode work items, indexed by w = (r * B + b) * n_kv + h
  int32_t* step_cnt;          // [U] combine blocks of a unit that finished the current fused step (0 between calls)
  void* k_pool;
  void* v_pool;
  // Paged cache: the pools are arrays of pages of page_rows rows (a multiple of 64) owned by a page pool that several
  // caches share; unit u's row r lives in page page_tab[u * page_stride + r / page_rows] at slot r % page_rows.
  // page_rows == 0: one contiguous segment per unit, starting at seg_off[u].
  int32_t page_rows, page_stride;
  int32_t pool_pages;         // pages of the pool (length of pool_free)
  int32_t* page_tab;          // [U][page_stride]
  int32_t* pool_free;         // the pool's stack of free page ids; the top `*pool_top` entries are free
  int32_t* pool_top;
  // decode scratch
  float* part_acc;            // [items][G][d]
  float* part_ml;             // [items][G][2]
  // workspace
  float* C;                   // scores, units concatenated
  float* pooled;              // [sum N] pooling-window sums of C (only for units too long for the register path)
  float* stat_part;           // [U][chunks_max][rows_pad][2]
  float* stat;                // [U][rows_pad][2]  per row: (max in log2 units, 1/Z), or one offset (tensor-core path)
  int32_t* topt;              // [U][top_t]
};

// launch bookkeeping (api.cu)
void note_launch_begin(int32_t id, cudaStream_t s);
void note_launch_end(int32_t id, cudaStream_t s);

struct LaunchScope {
  int32_t id;
  cudaStream_t s;
  LaunchScope(int32_t id_, cudaStream_t s_) : id(id_), s(s_) { note_launch_begin(id, s); }
  ~LaunchScope() { note_launch_end(id, s); }
};

// A launch over part of the units: `count` consecutive units starting at `first` inside every sequence's block of
// `per_seq` units (units are numbered [sequence][layer][kv head], so this is a range of layers of every sequence).
struct UnitRange {
  int32_t first, count, per_seq, blocks;   // blocks = sequences * count
  __host__ __device__ int unit(int block) const { return (block / count) * per_seq + first + block % count; }
};

// Host-side view of the inputs, for launchers that build per-sequence descriptors.
struct WindowHostInfo {
  int batch;
  const int32_t* seq_lens;      // host [batch]
  const void* const* q;         // host [batch] device pointers: [layers][n][L][d], first layer = base_layer
  const void* const* k;         // host [batch] device pointers: [layers][n_kv][N_b][d], first layer = base_layer
  const void* const* lse;       // host [batch] device pointers to fp32 [layers][n][L] natural-log normalisers of the
                                // window rows, or nullptr: then pass 1 computes them
  int base_layer = 0;           // the layer q[b], k[b], lse[b] point at (0: the tensors hold every layer; r: the
                                // caller passed layer r alone)
};

// The units of layers [layer0, layer0 + n_layers) of every sequence.
inline UnitRange layer_range(const DeviceProblem& p, int batch, int layer0, int n_layers) {
  return UnitRange{layer0 * p.n_kv, n_layers * p.n_kv, p.R * p.n_kv, batch * n_layers * p.n_kv};
}

// Row statistics from caller-supplied normalisers (replaces pass 1): units [u0, u0 + n_units) of one sequence.
cudaError_t launch_lse_to_stat(const DeviceProblem& p, int u0, int n_units, const float* lse, bool tensor_core_format,
                               cudaStream_t s);

// kernel launchers (one per translation unit).  Where a launcher takes (layer0, n_layers) it works on those layers
// of every sequence; n_layers < 0 means all of them.
cudaError_t launch_window_scores(const DeviceProblem& p, int dtype, int max_N, const WindowHostInfo& h,
                                 cudaStream_t s, int layer0 = 0, int n_layers = -1);
bool window_tc_supported(const DeviceProblem& p, int dtype);
cudaError_t launch_window_scores_tc(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0 = 0,
                                    int n_layers = -1);
cudaError_t launch_window_prefix(const DeviceProblem& p, const void* q, const void* k, int heads, int group, int N,
                                 cudaStream_t s);
bool window_res_supported(const DeviceProblem& p, const WindowHostInfo& h);
// layers [layer0, layer0 + n_layers) of every sequence; n_layers < 0: all of them
cudaError_t launch_window_scores_res(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0 = 0,
                                     int n_layers = -1);
cudaError_t launch_select(const DeviceProblem& p, int dtype, int max_N, cudaStream_t s,
                          const UnitRange* range = nullptr);
cudaError_t launch_separator_plan(const DeviceProblem& p, int batch, int layer0, int n_layers, cudaStream_t s);
// Per-unit input pointers of one layer written on the device from the per-sequence bases of that layer
// (q_win[b]: [n][L][d], k[b], v[b]: [n_kv][N_b][d]); host arrays of `batch` device pointers.
cudaError_t launch_set_layer_pointers(const DeviceProblem& p, int batch, int layer, int elem_size, const void* const* q_win,
                                      const void* const* k, const void* const* v, cudaStream_t s);
// paged caches: every page of the cache's units back onto the pool's stack
cudaError_t launch_release_pages(const DeviceProblem& p, cudaStream_t s);
// Eq. 17 on the device for the units of a range of layers (nothing to do unless budget_frac > 0)
cudaError_t launch_budget(const DeviceProblem& p, int batch, int layer0, int n_layers, cudaStream_t s);
// gather work items [item0, item0 + n_items) = those of layers [layer0, layer0 + n_layers) (layer-major numbering)
cudaError_t launch_gather(const DeviceProblem& p, int dtype, int batch, int layer0, int n_layers, int64_t item0,
                          int64_t n_items, cudaStream_t s);
cudaError_t launch_compensate(const DeviceProblem& p, int dtype, const UnitRange& ur, cudaStream_t s);
cudaError_t launch_append(const DeviceProblem& p, int dtype, const void* k_new, const void* v_new,
                          cudaStream_t s);
cudaError_t launch_decode(const DeviceProblem& p, int dtype, const void* q, const int32_t* lengths,
                          const void* k_new, const void* v_new, void* out, cudaStream_t s,
                          bool early_unit_data = false);

// Programmatic dependent launch: a kernel launched with launch_dependent() may be set up, and its blocks may become
// resident, while the kernel before it in the stream is still draining; grid_dependency_wait() at its start returns
// once that kernel has completed and its writes are visible, so the stream's order of effects is unchanged.  (Without
// the launch attribute the wait returns at once.)  This takes the launch latency out of chains of short dependent
// kernels: attention -> combine -> attention of a layer-by-layer decode loop, separator -> plan -> gather.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream (if launched with launch_dependent()) become resident once every block of this
// grid has got here or exited: its blocks then run whatever they do before their own grid_dependency_wait() -- reads
// of tables this grid does not write -- under this grid's tail.  Called after this kernel's own wait, so that by the
// time a dependent block runs, everything before this grid in the stream is complete.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <class... KArgs, class... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// Unit behind view unit v (identity when the view covers every layer).
__device__ __forceinline__ int view_unit(const DeviceProblem& p, int v) {
  if (p.view_nl == p.R) return v;
  const int per = p.view_nl * p.n_kv;
  const int b = v / per;
  return (b * p.R + p.view_l0) * p.n_kv + (v - b * per);
}
// The split-K decode work items are numbered once, at compression, for every unit at its capacity and in
// layer-major order w = (r * batch + b) * n_kv + h: a range of layers is then a contiguous range of items,
// and a decode call needs no planning pass (an item whose rows lie beyond the segment's length is skipped).
__device__ __forceinline__ int lm_batch(const DeviceProblem& p) { return p.U / (p.R * p.n_kv); }
__device__ __forceinline__ int lm_index(const DeviceProblem& p, int u) {      // unit -> layer-major index
  const int h = u % p.n_kv, br = u / p.n_kv;
  return ((br % p.R) * lm_batch(p) + br / p.R) * p.n_kv + h;
}
struct LmUnit { int u, v; };                                                 // unit and view unit
__device__ __forceinline__ LmUnit lm_unit(const DeviceProblem& p, int w) {   // layer-major index -> unit, view unit
  const int B = lm_batch(p);
  const int h = w % p.n_kv, rb = w / p.n_kv;
  const int r = rb / B, b = rb % B;
  LmUnit x;
  x.u = (b * p.R + r) * p.n_kv + h;
  x.v = (b * p.view_nl + (r - p.view_l0)) * p.n_kv + h;
  return x;
}
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Unpack a 16-byte vector of elements into floats: 4 for fp32, 8 for bf16.
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ __forceinline__ static void unpack(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x);
    f[1] = __uint_as_float(r.y);
    f[2] = __uint_as_float(r.z);
    f[3] = __uint_as_float(r.w);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ __forceinline__ static void unpack(const uint4& r, float* f) {
    // a bf16 is the high half of an fp32; the low half of a word is the earlier element
    f[0] = __uint_as_float(r.x << 16);
    f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16);
    f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16);
    f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16);
    f[7] = __uint_as_float(r.w & 0xffff0000u);
  }
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Largest index i in [0, n) with off[i] <= x, for a non-decreasing off[0..n]
// with off[0] <= x < off[n].
__device__ __forceinline__ int upper_unit(const int32_t* off, int n, int x) {
  int lo = 0, hi = n;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// The same by all 32 lanes of a converged warp: 32 probes per round, so 1024 entries take two dependent loads instead
// of ten.  Every lane returns the index.
__device__ __forceinline__ int upper_unit_warp(const int32_t* off, int n, int x, int lane) {
  int lo = 0, hi = n;                                   // off[lo] <= x < off[hi]
  while (hi - lo > 1) {
    const int step = (hi - lo + 31) >> 5;
    const int at = lo + (lane + 1) * step;
    const bool le = at < hi && off[at] <= x;            // true for the lanes below some point: off is non-decreasing
    const int c = __popc(__ballot_sync(0xffffffffu, le));
    hi = min(hi, lo + (c + 1) * step);
    lo += c * step;
  }
  return lo;
}

__device__ __forceinline__ void set_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

// Pool row of row r of unit u (seg = seg_off[u]).  Rows r .. r + n - 1 are consecutive pool rows as long as they do
// not cross a multiple of page_rows.
__device__ __forceinline__ size_t pool_row(const DeviceProblem& p, int u, int64_t seg, int r) {
  if (p.page_rows == 0) return (size_t)seg + (size_t)r;
  const int pg = p.page_tab[(size_t)u * p.page_stride + r / p.page_rows];
  return (size_t)pg * p.page_rows + (size_t)(r % p.page_rows);
}
// Takes n pages off the pool's stack; returns the index of the first of them in pool_free, or -1 (and ESTATE) if the
// pool has fewer -- the host keeps count and refuses such calls before they are launched.
__device__ __forceinline__ int pool_pop(const DeviceProblem& p, int n) {
  const int base = atomicSub(p.pool_top, n) - n;
  if (base < 0) {
    atomicAdd(p.pool_top, n);
    set_status(p.status, TASKKV_ESTATE);
    return -1;
  }
  return base;
}

#endif  // __CUDACC__

}  // namespace taskkv
