// Host side of the Task-KV library: argument validation, exact buffer planning,
// the cache handle, and the kernel sequences behind the exported calls.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"

using namespace taskkv;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct HostPlan {
  taskkv_plan_info info;
  int64_t c_total = 0;
  int32_t max_N = 0, min_N = 0;
  int32_t chunks_max = 0, rows = 0, rows_pad = 0, idx_stride = 0;
  std::vector<int32_t> seq_lens, mid, nhet;     // [B], [B*R] middle budget of a (sequence, layer), [B*R]
  std::vector<int32_t> full;                    // [B*R] full-cache heads
  std::vector<int64_t> layer_items;             // [R] split-K decode items of a layer over all sequences, at capacity
  // where each (sequence, layer) block starts: pool rows (block b * R + r), gather and decode work items (block
  // r * B + b, layer-major); one entry more than blocks
  std::vector<int64_t> seg_base;
  std::vector<int32_t> gather_base, dec_base;
  // paged cache: rows per page (0: contiguous pools inside the cache memory), table entries per unit, pages the
  // compression takes, rows a unit of each kind holds right after compression ([B*R] full / kept lengths)
  int32_t page_rows = 0, page_stride = 0;
  int64_t pages_compress = 0;
  std::vector<int32_t> kept_len;
  size_t o_ptab = 0;
  // byte offsets inside the cache memory
  size_t o_unit_N, o_unit_mid, o_nhet, o_c_off, o_seg_base, o_gbase, o_dbase, o_qp, o_kp, o_vp, meta_bytes;
  size_t o_status, o_len, o_cap, o_seg, o_cls, o_dist, o_sem, o_idx, o_goff, o_doff, o_step, o_pacc, o_pml, o_kpool,
      o_vpool;
  // inside the workspace
  size_t w_C, w_pool, w_spart, w_stat, w_topt;
};

int32_t hetero_count_impl(int32_t n, float beta, int32_t m, int32_t R, int32_t r) {
  const double top = (double)n * (double)beta;
  const double val = (R <= 1) ? top : top - (top - (double)m) / (double)(R - 1) * (double)r;
  long f = (long)std::floor(val + 0.5);
  if (f < 0) f = 0;
  if (f > n) f = n;
  return (int32_t)f;
}

// Eq. 17 with h full-cache heads: floor((B - N h) / (n - h)) - s1 - s2, clamped to [0, N - s1 - s2].
int32_t mid_budget_impl(double budget_tokens, int32_t N, int32_t h_full, int32_t n, int32_t sink, int32_t recent) {
  if (n <= h_full) return 0;
  const double per_head = std::floor((budget_tokens - (double)N * (double)h_full) / (double)(n - h_full));
  double k = per_head - (double)sink - (double)recent;
  const double room = std::max(0, N - sink - recent);
  if (k < 0) k = 0;
  if (k > room) k = room;
  return (int32_t)k;
}

taskkv_status make_plan(const taskkv_params* p, HostPlan& hp, int32_t page_rows = 0) {
  if (page_rows < 0 || page_rows % kGatherRows != 0) return TASKKV_EINVAL;
  if (page_rows > 0 && p && p->shard_kv_heads > 0) return TASKKV_EINVAL;
  hp.page_rows = page_rows;
  if (!p || !p->seq_lens) return TASKKV_EINVAL;
  if (p->n_layers < 1 || p->batch < 1 || p->n_heads < 1 || p->n_kv_heads < 1) return TASKKV_EINVAL;
  if (p->n_kv_heads > TASKKV_MAX_KV_HEADS || p->n_heads % p->n_kv_heads != 0) return TASKKV_EINVAL;
  if (p->head_dim != 64 && p->head_dim != 128) return TASKKV_EINVAL;
  if (p->dtype != TASKKV_F32 && p->dtype != TASKKV_BF16) return TASKKV_EINVAL;
  const int G = p->n_heads / p->n_kv_heads;
  if (G != 1 && G != 2 && G != 4 && G != 8) return TASKKV_EINVAL;
  if (p->window < 1 || (int64_t)G * p->window > TASKKV_MAX_WINDOW_ROWS) return TASKKV_EINVAL;
  if (p->sink < 0 || p->recent < 0 || p->mid_budget < 0 || p->max_new_tokens < 0) return TASKKV_EINVAL;
  if (p->top_t < 1 || p->top_t > TASKKV_MAX_TOP_T) return TASKKV_EINVAL;
  if (p->pool_kernel < 1 || p->pool_kernel > 31 || p->pool_kernel % 2 == 0) return TASKKV_EINVAL;
  if (p->force_class < -1 || p->force_class > 1) return TASKKV_EINVAL;
  if (p->mid_policy < TASKKV_MID_SELECT || p->mid_policy > TASKKV_MID_MEAN) return TASKKV_EINVAL;
  if (!(p->budget_frac >= 0.f) || p->budget_frac > 1.f) return TASKKV_EINVAL;
  if (p->shard_kv_heads < 0 || p->shard_kv_heads > TASKKV_MAX_KV_HEADS) return TASKKV_EINVAL;
  if (p->shard_kv_heads > 0 && (p->shard_first < 0 || p->shard_first + p->n_kv_heads > p->shard_kv_heads)) return TASKKV_EINVAL;
  const int B = p->batch, R = p->n_layers, nkv = p->n_kv_heads;
  const int n_model = p->shard_kv_heads > 0 ? p->shard_kv_heads : nkv;      // heads Eq. 16 / Eq. 17 count over
  if ((int64_t)B * R * nkv > (1 << 20)) return TASKKV_EINVAL;

  hp.seq_lens.assign(p->seq_lens, p->seq_lens + B);
  hp.max_N = 0;
  hp.min_N = INT32_MAX;
  for (int b = 0; b < B; ++b) {
    const int N = hp.seq_lens[b];
    if (N < 1 || N > (1 << 24)) return TASKKV_EINVAL;
    hp.max_N = std::max(hp.max_N, N);
    hp.min_N = std::min(hp.min_N, N);
  }
  if (p->window > hp.min_N) return TASKKV_EINVAL;
  hp.mid.resize((size_t)B * R);
  for (int r = 0; r < R; ++r) {
    const int32_t m = p->mid_budget_per_layer ? p->mid_budget_per_layer[r] : p->mid_budget;
    if (m < 0) return TASKKV_EINVAL;
    for (int b = 0; b < B; ++b) hp.mid[(size_t)b * R + r] = m;
  }
  hp.nhet.resize((size_t)B * R);
  hp.full.resize((size_t)B * R);
  for (int b = 0; b < B; ++b)
    for (int r = 0; r < R; ++r) {
      int f = p->n_hetero ? p->n_hetero[(size_t)b * R + r] : hetero_count_impl(n_model, p->beta, p->m_top, R, r);
      if (f < 0) return TASKKV_EINVAL;
      f = std::min(f, n_model);
      hp.nhet[(size_t)b * R + r] = f;
      int h = std::min(n_model, f + ((p->promote_center && f < n_model) ? 1 : 0));
      if (p->force_class == 1) h = n_model;
      if (p->force_class == 0) h = 0;
      // a shard plans for as many of the layer's full-cache heads as it has heads (which ones it gets is data dependent)
      hp.full[(size_t)b * R + r] = std::min(h, nkv);
      // a budget given as a fraction of the full cache: Eq. 17 per (sequence, layer), with the heads that really
      // keep everything (the device computes the same number for its own table, see budget_kernel)
      if (p->budget_frac > 0.f)
        hp.mid[(size_t)b * R + r] = mid_budget_impl((double)p->budget_frac * (double)n_model * (double)hp.seq_lens[b],
                                                    hp.seq_lens[b], h, n_model, p->sink, p->recent);
    }

  const int64_t U = (int64_t)B * R * nkv;
  const int s1 = p->sink, s2 = p->recent, mn = p->max_new_tokens;
  int64_t pool = 0, kept_rows = 0, gitems = 0, ditems = 0, c_total = 0;
  int32_t stride = 1;
  hp.layer_items.assign((size_t)R, 0);
  hp.seg_base.assign((size_t)B * R + 1, 0);
  hp.kept_len.assign((size_t)B * R, 0);
  hp.pages_compress = 0;
  hp.page_stride = 0;
  std::vector<int64_t> blk_g((size_t)B * R, 0), blk_d((size_t)B * R, 0);   // per block b * R + r
  for (int b = 0; b < B; ++b) {
    const int64_t N = hp.seq_lens[b];
    for (int r = 0; r < R; ++r) {
      const size_t br = (size_t)b * R + r;
      const int64_t h = hp.full[br];
      int64_t kept = N;
      if (N > (int64_t)s1 + s2) kept = s1 + s2 + std::min<int64_t>(hp.mid[br], N - s1 - s2);
      if (kept < N) stride = std::max<int32_t>(stride, (int32_t)kept);
      hp.seg_base[br] = pool;
      hp.kept_len[br] = (int32_t)kept;
      if (page_rows > 0) {
        hp.pages_compress += h * ((N + page_rows - 1) / page_rows) + (nkv - h) * ((kept + page_rows - 1) / page_rows);
        hp.page_stride = std::max<int32_t>(hp.page_stride, (int32_t)((N + mn + page_rows - 1) / page_rows));
      }
      pool += h * (N + mn) + (nkv - h) * (kept + mn);
      kept_rows += h * N + (nkv - h) * kept;
      blk_g[br] = h * ((N + kGatherRows - 1) / kGatherRows) + (nkv - h) * ((kept + kGatherRows - 1) / kGatherRows);
      gitems += blk_g[br];
      const int64_t li = h * ((N + mn + kDecodeChunk - 1) / kDecodeChunk) +
                         (nkv - h) * ((kept + mn + kDecodeChunk - 1) / kDecodeChunk);
      blk_d[br] = li;
      ditems += li;
      hp.layer_items[(size_t)r] += li;
      c_total += (int64_t)nkv * ((N + 3) / 4 * 4);
    }
  }
  hp.seg_base[(size_t)B * R] = pool;
  if (gitems > 0x7fffffff || ditems > 0x7fffffff) return TASKKV_EINVAL;
  // gather and decode work items are numbered layer-major: block r * B + b
  hp.gather_base.assign((size_t)R * B + 1, 0);
  hp.dec_base.assign((size_t)R * B + 1, 0);
  {
    int64_t g = 0, dd = 0;
    for (int r = 0; r < R; ++r)
      for (int b = 0; b < B; ++b) {
        hp.gather_base[(size_t)r * B + b] = (int32_t)g;
        hp.dec_base[(size_t)r * B + b] = (int32_t)dd;
        g += blk_g[(size_t)b * R + r];
        dd += blk_d[(size_t)b * R + r];
      }
    hp.gather_base[(size_t)R * B] = (int32_t)g;
    hp.dec_base[(size_t)R * B] = (int32_t)dd;
  }
  hp.idx_stride = (stride + 3) / 4 * 4;
  hp.c_total = c_total;
  hp.rows = G * p->window;
  hp.rows_pad = (hp.rows + 15) / 16 * 16;
  // partial-statistic slots per unit: one per 1024-key chunk on the CUDA-core path, one per epilogue warp and
  // work item on the tensor-core path
  {
    const int generic = (hp.max_N + kScoreChunk - 1) / kScoreChunk;
    const int tc = (hp.max_N + kTcChunk - 1) / kTcChunk * kTcParts;
    hp.chunks_max = generic > tc ? generic : tc;
  }

  const size_t es = p->dtype == TASKKV_F32 ? 4 : 2;
  const size_t d = p->head_dim;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  hp.o_unit_N = take(U * 4);
  hp.o_unit_mid = take(U * 4);
  hp.o_nhet = take((size_t)B * R * 4);
  hp.o_c_off = take((U + 1) * 8);
  hp.o_seg_base = take(((size_t)B * R + 1) * 8);
  hp.o_gbase = take(((size_t)B * R + 1) * 4);
  hp.o_dbase = take(((size_t)B * R + 1) * 4);
  hp.o_qp = take(U * 8);
  hp.o_kp = take(U * 8);
  hp.o_vp = take(U * 8);
  hp.meta_bytes = o;
  hp.o_status = take(64);
  hp.o_len = take(U * 4);
  hp.o_cap = take(U * 4);
  hp.o_seg = take((U + 1) * 8);
  hp.o_cls = take(U * 4);
  hp.o_dist = take(U * 4);
  hp.o_sem = take(U * d * 4);
  hp.o_idx = take((size_t)U * hp.idx_stride * 4);
  hp.o_goff = take((U + 1) * 4);
  hp.o_doff = take((U + 1) * 4);
  hp.o_step = take(U * 4);
  hp.o_pacc = take((size_t)ditems * G * d * 4);
  hp.o_pml = take((size_t)ditems * G * 2 * 4);
  hp.o_ptab = take(page_rows > 0 ? (size_t)U * hp.page_stride * 4 : 0);
  hp.o_kpool = take(page_rows > 0 ? 0 : (size_t)pool * d * es);      // a paged cache keeps its rows in the pool's pages
  hp.o_vpool = take(page_rows > 0 ? 0 : (size_t)pool * d * es);
  const size_t cache_bytes = o;
  o = 0;
  hp.w_C = take((size_t)c_total * 4);
  // the streaming selection of long units keeps the pooled scores beside C
  hp.w_pool = take(hp.max_N > 32768 || (p->pool_kernel != 7 && p->pool_kernel != 1) ? (size_t)c_total * 4 : 0);
  hp.w_spart = take((size_t)U * hp.chunks_max * hp.rows_pad * 8);
  hp.w_stat = take((size_t)U * hp.rows_pad * 8);
  hp.w_topt = take((size_t)U * p->top_t * 4);
  const size_t work_bytes = o;

  hp.info.n_units = U;
  hp.info.pool_rows = pool;
  hp.info.retained_rows = kept_rows;
  hp.info.cache_bytes = (int64_t)cache_bytes;
  hp.info.workspace_bytes = (int64_t)work_bytes;
  hp.info.max_decode_items = ditems;
  hp.info.gather_items = gitems;
  hp.info.index_stride = hp.idx_stride;
  return TASKKV_OK;
}

// ---------------------------------------------------------------- launch log
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_timing{0};
struct TimingRec { int32_t id; cudaEvent_t a, b; };
std::mutex g_tmu;
std::vector<TimingRec> g_trecs;
thread_local cudaEvent_t tl_start = nullptr;

const char* kKernelNames[K_COUNT] = {
    "window_stats", "window_reduce", "window_scores", "select", "separator", "plan",
    "gather", "append", "decode_attn", "decode_combine", "window_tc", "compensate", "exact_sum", "selftest"};

}  // namespace

namespace taskkv {
void note_launch_begin(int32_t, cudaStream_t s) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g_timing.load(std::memory_order_relaxed)) {
    cudaEventCreate(&tl_start);
    cudaEventRecord(tl_start, s);
  }
}
void note_launch_end(int32_t id, cudaStream_t s) {
  if (g_timing.load(std::memory_order_relaxed) && tl_start) {
    TimingRec r;
    r.id = id;
    r.a = tl_start;
    tl_start = nullptr;
    cudaEventCreate(&r.b);
    cudaEventRecord(r.b, s);
    std::lock_guard<std::mutex> lk(g_tmu);
    g_trecs.push_back(r);
  }
}
}  // namespace taskkv

struct taskkv_pool {
  int32_t page_rows = 0, n_pages = 0, head_dim = 0, dtype = 0;
  void* mem = nullptr;
  bool own = false;
  unsigned char* k_pages = nullptr;   // [n_pages][page_rows][d]
  unsigned char* v_pages = nullptr;
  int32_t* free_ids = nullptr;        // device stack of free page ids
  int32_t* top = nullptr;             // device: number of free pages
  int64_t free_host = 0;              // the host's count (exact: what a call takes follows from the schedules)
  int32_t caches = 0;                 // caches alive
  bool orphan = false;                // taskkv_pool_destroy came while caches were alive: the last one frees the pool
};

struct taskkv_cache {
  taskkv_pool* pool = nullptr;             // paged caches
  std::vector<int32_t> appended;           // [R] tokens appended to layer r so far (paged caches: page accounting)
  int64_t pages_held = 0;                  // pages this cache has taken off its pool
  taskkv_params prm;
  HostPlan hp;
  DeviceProblem dp;
  std::vector<unsigned char> meta;
  void* cache_mem = nullptr;
  void* work_mem = nullptr;
  bool own_cache = false, own_work = false;
  // staging for the host-buffer decode path
  void* stage = nullptr;
  size_t stage_bytes = 0;
  std::vector<unsigned char> layer_done;   // [R] layers compressed so far (layer-streamed caches)
  int shard_stage = 0;                     // head-sharded caches: 1 after begin (vectors ready), 2 after finish
  // The last call that wrote lengths or page tables (compression, append, fused step): its stream and layers.  A
  // decode on the same stream over other layers may read its unit data before its dependency wait (launch_decode).
  bool lw_valid = false;
  cudaStream_t lw_stream = nullptr;
  int32_t lw_l0 = 0, lw_nl = 0;
  unsigned long long lw_capture = 0;       // id of the stream capture that call was recorded in (0: launched directly)
};

namespace {
// Id of the capture `s` is recording into, 0 if it is not capturing.
unsigned long long capture_id(cudaStream_t s) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  unsigned long long id = 0;
  if (cudaStreamGetCaptureInfo(s, &st, &id) != cudaSuccess) {
    cudaGetLastError();
    return ~0ull;                          // unknown: matches nothing
  }
  return st == cudaStreamCaptureStatusActive ? id : 0;
}
void note_length_writer(taskkv_cache* c, int32_t l0, int32_t nl, cudaStream_t s) {
  c->lw_valid = true;
  c->lw_stream = s;
  c->lw_l0 = l0;
  c->lw_nl = nl;
  c->lw_capture = capture_id(s);
}
// Whether the kernel before the next launch on `s` cannot be one of this cache's that writes the lengths or page
// tables of layers [l0, l0 + nl): the last such call went to the same stream (so anything launched on `s` since is
// not one), in the same way -- both launched directly, or both recorded into the same graph, whose replays keep
// their order; a graph's first call never qualifies, whatever ran before a replay -- and covered other layers.
// Conservative otherwise.
bool unit_data_settled(const taskkv_cache* c, int32_t l0, int32_t nl, cudaStream_t s) {
  if (!c->lw_valid || c->lw_stream != s) return false;
  const unsigned long long id = capture_id(s);
  if (id == ~0ull || id != c->lw_capture) return false;
  return l0 + nl <= c->lw_l0 || c->lw_l0 + c->lw_nl <= l0;
}
}  // namespace

namespace {
// Two ways of overlapping the steps of different layers, both over chunks of layers and with streams the library
// owns (per device, created on first use):
//  (1) Multi-head attention (32 window rows): the single-read window kernel is bound by the K stream and its clusters
//      leave part of the SMs empty; the selection is bound by integer work on scores that sit in L2.  The window
//      kernel of chunk i+1 runs on the caller's stream while the selection of chunk i runs on a side stream, joined
//      back before the separator.
//  (2) Grouped queries (64 / 128 window rows): the two-pass window kernel is bound by its epilogue (one exponential
//      per score and pass) and leaves two fifths of the HBM bandwidth unused, while the gather is a pure copy whose
//      blocks need few registers and no shared memory.  Window scores and selection of chunk i+1 run on a
//      high-priority stream; separator, plan and gather of chunk i run beside them on the caller's stream, their
//      blocks placed on the same SMs as the (persistent, one per SM) window CTAs.  Every (sequence, layer) is planned
//      on its own (the host knows where its block of segments starts), which is what lets a chunk be gathered
//      before later layers are classified.
constexpr int kMaxChunks = 8;
struct SideStream {
  cudaStream_t stream = nullptr;      // selection beside window scores (1)
  cudaStream_t hi = nullptr;          // window scores + selection, above the caller's gather in priority (2)
  cudaEvent_t ev[kMaxChunks + 2] = {};
  bool ok = false, tried = false;
};
std::mutex g_side_mu;
SideStream g_side[64];

SideStream* side_stream() {   // call with g_side_mu held
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SideStream& ss = g_side[dev];
  if (!ss.tried) {
    ss.tried = true;
    int lo = 0, hi = 0;
    ss.ok = cudaDeviceGetStreamPriorityRange(&lo, &hi) == cudaSuccess;
    ss.ok = ss.ok && cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking) == cudaSuccess;
    ss.ok = ss.ok && cudaStreamCreateWithPriority(&ss.hi, cudaStreamNonBlocking, hi) == cudaSuccess;
    for (int i = 0; ss.ok && i < kMaxChunks + 2; ++i)
      ss.ok = cudaEventCreateWithFlags(&ss.ev[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ss.ok) cudaGetLastError();
  }
  return ss.ok ? &ss : nullptr;
}

// How many chunks of layers to overlap as in (1) (1 = do not): only where the single-read window kernel and the
// register-resident selection run, with enough units per chunk to fill the window kernel's clusters many times over,
// and not while per-kernel durations are being recorded (they are meant to be those of a kernel running alone).
int overlap_chunks(const DeviceProblem& dp, int dtype, const WindowHostInfo& wh) {
  if (g_timing.load(std::memory_order_relaxed)) return 1;
  if (!window_tc_supported(dp, dtype) || !window_res_supported(dp, wh)) return 1;
  const int batch = wh.batch;
  int chunks = 1;
  while (chunks * 2 <= kMaxChunks && chunks * 2 <= dp.R && (int64_t)(dp.R / (chunks * 2)) * dp.n_kv * batch >= 256)
    chunks *= 2;
  return chunks;
}

// Chunks for (2): where the two-pass tensor-core window kernel runs, up to four chunks of at least 64 units each
// (measured on the 131072-key and the ragged-batch shapes: two chunks hide less of the gather, eight add launches
// and part-filled grids for nothing), and not while per-kernel durations are being recorded.
int gather_overlap_chunks(const DeviceProblem& dp, int dtype, const WindowHostInfo& wh) {
  if (g_timing.load(std::memory_order_relaxed)) return 1;
  if (!window_tc_supported(dp, dtype) || window_res_supported(dp, wh)) return 1;
  int chunks = 1;
  while (chunks * 2 <= 4 && chunks * 2 <= dp.R && (int64_t)(dp.R / (chunks * 2)) * dp.n_kv * wh.batch >= 64)
    chunks *= 2;
  return chunks;
}

// Steps a1-a5 for layers [l0, l0 + nl) of every sequence, one after the other on `s`.
cudaError_t compress_layers(taskkv_cache* c, const WindowHostInfo& wh, int l0, int nl, cudaStream_t s) {
  const DeviceProblem& dp = c->dp;
  const int dtype = c->prm.dtype, B = c->prm.batch;
  const UnitRange ur = layer_range(dp, B, l0, nl);
  cudaError_t e = launch_budget(dp, B, l0, nl, s);
  if (e == cudaSuccess) e = launch_window_scores(dp, dtype, c->hp.max_N, wh, s, l0, nl);
  if (e == cudaSuccess) e = launch_select(dp, dtype, c->hp.max_N, s, &ur);
  if (e == cudaSuccess) e = launch_separator_plan(dp, B, l0, nl, s);
  const int64_t g0 = c->hp.gather_base[(size_t)l0 * B], g1 = c->hp.gather_base[(size_t)(l0 + nl) * B];
  if (e == cudaSuccess) e = launch_gather(dp, dtype, B, l0, nl, g0, g1 - g0, s);
  if (e == cudaSuccess && c->prm.mid_policy == TASKKV_MID_MEAN) e = launch_compensate(dp, dtype, ur, s);
  return e;
}

// (1): window scores of chunk i+1 beside the selection of chunk i; then separator, plan and gather of everything.
cudaError_t compress_window_select_overlapped(taskkv_cache* c, const WindowHostInfo& wh, int n_chunks, cudaStream_t s) {
  const DeviceProblem& dp = c->dp;
  const int dtype = c->prm.dtype, B = c->prm.batch, R = dp.R;
  std::lock_guard<std::mutex> lk(g_side_mu);
  SideStream* ss = side_stream();
  if (!ss) return compress_layers(c, wh, 0, R, s);
  cudaError_t e = launch_budget(dp, B, 0, R, s);
  for (int ch = 0; ch < n_chunks && e == cudaSuccess; ++ch) {
    const int l0 = (int)((int64_t)R * ch / n_chunks), l1 = (int)((int64_t)R * (ch + 1) / n_chunks);
    e = launch_window_scores_res(dp, wh, s, l0, l1 - l0);
    if (e == cudaSuccess) e = cudaEventRecord(ss->ev[ch], s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ss->stream, ss->ev[ch], 0);
    const UnitRange ur = layer_range(dp, B, l0, l1 - l0);
    if (e == cudaSuccess) e = launch_select(dp, dtype, c->hp.max_N, ss->stream, &ur);
  }
  // always join, so that nothing of this call is left running on the side stream when the caller's stream moves on
  cudaError_t j = cudaEventRecord(ss->ev[kMaxChunks], ss->stream);
  if (j == cudaSuccess) j = cudaStreamWaitEvent(s, ss->ev[kMaxChunks], 0);
  if (e == cudaSuccess) e = j;
  if (e == cudaSuccess) e = launch_separator_plan(dp, B, 0, R, s);
  if (e == cudaSuccess) e = launch_gather(dp, dtype, B, 0, R, 0, c->hp.info.gather_items, s);
  if (e == cudaSuccess && c->prm.mid_policy == TASKKV_MID_MEAN) e = launch_compensate(dp, dtype, layer_range(dp, B, 0, R), s);
  return e;
}

// (2): window scores and selection of chunk i+1 (high-priority stream) beside separator, plan and gather of chunk i
// (caller's stream).
cudaError_t compress_gather_overlapped(taskkv_cache* c, const WindowHostInfo& wh, int n_chunks, cudaStream_t s) {
  const DeviceProblem& dp = c->dp;
  const int dtype = c->prm.dtype, B = c->prm.batch, R = dp.R;
  std::lock_guard<std::mutex> lk(g_side_mu);
  SideStream* ss = side_stream();
  if (!ss) return compress_layers(c, wh, 0, R, s);
  // fork: the library's stream starts after everything the caller's stream holds (table upload included)
  cudaError_t e = cudaEventRecord(ss->ev[kMaxChunks + 1], s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ss->hi, ss->ev[kMaxChunks + 1], 0);
  if (e != cudaSuccess) return e;
  e = launch_budget(dp, B, 0, R, ss->hi);
  int joined = -1;
  for (int ch = 0; ch < n_chunks && e == cudaSuccess; ++ch) {
    const int l0 = (int)((int64_t)R * ch / n_chunks), l1 = (int)((int64_t)R * (ch + 1) / n_chunks);
    const UnitRange ur = layer_range(dp, B, l0, l1 - l0);
    e = launch_window_scores(dp, dtype, c->hp.max_N, wh, ss->hi, l0, l1 - l0);
    if (e == cudaSuccess) e = launch_select(dp, dtype, c->hp.max_N, ss->hi, &ur);
    if (e == cudaSuccess) e = cudaEventRecord(ss->ev[ch], ss->hi);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ss->ev[ch], 0);
    if (e != cudaSuccess) break;
    joined = ch;
    e = launch_separator_plan(dp, B, l0, l1 - l0, s);
    const int64_t g0 = c->hp.gather_base[(size_t)l0 * B], g1 = c->hp.gather_base[(size_t)l1 * B];
    if (e == cudaSuccess) e = launch_gather(dp, dtype, B, l0, l1 - l0, g0, g1 - g0, s);
    if (e == cudaSuccess && c->prm.mid_policy == TASKKV_MID_MEAN) e = launch_compensate(dp, dtype, ur, s);
  }
  // always join: nothing of this call may be left running on the library's stream when the caller's stream moves on
  if (joined != n_chunks - 1) {
    cudaError_t j = cudaEventRecord(ss->ev[kMaxChunks], ss->hi);
    if (j == cudaSuccess) j = cudaStreamWaitEvent(s, ss->ev[kMaxChunks], 0);
    if (e == cudaSuccess) e = j;
  }
  return e;
}

// Every layer of every sequence, in the order that suits the shape.
cudaError_t compress_all(taskkv_cache* c, const WindowHostInfo& wh, cudaStream_t s) {
  const int n1 = overlap_chunks(c->dp, c->prm.dtype, wh);
  if (n1 > 1) return compress_window_select_overlapped(c, wh, n1, s);
  const int n2 = gather_overlap_chunks(c->dp, c->prm.dtype, wh);
  if (n2 > 1) return compress_gather_overlapped(c, wh, n2, s);
  return compress_layers(c, wh, 0, c->dp.R, s);
}
}  // namespace

namespace {

void fill_device_problem(taskkv_cache* c) {
  const taskkv_params& p = c->prm;
  const HostPlan& hp = c->hp;
  DeviceProblem& d = c->dp;
  unsigned char* cm = static_cast<unsigned char*>(c->cache_mem);
  unsigned char* wm = static_cast<unsigned char*>(c->work_mem);
  std::memset(&d, 0, sizeof(d));
  d.U = (int32_t)hp.info.n_units;
  d.R = p.n_layers;
  d.n_heads = p.n_heads;
  d.n_kv = p.n_kv_heads;
  d.G = p.n_heads / p.n_kv_heads;
  d.d = p.head_dim;
  d.L = p.window;
  d.rows = hp.rows;
  d.rows_pad = hp.rows_pad;
  d.top_t = p.top_t;
  d.pool_w = p.pool_kernel;
  d.sink = p.sink;
  d.recent = p.recent;
  d.promote_center = p.promote_center;
  d.force_class = p.force_class;
  d.mid_policy = p.mid_policy;
  d.view_l0 = 0;
  d.view_nl = p.n_layers;
  d.view_U = (int32_t)hp.info.n_units;
  d.max_mid = 0;
  for (int32_t m : hp.mid) d.max_mid = m > d.max_mid ? m : d.max_mid;
  if (d.max_mid > hp.max_N) d.max_mid = hp.max_N;
  d.max_new = p.max_new_tokens;
  d.idx_stride = hp.idx_stride;
  d.chunks_max = hp.chunks_max;
  d.pool_rows = hp.info.pool_rows;
  d.max_items = hp.info.max_decode_items;
  d.unit_N = reinterpret_cast<const int32_t*>(cm + hp.o_unit_N);
  d.unit_mid = reinterpret_cast<int32_t*>(cm + hp.o_unit_mid);
  d.seg_base = reinterpret_cast<const int64_t*>(cm + hp.o_seg_base);
  d.gather_base = reinterpret_cast<const int32_t*>(cm + hp.o_gbase);
  d.dec_base = reinterpret_cast<const int32_t*>(cm + hp.o_dbase);
  d.budget_frac = p.budget_frac;
  d.n_kv_model = p.shard_kv_heads > 0 ? p.shard_kv_heads : p.n_kv_heads;
  d.kv_first = p.shard_kv_heads > 0 ? p.shard_first : 0;
  d.sem_all = nullptr;
  d.nhet = reinterpret_cast<const int32_t*>(cm + hp.o_nhet);
  d.c_off = reinterpret_cast<const int64_t*>(cm + hp.o_c_off);
  d.q_ptr = reinterpret_cast<const void**>(cm + hp.o_qp);
  d.k_ptr = reinterpret_cast<const void**>(cm + hp.o_kp);
  d.v_ptr = reinterpret_cast<const void**>(cm + hp.o_vp);
  d.status = reinterpret_cast<int32_t*>(cm + hp.o_status);
  d.len = reinterpret_cast<int32_t*>(cm + hp.o_len);
  d.cap = reinterpret_cast<int32_t*>(cm + hp.o_cap);
  d.seg_off = reinterpret_cast<int64_t*>(cm + hp.o_seg);
  d.cls = reinterpret_cast<int32_t*>(cm + hp.o_cls);
  d.dist = reinterpret_cast<float*>(cm + hp.o_dist);
  d.sem = reinterpret_cast<float*>(cm + hp.o_sem);
  d.idx = reinterpret_cast<int32_t*>(cm + hp.o_idx);
  d.gather_off = reinterpret_cast<int32_t*>(cm + hp.o_goff);
  d.dec_off = reinterpret_cast<int32_t*>(cm + hp.o_doff);
  d.step_cnt = reinterpret_cast<int32_t*>(cm + hp.o_step);
  d.part_acc = reinterpret_cast<float*>(cm + hp.o_pacc);
  d.part_ml = reinterpret_cast<float*>(cm + hp.o_pml);
  d.k_pool = cm + hp.o_kpool;
  d.v_pool = cm + hp.o_vpool;
  d.page_rows = hp.page_rows;
  d.page_stride = hp.page_stride;
  d.page_tab = reinterpret_cast<int32_t*>(cm + hp.o_ptab);
  if (c->pool) {
    d.k_pool = c->pool->k_pages;
    d.v_pool = c->pool->v_pages;
    d.pool_free = c->pool->free_ids;
    d.pool_pages = c->pool->n_pages;
    d.pool_top = c->pool->top;
  }
  if (wm) {
    d.C = reinterpret_cast<float*>(wm + hp.w_C);
    d.pooled = reinterpret_cast<float*>(wm + hp.w_pool);
    d.stat_part = reinterpret_cast<float*>(wm + hp.w_spart);
    d.stat = reinterpret_cast<float*>(wm + hp.w_stat);
    d.topt = reinterpret_cast<int32_t*>(wm + hp.w_topt);
  }
}

// Host copy of the tables at the head of the cache memory: everything but the per-unit input pointers.
void fill_tables(taskkv_cache* c) {
  const taskkv_params& p = c->prm;
  const HostPlan& hp = c->hp;
  const int B = p.batch, R = p.n_layers, nkv = p.n_kv_heads;
  c->meta.assign(hp.meta_bytes, 0);
  unsigned char* m = c->meta.data();
  int32_t* unit_N = reinterpret_cast<int32_t*>(m + hp.o_unit_N);
  int32_t* unit_mid = reinterpret_cast<int32_t*>(m + hp.o_unit_mid);
  int32_t* nhet = reinterpret_cast<int32_t*>(m + hp.o_nhet);
  int64_t* c_off = reinterpret_cast<int64_t*>(m + hp.o_c_off);
  std::memcpy(nhet, hp.nhet.data(), hp.nhet.size() * 4);
  std::memcpy(m + hp.o_seg_base, hp.seg_base.data(), hp.seg_base.size() * 8);
  std::memcpy(m + hp.o_gbase, hp.gather_base.data(), hp.gather_base.size() * 4);
  std::memcpy(m + hp.o_dbase, hp.dec_base.data(), hp.dec_base.size() * 4);
  int64_t coff = 0;
  size_t u = 0;
  for (int b = 0; b < B; ++b) {
    const size_t N = hp.seq_lens[b];
    for (int r = 0; r < R; ++r)
      for (int h = 0; h < nkv; ++h, ++u) {
        unit_N[u] = (int32_t)N;
        unit_mid[u] = hp.mid[(size_t)b * R + r];
        c_off[u] = coff;
        coff += (int64_t)((N + 3) / 4 * 4);
      }
  }
  c_off[u] = coff;
}

// Per-unit input pointers of layers [layer0, layer0 + n_layers): q_win[b], k[b], v[b] point at layer layer0 of
// sequence b ([n_layers][n][L][d] resp. [n_layers][n_kv][N_b][d], contiguous).
void set_layer_pointers(taskkv_cache* c, int layer0, int n_layers, const void* const* q_win, const void* const* k,
                        const void* const* v) {
  const taskkv_params& p = c->prm;
  const HostPlan& hp = c->hp;
  const int B = p.batch, R = p.n_layers, nkv = p.n_kv_heads;
  const int G = p.n_heads / nkv;
  const size_t es = p.dtype == TASKKV_F32 ? 4 : 2;
  const size_t d = p.head_dim;
  unsigned char* m = c->meta.data();
  const void** qp = reinterpret_cast<const void**>(m + hp.o_qp);
  const void** kp = reinterpret_cast<const void**>(m + hp.o_kp);
  const void** vp = reinterpret_cast<const void**>(m + hp.o_vp);
  for (int b = 0; b < B; ++b) {
    const size_t N = hp.seq_lens[b];
    for (int i = 0; i < n_layers; ++i)
      for (int h = 0; h < nkv; ++h) {
        const size_t u = ((size_t)b * R + layer0 + i) * nkv + h;
        qp[u] = static_cast<const unsigned char*>(q_win[b]) + (((size_t)i * p.n_heads + (size_t)h * G) * p.window) * d * es;
        kp[u] = static_cast<const unsigned char*>(k[b]) + (((size_t)i * nkv + h) * N) * d * es;
        vp[u] = static_cast<const unsigned char*>(v[b]) + (((size_t)i * nkv + h) * N) * d * es;
      }
  }
}

taskkv_status cuda_status(cudaError_t e) { return e == cudaSuccess ? TASKKV_OK : TASKKV_ECUDA; }

// The cache's sticky device status word, read after everything on `s` has finished (the synchronising entry points
// report it; the asynchronous ones leave it to the next synchronising call or to taskkv_cache_query).
taskkv_status sticky_status(const taskkv_cache* c, cudaStream_t s) {
  int32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, c->dp.status, sizeof(word), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return TASKKV_ECUDA;
  return (taskkv_status)word;
}

}  // namespace

// ================================================================ exported calls
extern "C" {

void taskkv_params_default(taskkv_params* p) {
  if (!p) return;
  std::memset(p, 0, sizeof(*p));
  p->n_layers = 1;
  p->batch = 1;
  p->sink = 16;
  p->recent = 256;
  p->mid_budget = 0;
  p->window = 32;
  p->top_t = 256;
  p->pool_kernel = 7;
  p->beta = 0.25f;
  p->m_top = 4;
  p->promote_center = 1;
  p->force_class = -1;
  p->mid_policy = TASKKV_MID_SELECT;
  p->dtype = TASKKV_BF16;
  p->max_new_tokens = 0;
}

taskkv_status taskkv_plan(const taskkv_params* p, taskkv_plan_info* out) {
  if (!out) return TASKKV_EINVAL;
  HostPlan hp;
  const taskkv_status st = make_plan(p, hp);
  if (st != TASKKV_OK) return st;
  *out = hp.info;
  return TASKKV_OK;
}

namespace {
taskkv_status compress_impl(const taskkv_params* p, const void* const* q_win, const void* const* k,
                            const void* const* v, const void* const* window_lse, void* cache_mem,
                            size_t cache_bytes, void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                            taskkv_cache** out_cache, taskkv_pool* pool = nullptr);
}  // namespace

taskkv_status taskkv_compress_ex(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                 const void* const* v, void* cache_mem, size_t cache_bytes,
                                 void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                                 taskkv_cache** out_cache) {
  return compress_impl(p, q_win, k, v, nullptr, cache_mem, cache_bytes, workspace_mem, workspace_bytes, stream,
                       out_cache);
}

taskkv_status taskkv_compress_lse(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                  const void* const* v, const void* const* window_lse, void* cache_mem,
                                  size_t cache_bytes, void* workspace_mem, size_t workspace_bytes,
                                  taskkv_stream stream, taskkv_cache** out_cache) {
  if (!window_lse) return TASKKV_EINVAL;
  return compress_impl(p, q_win, k, v, window_lse, cache_mem, cache_bytes, workspace_mem, workspace_bytes, stream,
                       out_cache);
}

namespace {
// Plans the problem, takes or allocates the memory, and puts the tables and a clean state on the device (enqueued
// on `s`); no layer is compressed yet.
taskkv_status cache_create_impl(const taskkv_params* p, void* cache_mem, size_t cache_bytes, void* workspace_mem,
                                size_t workspace_bytes, cudaStream_t s, taskkv_cache** out_cache,
                                taskkv_pool* pool = nullptr) {
  if (!p || !out_cache) return TASKKV_EINVAL;
  *out_cache = nullptr;
  taskkv_cache* c = new (std::nothrow) taskkv_cache();
  if (!c) return TASKKV_EALLOC;
  taskkv_status st = make_plan(p, c->hp, pool ? pool->page_rows : 0);
  if (st != TASKKV_OK) { delete c; return st; }
  if (pool) {
    if (pool->head_dim != p->head_dim || pool->dtype != p->dtype) { delete c; return TASKKV_EINVAL; }
    if (c->hp.pages_compress > pool->free_host) { delete c; return TASKKV_EALLOC; }     // would not fit: nothing launched
    c->pool = pool;
  }
  c->appended.assign((size_t)p->n_layers, 0);
  c->prm = *p;
  c->prm.seq_lens = c->hp.seq_lens.data();
  c->prm.mid_budget_per_layer = nullptr;          // the per-(sequence, layer) budgets live in the plan
  c->prm.n_hetero = c->hp.nhet.data();
  c->layer_done.assign((size_t)p->n_layers, 0);

  if (cache_mem) {
    if (cache_bytes < (size_t)c->hp.info.cache_bytes || ((uintptr_t)cache_mem & (kAlign - 1))) {
      const bool small = cache_bytes < (size_t)c->hp.info.cache_bytes;
      delete c;
      return small ? TASKKV_EALLOC : TASKKV_EINVAL;
    }
    c->cache_mem = cache_mem;
  } else {
    if (cudaMalloc(&c->cache_mem, (size_t)c->hp.info.cache_bytes) != cudaSuccess) {
      cudaGetLastError();
      delete c;
      return TASKKV_EALLOC;
    }
    c->own_cache = true;
  }
  if (workspace_mem) {
    if (workspace_bytes < (size_t)c->hp.info.workspace_bytes || ((uintptr_t)workspace_mem & (kAlign - 1))) {
      const bool small = workspace_bytes < (size_t)c->hp.info.workspace_bytes;
      taskkv_cache_destroy(c);
      return small ? TASKKV_EALLOC : TASKKV_EINVAL;
    }
    c->work_mem = workspace_mem;
  } else {
    if (cudaMalloc(&c->work_mem, (size_t)c->hp.info.workspace_bytes) != cudaSuccess) {
      cudaGetLastError();
      taskkv_cache_destroy(c);
      return TASKKV_EALLOC;
    }
    c->own_work = true;
  }
  fill_device_problem(c);
  fill_tables(c);
  // the tables, then zeros over everything between them and the pools: status word, lengths, capacities, offsets,
  // classes, work lists (a layer that has not been compressed yet has length 0 everywhere)
  cudaError_t e = cudaMemcpyAsync(c->cache_mem, c->meta.data(), c->hp.meta_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(static_cast<unsigned char*>(c->cache_mem) + c->hp.o_status, 0, c->hp.o_pacc - c->hp.o_status, s);
  // page tables: entries of pages a unit does not hold are 0, so that no table entry ever names memory outside the pool
  if (e == cudaSuccess && c->hp.page_rows > 0)
    e = cudaMemsetAsync(static_cast<unsigned char*>(c->cache_mem) + c->hp.o_ptab, 0,
                        (size_t)c->hp.info.n_units * c->hp.page_stride * 4, s);
  if (e != cudaSuccess) {
    cudaGetLastError();
    taskkv_cache_destroy(c);
    return TASKKV_ECUDA;
  }
  *out_cache = c;
  return TASKKV_OK;
}

// Uploads the per-unit input pointer tables (three adjacent arrays of the table area).
cudaError_t upload_pointers(taskkv_cache* c, cudaStream_t s) {
  const HostPlan& hp = c->hp;
  return cudaMemcpyAsync(static_cast<unsigned char*>(c->cache_mem) + hp.o_qp, c->meta.data() + hp.o_qp,
                         hp.meta_bytes - hp.o_qp, cudaMemcpyHostToDevice, s);
}

bool pointers_ok(const taskkv_params* p, const void* const* q_win, const void* const* k, const void* const* v,
                 const void* const* window_lse) {
  for (int b = 0; b < p->batch; ++b) {
    if (!q_win[b] || !k[b] || !v[b] || ((uintptr_t)q_win[b] | (uintptr_t)k[b] | (uintptr_t)v[b]) & 15) return false;
    if (window_lse && (!window_lse[b] || ((uintptr_t)window_lse[b] & 3))) return false;
  }
  return true;
}

taskkv_status compress_impl(const taskkv_params* p, const void* const* q_win, const void* const* k,
                            const void* const* v, const void* const* window_lse, void* cache_mem,
                            size_t cache_bytes, void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                            taskkv_cache** out_cache, taskkv_pool* pool) {
  if (!p || !q_win || !k || !v || !out_cache) return TASKKV_EINVAL;
  *out_cache = nullptr;
  if (p->batch < 1 || !pointers_ok(p, q_win, k, v, window_lse)) return TASKKV_EINVAL;
  if (p->shard_kv_heads > 0) return TASKKV_EINVAL;      // a shard needs the other shards' vectors: begin / finish
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  taskkv_cache* c = nullptr;
  const taskkv_status st = cache_create_impl(p, cache_mem, cache_bytes, workspace_mem, workspace_bytes, s, &c, pool);
  if (st != TASKKV_OK) return st;
  if (pool) {
    pool->free_host -= c->hp.pages_compress;
    c->pages_held = c->hp.pages_compress;
    ++pool->caches;
  }
  set_layer_pointers(c, 0, p->n_layers, q_win, k, v);
  cudaError_t e = upload_pointers(c, s);
  WindowHostInfo wh;
  wh.batch = p->batch;
  wh.seq_lens = c->hp.seq_lens.data();
  wh.q = q_win;
  wh.k = k;
  wh.lse = window_lse;
  wh.base_layer = 0;
  if (e == cudaSuccess) e = compress_all(c, wh, s);
  if (e != cudaSuccess) {
    std::fprintf(stderr, "taskkv_compress_ex: CUDA error: %s\n", cudaGetErrorString(e));
    cudaGetLastError();
    taskkv_cache_destroy(c);
    return TASKKV_ECUDA;
  }
  std::fill(c->layer_done.begin(), c->layer_done.end(), (unsigned char)1);
  *out_cache = c;
  return TASKKV_OK;
}
}  // namespace

size_t taskkv_pool_bytes(int32_t page_rows, int32_t n_pages, int32_t head_dim, int32_t dtype) {
  if (page_rows < kGatherRows || page_rows % kGatherRows != 0 || n_pages < 1) return 0;
  if ((head_dim != 64 && head_dim != 128) || (dtype != TASKKV_F32 && dtype != TASKKV_BF16)) return 0;
  const size_t page = (size_t)page_rows * head_dim * (dtype == TASKKV_F32 ? 4 : 2);
  return 2 * align_up((size_t)n_pages * page) + align_up((size_t)n_pages * 4) + kAlign;
}

taskkv_status taskkv_pool_create(int32_t page_rows, int32_t n_pages, int32_t head_dim, int32_t dtype, void* mem,
                                 size_t bytes, taskkv_stream stream, taskkv_pool** out_pool) {
  if (!out_pool) return TASKKV_EINVAL;
  *out_pool = nullptr;
  const size_t need = taskkv_pool_bytes(page_rows, n_pages, head_dim, dtype);
  if (need == 0) return TASKKV_EINVAL;
  if (mem && (((uintptr_t)mem & (kAlign - 1)) != 0)) return TASKKV_EINVAL;
  if (mem && bytes < need) return TASKKV_EALLOC;
  taskkv_pool* pool = new (std::nothrow) taskkv_pool();
  if (!pool) return TASKKV_EALLOC;
  pool->page_rows = page_rows;
  pool->n_pages = n_pages;
  pool->head_dim = head_dim;
  pool->dtype = dtype;
  if (mem) {
    pool->mem = mem;
  } else {
    if (cudaMalloc(&pool->mem, need) != cudaSuccess) {
      cudaGetLastError();
      delete pool;
      return TASKKV_EALLOC;
    }
    pool->own = true;
  }
  const size_t page = (size_t)page_rows * head_dim * (dtype == TASKKV_F32 ? 4 : 2);
  unsigned char* m = static_cast<unsigned char*>(pool->mem);
  pool->k_pages = m;
  pool->v_pages = m + align_up((size_t)n_pages * page);
  pool->free_ids = reinterpret_cast<int32_t*>(m + 2 * align_up((size_t)n_pages * page));
  pool->top = reinterpret_cast<int32_t*>(m + 2 * align_up((size_t)n_pages * page) + align_up((size_t)n_pages * 4));
  // every page is free: the stack holds n_pages - 1 ... 0, so that page 0 is taken first
  std::vector<int32_t> ids((size_t)n_pages);
  for (int32_t i = 0; i < n_pages; ++i) ids[(size_t)i] = n_pages - 1 - i;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(pool->free_ids, ids.data(), ids.size() * 4, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(pool->top, &n_pages, 4, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);       // the host buffers above go out of scope
  if (e != cudaSuccess) {
    cudaGetLastError();
    taskkv_pool_destroy(pool);
    return TASKKV_ECUDA;
  }
  pool->free_host = n_pages;
  *out_pool = pool;
  return TASKKV_OK;
}

int32_t taskkv_pool_free_pages(const taskkv_pool* pool) { return pool ? (int32_t)pool->free_host : -1; }

namespace {
void free_pool(taskkv_pool* pool) {
  if (pool->own) {
    cudaDeviceSynchronize();
    cudaFree(pool->mem);
  }
  delete pool;
}
}  // namespace

void taskkv_pool_destroy(taskkv_pool* pool) {
  if (!pool) return;
  if (pool->caches > 0) {      // caches still point at it: the last of them to be destroyed frees the pool
    pool->orphan = true;
    return;
  }
  free_pool(pool);
}

taskkv_status taskkv_plan_paged(const taskkv_params* p, int32_t page_rows, taskkv_plan_info* out, int64_t* pages_needed) {
  if (!out || page_rows < kGatherRows) return TASKKV_EINVAL;
  HostPlan hp;
  const taskkv_status st = make_plan(p, hp, page_rows);
  if (st != TASKKV_OK) return st;
  *out = hp.info;
  if (pages_needed) *pages_needed = hp.pages_compress;
  return TASKKV_OK;
}

taskkv_status taskkv_compress_paged(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                    const void* const* v, taskkv_pool* pool, void* cache_mem, size_t cache_bytes,
                                    void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                                    taskkv_cache** out_cache) {
  if (!pool) return TASKKV_EINVAL;
  return compress_impl(p, q_win, k, v, nullptr, cache_mem, cache_bytes, workspace_mem, workspace_bytes, stream,
                       out_cache, pool);
}

taskkv_status taskkv_cache_create(const taskkv_params* p, void* cache_mem, size_t cache_bytes, void* workspace_mem,
                                  size_t workspace_bytes, taskkv_stream stream, taskkv_cache** out_cache) {
  if (p && p->shard_kv_heads > 0) return TASKKV_EINVAL;
  return cache_create_impl(p, cache_mem, cache_bytes, workspace_mem, workspace_bytes,
                           static_cast<cudaStream_t>(stream), out_cache);
}

taskkv_status taskkv_compress_shard_begin(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                          const void* const* v, const void* const* window_lse, void* cache_mem,
                                          size_t cache_bytes, void* workspace_mem, size_t workspace_bytes,
                                          taskkv_stream stream, taskkv_cache** out_cache) {
  if (!p || !q_win || !k || !v || !out_cache) return TASKKV_EINVAL;
  *out_cache = nullptr;
  if (p->batch < 1 || p->shard_kv_heads < 1 || !pointers_ok(p, q_win, k, v, window_lse)) return TASKKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  taskkv_cache* c = nullptr;
  const taskkv_status st = cache_create_impl(p, cache_mem, cache_bytes, workspace_mem, workspace_bytes, s, &c);
  if (st != TASKKV_OK) return st;
  set_layer_pointers(c, 0, p->n_layers, q_win, k, v);
  cudaError_t e = upload_pointers(c, s);
  WindowHostInfo wh;
  wh.batch = p->batch;
  wh.seq_lens = c->hp.seq_lens.data();
  wh.q = q_win;
  wh.k = k;
  wh.lse = window_lse;
  wh.base_layer = 0;
  // Eq. 12-15 for this shard's heads: window scores, top-t, semantic vectors (and the middle top-k, which the select
  // kernels produce in the same pass for every unit; only non-heterogeneous heads will use it)
  if (e == cudaSuccess) e = launch_budget(c->dp, p->batch, 0, p->n_layers, s);
  if (e == cudaSuccess) e = launch_window_scores(c->dp, p->dtype, c->hp.max_N, wh, s);
  if (e == cudaSuccess) e = launch_select(c->dp, p->dtype, c->hp.max_N, s);
  if (e != cudaSuccess) {
    std::fprintf(stderr, "taskkv_compress_shard_begin: CUDA error: %s\n", cudaGetErrorString(e));
    cudaGetLastError();
    taskkv_cache_destroy(c);
    return TASKKV_ECUDA;
  }
  c->shard_stage = 1;
  *out_cache = c;
  return TASKKV_OK;
}

taskkv_status taskkv_cache_semantic(const taskkv_cache* c, const float** device_ptr, int64_t* n_floats) {
  if (!c || !device_ptr) return TASKKV_EINVAL;
  *device_ptr = c->dp.sem;
  if (n_floats) *n_floats = (int64_t)c->dp.U * c->dp.d;
  return TASKKV_OK;
}

taskkv_status taskkv_compress_shard_finish(taskkv_cache* c, const float* sem_all, taskkv_stream stream) {
  if (!c || !sem_all || ((uintptr_t)sem_all & 3)) return TASKKV_EINVAL;
  if (c->shard_stage != 1) return TASKKV_ESTATE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int B = c->prm.batch, R = c->prm.n_layers;
  c->dp.sem_all = sem_all;         // only the separator reads it; the cache keeps no reference afterwards
  c->lw_valid = false;
  cudaError_t e = launch_separator_plan(c->dp, B, 0, R, s);
  c->dp.sem_all = nullptr;
  if (e == cudaSuccess) e = launch_gather(c->dp, c->prm.dtype, B, 0, R, 0, c->hp.info.gather_items, s);
  if (e == cudaSuccess && c->prm.mid_policy == TASKKV_MID_MEAN)
    e = launch_compensate(c->dp, c->prm.dtype, layer_range(c->dp, B, 0, R), s);
  if (e != cudaSuccess) {
    std::fprintf(stderr, "taskkv_compress_shard_finish: CUDA error: %s\n", cudaGetErrorString(e));
    cudaGetLastError();
    return TASKKV_ECUDA;
  }
  c->shard_stage = 2;
  std::fill(c->layer_done.begin(), c->layer_done.end(), (unsigned char)1);
  return TASKKV_OK;
}

taskkv_status taskkv_compress_layer(taskkv_cache* c, int32_t layer, const void* const* q_win, const void* const* k,
                                    const void* const* v, const void* const* window_lse, taskkv_stream stream) {
  if (!c || !q_win || !k || !v) return TASKKV_EINVAL;
  if (c->prm.shard_kv_heads > 0) return TASKKV_EINVAL;
  if (layer < 0 || layer >= c->prm.n_layers || !c->work_mem) return TASKKV_EINVAL;
  if (!pointers_ok(&c->prm, q_win, k, v, window_lse)) return TASKKV_EINVAL;
  if (c->layer_done[(size_t)layer]) return TASKKV_ESTATE;      // a layer's segments are written once
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // this layer's entries of the pointer tables, written on the device: calls for other layers touch other words
  cudaError_t e = launch_set_layer_pointers(c->dp, c->prm.batch, layer, c->prm.dtype == TASKKV_F32 ? 4 : 2, q_win, k, v, s);
  WindowHostInfo wh;
  wh.batch = c->prm.batch;
  wh.seq_lens = c->hp.seq_lens.data();
  wh.q = q_win;
  wh.k = k;
  wh.lse = window_lse;
  wh.base_layer = layer;
  c->lw_valid = false;      // the plan kernel writes this layer's lengths: the next decode reads nothing early
  if (e == cudaSuccess) e = compress_layers(c, wh, layer, 1, s);
  if (e != cudaSuccess) {
    std::fprintf(stderr, "taskkv_compress_layer: CUDA error: %s\n", cudaGetErrorString(e));
    cudaGetLastError();
    return TASKKV_ECUDA;
  }
  c->layer_done[(size_t)layer] = 1;
  return TASKKV_OK;
}

taskkv_status taskkv_compress(const void* q_win, const void* k, const void* v, int32_t n_layers,
                              int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, int32_t seq_len,
                              int32_t sink, int32_t recent, int32_t mid_budget, int32_t window,
                              taskkv_stream stream, taskkv_cache** out_cache) {
  taskkv_params p;
  taskkv_params_default(&p);
  p.n_layers = n_layers;
  p.n_heads = n_heads;
  p.n_kv_heads = n_kv_heads;
  p.head_dim = head_dim;
  p.batch = 1;
  p.seq_lens = &seq_len;
  p.sink = sink;
  p.recent = recent;
  p.mid_budget = mid_budget;
  p.window = window;
  if (n_kv_heads != n_heads) { p.beta = 0.3f; p.m_top = 1; }   // the grouped-query setting of Sec. V-D
  p.max_new_tokens = 4096;
  const void* qa[1] = {q_win};
  const void* ka[1] = {k};
  const void* va[1] = {v};
  return taskkv_compress_ex(&p, qa, ka, va, nullptr, 0, nullptr, 0, stream, out_cache);
}

taskkv_status taskkv_compress_host(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                   const void* const* v, taskkv_stream stream, taskkv_cache** out_cache) {
  if (!p || !q_win || !k || !v || !out_cache) return TASKKV_EINVAL;
  *out_cache = nullptr;
  HostPlan hp;
  taskkv_status st = make_plan(p, hp);
  if (st != TASKKV_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t es = p->dtype == TASKKV_F32 ? 4 : 2;
  const size_t d = p->head_dim;
  const int B = p->batch;
  std::vector<void*> dq(B, nullptr), dk(B, nullptr), dv(B, nullptr);
  auto release = [&]() {
    for (int b = 0; b < B; ++b) { cudaFree(dq[b]); cudaFree(dk[b]); cudaFree(dv[b]); }
  };
  cudaError_t e = cudaSuccess;
  for (int b = 0; b < B && e == cudaSuccess; ++b) {
    if (!q_win[b] || !k[b] || !v[b]) { release(); return TASKKV_EINVAL; }
    const size_t qb = (size_t)p->n_layers * p->n_heads * p->window * d * es;
    const size_t kb = (size_t)p->n_layers * p->n_kv_heads * (size_t)hp.seq_lens[b] * d * es;
    e = cudaMalloc(&dq[b], qb);
    if (e == cudaSuccess) e = cudaMalloc(&dk[b], kb);
    if (e == cudaSuccess) e = cudaMalloc(&dv[b], kb);
    if (e != cudaSuccess) { cudaGetLastError(); release(); return TASKKV_EALLOC; }
    e = cudaMemcpyAsync(dq[b], q_win[b], qb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dk[b], k[b], kb, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv[b], v[b], kb, cudaMemcpyHostToDevice, s);
  }
  if (e != cudaSuccess) { release(); return TASKKV_ECUDA; }
  st = taskkv_compress_ex(p, dq.data(), dk.data(), dv.data(), nullptr, 0, nullptr, 0, stream, out_cache);
  e = cudaStreamSynchronize(s);
  release();
  if (st == TASKKV_OK && e != cudaSuccess) st = TASKKV_ECUDA;
  // a kernel that gave up on a bounded wait leaves its code in the cache's status word: the cache is then unusable
  if (st == TASKKV_OK) st = sticky_status(*out_cache, s);
  if (st != TASKKV_OK && *out_cache) {
    taskkv_cache_destroy(*out_cache);
    *out_cache = nullptr;
  }
  return st;
}

namespace {
// The cache's problem description restricted to layers [layer_begin, layer_begin + layer_count) of every sequence.
bool layer_view(const taskkv_cache* c, int32_t layer_begin, int32_t layer_count, taskkv::DeviceProblem* out) {
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c->dp.R) return false;
  *out = c->dp;
  out->view_l0 = layer_begin;
  out->view_nl = layer_count;
  out->view_U = c->prm.batch * layer_count * c->dp.n_kv;
  // the attention grid is sized by the work items of the layers in view, not of the whole cache
  int64_t items = 0;
  for (int32_t r = layer_begin; r < layer_begin + layer_count; ++r) items += c->hp.layer_items[(size_t)r];
  out->max_items = items;
  return true;
}
}  // namespace

namespace {
// Paged caches: the pages that appending one token to layers [l0, l0 + nl) takes off the pool -- a unit needs one when
// its last page is full -- and the bookkeeping once the call is accepted.  Which units are the long ones is known only
// on the device, how many of each kind a (sequence, layer) has is fixed by Eq. 16, so the count is exact.
int64_t append_pages(const taskkv_cache* c, int32_t l0, int32_t nl) {
  if (!c->pool) return 0;
  const int P = c->hp.page_rows, B = c->prm.batch, R = c->prm.n_layers, nkv = c->prm.n_kv_heads;
  int64_t need = 0;
  for (int r = l0; r < l0 + nl; ++r) {
    const int a = c->appended[(size_t)r];
    if (a >= c->prm.max_new_tokens) continue;                 // at capacity: nothing is appended
    for (int b = 0; b < B; ++b) {
      const size_t br = (size_t)b * R + r;
      const int64_t h = c->hp.full[br];
      if ((c->hp.seq_lens[b] + a) % P == 0) need += h;
      if ((c->hp.kept_len[br] + a) % P == 0) need += nkv - h;
    }
  }
  return need;
}
taskkv_status take_append_pages(taskkv_cache* c, int32_t l0, int32_t nl) {
  if (!c->pool) return TASKKV_OK;
  const int64_t need = append_pages(c, l0, nl);
  if (need > c->pool->free_host) return TASKKV_EALLOC;
  c->pool->free_host -= need;
  c->pages_held += need;
  for (int r = l0; r < l0 + nl; ++r)
    if (c->appended[(size_t)r] < c->prm.max_new_tokens) ++c->appended[(size_t)r];
  return TASKKV_OK;
}
}  // namespace

taskkv_status taskkv_append_ex(taskkv_cache* c, const void* k_new, const void* v_new, int32_t layer_begin,
                               int32_t layer_count, taskkv_stream stream) {
  if (!c || !k_new || !v_new || (((uintptr_t)k_new | (uintptr_t)v_new) & 15)) return TASKKV_EINVAL;
  taskkv::DeviceProblem view;
  if (!layer_view(c, layer_begin, layer_count, &view)) return TASKKV_EINVAL;
  const taskkv_status st = take_append_pages(c, layer_begin, layer_count);
  if (st != TASKKV_OK) return st;
  note_length_writer(c, layer_begin, layer_count, static_cast<cudaStream_t>(stream));
  return cuda_status(launch_append(view, c->prm.dtype, k_new, v_new, static_cast<cudaStream_t>(stream)));
}

taskkv_status taskkv_append(taskkv_cache* c, const void* k_new, const void* v_new, taskkv_stream stream) {
  if (!c) return TASKKV_EINVAL;
  return taskkv_append_ex(c, k_new, v_new, 0, c->dp.R, stream);
}

taskkv_status taskkv_decode_ex(const void* q, taskkv_cache* c, const int32_t* lengths, void* out,
                               int32_t layer_begin, int32_t layer_count, taskkv_stream stream) {
  if (!c || !q || !out || (((uintptr_t)q | (uintptr_t)out) & 15)) return TASKKV_EINVAL;
  taskkv::DeviceProblem view;
  if (!layer_view(c, layer_begin, layer_count, &view)) return TASKKV_EINVAL;
  return cuda_status(launch_decode(view, c->prm.dtype, q, lengths, nullptr, nullptr, out,
                                   static_cast<cudaStream_t>(stream),
                                   unit_data_settled(c, layer_begin, layer_count, static_cast<cudaStream_t>(stream))));
}

taskkv_status taskkv_decode_step_ex(const void* q, const void* k_new, const void* v_new, taskkv_cache* c, void* out,
                                    int32_t layer_begin, int32_t layer_count, taskkv_stream stream) {
  if (!c || !q || !out || !k_new || !v_new) return TASKKV_EINVAL;
  if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)k_new | (uintptr_t)v_new) & 15) return TASKKV_EINVAL;
  taskkv::DeviceProblem view;
  if (!layer_view(c, layer_begin, layer_count, &view)) return TASKKV_EINVAL;
  const taskkv_status st = take_append_pages(c, layer_begin, layer_count);
  if (st != TASKKV_OK) return st;
  const bool early = unit_data_settled(c, layer_begin, layer_count, static_cast<cudaStream_t>(stream));
  note_length_writer(c, layer_begin, layer_count, static_cast<cudaStream_t>(stream));
  return cuda_status(launch_decode(view, c->prm.dtype, q, nullptr, k_new, v_new, out,
                                   static_cast<cudaStream_t>(stream), early));
}

taskkv_status taskkv_decode_step(const void* q, const void* k_new, const void* v_new, taskkv_cache* c, void* out,
                                 taskkv_stream stream) {
  if (!c) return TASKKV_EINVAL;
  return taskkv_decode_step_ex(q, k_new, v_new, c, out, 0, c->dp.R, stream);
}

taskkv_status taskkv_decode(const void* q, taskkv_cache* c, const int32_t* lengths, void* out,
                            taskkv_stream stream) {
  if (!c) return TASKKV_EINVAL;
  return taskkv_decode_ex(q, c, lengths, out, 0, c->dp.R, stream);
}

taskkv_status taskkv_decode_host(const void* q, const void* k_new, const void* v_new, taskkv_cache* c,
                                 void* out, taskkv_stream stream) {
  if (!c || !q || !out || ((k_new == nullptr) != (v_new == nullptr))) return TASKKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t es = c->prm.dtype == TASKKV_F32 ? 4 : 2;
  const size_t qb = align_up((size_t)c->dp.U * c->dp.G * c->dp.d * es);
  const size_t kb = align_up((size_t)c->dp.U * c->dp.d * es);
  const size_t need = 2 * qb + 2 * kb;
  if (c->stage_bytes < need) {
    cudaFree(c->stage);
    c->stage = nullptr;
    c->stage_bytes = 0;
    if (cudaMalloc(&c->stage, need) != cudaSuccess) { cudaGetLastError(); return TASKKV_EALLOC; }
    c->stage_bytes = need;
  }
  unsigned char* st = static_cast<unsigned char*>(c->stage);
  void* dq = st;
  void* dout = st + qb;
  void* dkn = st + 2 * qb;
  void* dvn = st + 2 * qb + kb;
  const size_t q_bytes = (size_t)c->dp.U * c->dp.G * c->dp.d * es;
  const size_t k_bytes = (size_t)c->dp.U * c->dp.d * es;
  cudaError_t e = cudaMemcpyAsync(dq, q, q_bytes, cudaMemcpyHostToDevice, s);
  if (k_new && e == cudaSuccess) {
    e = cudaMemcpyAsync(dkn, k_new, k_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dvn, v_new, k_bytes, cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess && k_new && take_append_pages(c, 0, c->dp.R) != TASKKV_OK) return TASKKV_EALLOC;
  if (e == cudaSuccess)
    if (k_new) note_length_writer(c, 0, c->dp.R, s);
    e = launch_decode(c->dp, c->prm.dtype, dq, nullptr, k_new ? dkn : nullptr, k_new ? dvn : nullptr, dout, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(out, dout, q_bytes, cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return TASKKV_ECUDA;
  return sticky_status(c, s);      // synchronises; ESTATE if a unit was at capacity, ETIMEOUT after a device time-out
}

int64_t taskkv_cache_query_bytes(const taskkv_cache* c, int32_t what) {
  if (!c) return -1;
  const int64_t U = c->dp.U;
  const int64_t es = c->prm.dtype == TASKKV_F32 ? 4 : 2;
  switch (what) {
    case TASKKV_Q_LENGTHS: case TASKKV_Q_CLASSES: case TASKKV_Q_DIST: case TASKKV_Q_CAPACITY: return U * 4;
    case TASKKV_Q_SEMVEC: return U * c->dp.d * 4;
    case TASKKV_Q_OFFSETS: return (U + 1) * 8;
    case TASKKV_Q_INDICES: return U * c->dp.idx_stride * 4;
    case TASKKV_Q_SCORES: return c->work_mem ? c->hp.c_total * 4 : -1;
    case TASKKV_Q_TOPT: return c->work_mem ? U * c->dp.top_t * 4 : -1;
    case TASKKV_Q_STATUS: return 4;
    case TASKKV_Q_KPOOL: case TASKKV_Q_VPOOL:
      return (c->pool ? (int64_t)c->pool->n_pages * c->pool->page_rows : c->dp.pool_rows) * c->dp.d * es;
    case TASKKV_Q_PAGETAB: return c->pool ? U * c->dp.page_stride * 4 : -1;
    default: return -1;
  }
}

taskkv_status taskkv_cache_query(const taskkv_cache* c, int32_t what, void* host_dst, size_t bytes) {
  if (!c || !host_dst) return TASKKV_EINVAL;
  const int64_t need = taskkv_cache_query_bytes(c, what);
  if (need < 0 || bytes < (size_t)need) return TASKKV_EINVAL;
  const void* src = nullptr;
  switch (what) {
    case TASKKV_Q_LENGTHS: src = c->dp.len; break;
    case TASKKV_Q_CLASSES: src = c->dp.cls; break;
    case TASKKV_Q_DIST: src = c->dp.dist; break;
    case TASKKV_Q_CAPACITY: src = c->dp.cap; break;
    case TASKKV_Q_SEMVEC: src = c->dp.sem; break;
    case TASKKV_Q_OFFSETS: src = c->dp.seg_off; break;
    case TASKKV_Q_INDICES: src = c->dp.idx; break;
    case TASKKV_Q_SCORES: src = c->dp.C; break;
    case TASKKV_Q_TOPT: src = c->dp.topt; break;
    case TASKKV_Q_STATUS: src = c->dp.status; break;
    case TASKKV_Q_KPOOL: src = c->dp.k_pool; break;
    case TASKKV_Q_VPOOL: src = c->dp.v_pool; break;
    case TASKKV_Q_PAGETAB: src = c->dp.page_tab; break;
    default: return TASKKV_EINVAL;
  }
  if (cudaDeviceSynchronize() != cudaSuccess) return TASKKV_ECUDA;
  if (need == 0) return TASKKV_OK;
  return cuda_status(cudaMemcpy(host_dst, src, (size_t)need, cudaMemcpyDeviceToHost));
}

taskkv_status taskkv_cache_plan(const taskkv_cache* c, taskkv_plan_info* out) {
  if (!c || !out) return TASKKV_EINVAL;
  *out = c->hp.info;
  return TASKKV_OK;
}

void taskkv_cache_destroy(taskkv_cache* c) {
  if (!c) return;
  if (c->pool) {
    // the pages go back onto the pool's stack once everything that uses them has finished
    cudaDeviceSynchronize();
    if (c->cache_mem && launch_release_pages(c->dp, nullptr) == cudaSuccess) cudaDeviceSynchronize();
    c->pool->free_host += c->pages_held;
    if (--c->pool->caches == 0 && c->pool->orphan) free_pool(c->pool);
  }
  if (c->own_cache || c->own_work || c->stage) cudaDeviceSynchronize();
  if (c->own_cache) cudaFree(c->cache_mem);
  if (c->own_work) cudaFree(c->work_mem);
  if (c->stage) cudaFree(c->stage);
  delete c;
}

const char* taskkv_status_str(taskkv_status s) {
  switch (s) {
    case TASKKV_OK: return "ok";
    case TASKKV_EINVAL: return "invalid argument";
    case TASKKV_EALLOC: return "allocation failed or buffer too small";
    case TASKKV_ECUDA: return "CUDA runtime error";
    case TASKKV_ETIMEOUT: return "device-side wait timed out";
    case TASKKV_ESTATE: return "cache in wrong state";
    default: return "unknown status";
  }
}

int32_t taskkv_hetero_count(int32_t n, float beta, int32_t m, int32_t R, int32_t r) {
  if (n < 0) return 0;
  return hetero_count_impl(n, beta, m, R, r);
}

int32_t taskkv_mid_budget(double budget_tokens, int32_t N, int32_t h_full, int32_t n, int32_t sink,
                          int32_t recent) {
  return mid_budget_impl(budget_tokens, N, h_full, n, sink, recent);
}

int32_t taskkv_mid_budget_ex(double budget_tokens, int32_t N, int32_t f, int32_t n, int32_t sink, int32_t recent,
                             int32_t promote_center, int32_t literal) {
  if (f < 0) f = 0;
  if (f > n) f = n;
  const int32_t h = literal ? f : std::min(n, f + ((promote_center && f < n) ? 1 : 0));
  return taskkv_mid_budget(budget_tokens, N, h, n, sink, recent);
}

int64_t taskkv_launch_count(void) { return g_launches.load(); }

void taskkv_timing_enable(int32_t on) { g_timing.store(on ? 1 : 0); }

int32_t taskkv_timing_collect(int32_t* ids, float* ms, int32_t max) {
  cudaDeviceSynchronize();
  std::lock_guard<std::mutex> lk(g_tmu);
  int32_t n = 0;
  for (auto& r : g_trecs) {
    float t = 0.f;
    cudaEventElapsedTime(&t, r.a, r.b);
    if (ids && ms && n < max) { ids[n] = r.id; ms[n] = t; ++n; }
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  g_trecs.clear();
  return n;
}

const char* taskkv_timing_name(int32_t id) { return (id >= 0 && id < K_COUNT) ? kKernelNames[id] : "?"; }

}  // extern "C"
