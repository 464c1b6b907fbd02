/*
 * taskkv.h -- C ABI of the Task-KV hot path for NVIDIA B200 (sm_100a).
 *
 * Task-KV (arXiv 2501.15113) compresses a transformer's KV cache per attention
 * head after prefill and then decodes over the compacted, ragged cache:
 *
 *   prefill side (Sec. IV-A, IV-B)
 *     window scores      C  = mean over the observation window's softmax rows   (Eq. 12, 13)
 *     semantic vector    v' = sum over the top-t positions of C[j] V[j,:]       (Eq. 14, 15)
 *     semantic separator center = mean of the layer's v' (Eq. 8), distance =
 *                        L2 norm of the offset (Eq. 7), the f(r) farthest heads
 *                        are heterogeneous (Eq. 16), the closest remaining head
 *                        joins them                                             (Sec. IV-A)
 *     allocation         heterogeneous heads keep every position; the others keep
 *                        sinks + recent + the k middle positions of highest
 *                        pooled score                                           (Sec. IV-B, V-D, Eq. 17)
 *     gather             retained K/V rows copied into one segment per KV head
 *   decode side
 *     append             the new token's k, v join every head's segment
 *     attention          softmax(q K^T / sqrt(d)) V over each head's segment    (Eq. 1)
 *
 * Every step runs in CUDA kernels; the library has no CPU fallback.  All calls
 * return a status code and never throw or abort.  Unless stated otherwise a
 * pointer is a DEVICE pointer, 16-byte aligned, and work is enqueued on the
 * caller's stream without synchronising.  "Host" arrays are read before the
 * call returns and may be freed afterwards.
 *
 * A "unit" is one (sequence b, layer r, KV head h); units are numbered
 * u = (b * n_layers + r) * n_kv_heads + h.  With grouped-query attention the
 * G = n_heads / n_kv_heads query heads a = h*G .. h*G+G-1 share unit h, and
 * heads are classified per KV head (one semantic vector per KV head, from the
 * mean of the group's G*L window rows).
 */
#ifndef TASKKV_H_
#define TASKKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t taskkv_status;
#define TASKKV_OK        0
#define TASKKV_EINVAL   (-1)  /* bad argument; nothing was launched */
#define TASKKV_EALLOC   (-2)  /* device or host allocation failed, or a caller buffer is too small */
#define TASKKV_ECUDA    (-3)  /* a CUDA runtime call failed */
#define TASKKV_ETIMEOUT (-4)  /* a bounded device-side wait ran out */
#define TASKKV_ESTATE   (-5)  /* cache in a wrong state (e.g. append beyond capacity) */

#define TASKKV_F32  0
#define TASKKV_BF16 1

#define TASKKV_CLASS_NON_HETERO 0
#define TASKKV_CLASS_HETERO     1
#define TASKKV_CLASS_CENTER     2   /* the head closest to the center, promoted to a full cache */

/* The information-compensation methods compared in Sec. V-G, at equal cache size (mid_budget rows):
 *   SELECT  the middle activations of Sec. IV-B (the method itself; default)
 *   RECENT  "No Cache": the budget goes to the recent window, nothing is kept from the middle
 *   MEAN    "Compressed Cache": the intermediate positions [s1, N - s2) are cut into mid_budget contiguous
 *           groups of near-equal size (group g starts at s1 + floor(g * M / mid_budget), M = N - s1 - s2) and
 *           each group is replaced by one compensation row, the mean of its K rows resp. V rows (fp32
 *           accumulation in position order, stored in the cache's element type).  In the retained-index
 *           table a compensation row is listed with the first position of its group.
 * Classes, lengths, capacities and every buffer size are the same under all three. */
#define TASKKV_MID_SELECT 0
#define TASKKV_MID_RECENT 1
#define TASKKV_MID_MEAN   2

#define TASKKV_MAX_TOP_T       1024
#define TASKKV_MAX_KV_HEADS    64
#define TASKKV_MAX_WINDOW_ROWS 128  /* G * window */

typedef struct taskkv_cache taskkv_cache;   /* opaque; owns pools, lengths, indices, statistics */
typedef void* taskkv_stream;                /* a cudaStream_t */

/* Problem statement of Sec. IV.  Pointers inside are HOST arrays. */
typedef struct taskkv_params {
  int32_t n_layers;      /* R */
  int32_t n_heads;       /* query heads n */
  int32_t n_kv_heads;    /* n_kv; n_heads % n_kv_heads == 0, <= TASKKV_MAX_KV_HEADS */
  int32_t head_dim;      /* d: 64 or 128 */
  int32_t batch;         /* number of sequences */
  int32_t sink;          /* s1: leading positions every head keeps (Sec. IV-B) */
  int32_t recent;        /* s2: trailing positions every head keeps */
  int32_t mid_budget;    /* k: middle activations per non-heterogeneous head (Eq. 17) */
  int32_t window;        /* L: observation window (Eq. 12); G*L <= TASKKV_MAX_WINDOW_ROWS, L <= min N_b */
  int32_t top_t;         /* t of Eq. 14 (256 in Sec. V-D); <= TASKKV_MAX_TOP_T */
  int32_t pool_kernel;   /* average-pooling kernel of Sec. V-D (7), odd, <= 31; 1 = off */
  int32_t m_top;         /* m of Eq. 16 */
  float   beta;          /* beta of Eq. 16 */
  int32_t promote_center;    /* 1: the closest remaining head also keeps a full cache (Sec. IV-A) */
  int32_t force_class;       /* -1: run the separator; 1: every head heterogeneous; 0: none */
  int32_t dtype;             /* TASKKV_F32 or TASKKV_BF16: element type of q, k, v, out and the pools */
  int32_t max_new_tokens;    /* rows reserved per unit for taskkv_append */
  int32_t mid_policy;        /* TASKKV_MID_*: what a non-heterogeneous head keeps beside sinks and recent window */
  const int32_t* seq_lens;   /* host [batch]: N_b (ragged batches allowed) */
  const int32_t* mid_budget_per_layer;  /* host [n_layers] or NULL; overrides mid_budget */
  const int32_t* n_hetero;   /* host [batch][n_layers] or NULL; overrides Eq. 16 */
  float   budget_frac;       /* 0: mid_budget (or mid_budget_per_layer) is used as given.  In (0, 1]: the KV budget of
                                Sec. IV-B as a fraction of the full cache; every (sequence, layer) then gets the middle
                                budget of Eq. 17, k = floor((B - N h) / (n - h)) - s1 - s2 with B = fraction * n_kv * N_b
                                and h the heads of that layer that keep everything, computed on the device (and, for
                                the exact sizing of the pools, by the same formula on the host) */
  int32_t shard_kv_heads;    /* 0: the problem holds every KV head of the model.  > 0: head sharding -- the model has this
                                many KV heads per layer and this problem holds n_kv_heads of them, starting at shard_first
                                (and their query heads); see taskkv_compress_shard_begin */
  int32_t shard_first;
} taskkv_params;

typedef struct taskkv_plan_info {
  int64_t n_units;
  int64_t pool_rows;         /* rows of K (and of V) in the compacted pools, reserve included */
  int64_t retained_rows;     /* rows kept right after compression */
  int64_t cache_bytes;       /* persistent device memory of one cache */
  int64_t workspace_bytes;   /* device memory needed only while taskkv_compress_ex runs on the stream */
  int64_t max_decode_items;  /* split-K work items of one decode call at full capacity */
  int64_t gather_items;      /* row blocks the gather step copies */
  int64_t index_stride;      /* ints per unit of the retained-index table */
} taskkv_plan_info;

/* Fills the defaults of Sec. V-D: top_t 256, pool_kernel 7, sink 16, recent 256,
 * window 32, beta 0.25 / m 4, promote_center 1, force_class -1, dtype bf16. */
void taskkv_params_default(taskkv_params* p);

/* Host only.  Validates p and sizes every buffer.  The number of full-cache
 * heads per layer is fixed by Eq. 16 (only WHICH heads is data dependent), so
 * pool sizes are exact before any kernel runs. */
taskkv_status taskkv_plan(const taskkv_params* p, taskkv_plan_info* out);

/*
 * Prefill-side compression of every layer of every sequence (Sec. IV-A, IV-B).
 *   q_win[b]  device [n_layers][n_heads][L][d]      the last L query rows, Q[-L:,:] of Eq. 12
 *   k[b],v[b] device [n_layers][n_kv_heads][N_b][d] post-RoPE keys / values as a model caches them
 *   q_win, k, v themselves are host arrays of `batch` device pointers.
 *   cache_mem / workspace_mem: device buffers of at least the planned sizes, 256-byte
 *   aligned, owned by the caller; NULL lets the library allocate (cudaMalloc) and
 *   own them.  The workspace may be released once the stream has passed this
 *   call; the cache memory must outlive the cache.  K and V are copied, never
 *   aliased: the caller may free them once the stream has passed this call.
 * On success *out_cache holds the compacted cache: per unit a segment of
 * retained rows in ascending position, its length, class, distance and
 * semantic vector.  Errors: EINVAL (arguments), EALLOC, ECUDA.
 * Streams: all work is ordered after what `stream` holds at the call and is
 * complete, for every later operation on `stream`, when the call's last kernel is.
 * For large bf16 problems the steps of different chunks of layers overlap on
 * streams the library owns (with 32 window rows the selection of one chunk
 * beside the window scores of the next; with more window rows the gather of
 * one chunk beside window scores and selection of the next; two streams per
 * device, created by the first such call: make that call before capturing
 * `stream` into a graph); they are forked from and joined back into `stream`
 * with events, and calls that use them are serialised on the host.
 */
taskkv_status taskkv_compress_ex(const taskkv_params* p, const void* const* q_win,
                                 const void* const* k, const void* const* v,
                                 void* cache_mem, size_t cache_bytes,
                                 void* workspace_mem, size_t workspace_bytes,
                                 taskkv_stream stream, taskkv_cache** out_cache);

/*
 * The exact semantic vectors of Sec. III-A (Eq. 1-2) of one sequence: for every KV head
 *   C[j] = (1 / (G N)) sum over the G query heads of the group and all N query rows i of A[i, j],
 *          A = softmax(Q K^T / sqrt(d) + causal mask) row by row (G = 1: exactly the column mean of Eq. 2),
 *   v    = sum_j C[j] V[j, :],
 * i.e. what the observation window, the top-t selection and Eq. 15 approximate.  The cost is quadratic in N (two
 * tensor-core passes over the causal half of Q K^T); this is an analysis routine beside the compression path.
 *   q        device bf16 [n_layers][n_heads][N][d]     every query row (post-RoPE), 16-byte aligned
 *   k, v     device bf16 [n_layers][n_kv_heads][N][d]
 *   sem_out  device fp32 [n_layers][n_kv_heads][d]     v
 *   c_out    device fp32 [n_layers][n_kv_heads][N], or NULL if the column means are not wanted
 *   workspace_mem  device scratch, 256-byte aligned, owned by the caller, or NULL: then up to ~1.5 GB come from the
 *            stream's memory pool (cudaMallocAsync) and go back to it, which can cost more than the kernels.
 *            taskkv_exact_semantic_bytes gives the size with which all heads (or as many as fit 1.5 GB) go through
 *            in one batch; with less, fewer heads go per batch; EALLOC if not even one KV group fits.
 * head_dim 64 or 128, bf16 only.  The call returns after the stream has finished the work.
 * Errors: EINVAL (arguments), EALLOC, ECUDA, ETIMEOUT (a bounded wait inside a kernel ran out).
 */
taskkv_status taskkv_exact_semantic(const void* q, const void* k, const void* v, int32_t n_layers, int32_t n_heads,
                                    int32_t n_kv_heads, int32_t head_dim, int32_t seq_len, float* sem_out,
                                    float* c_out, void* workspace_mem, size_t workspace_bytes, taskkv_stream stream);
/* Scratch size for taskkv_exact_semantic (host only; 0 for arguments it would reject). */
size_t taskkv_exact_semantic_bytes(int32_t n_layers, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                   int32_t seq_len);

/* As taskkv_compress_ex, for callers that already hold the normalisers of the observation window's rows:
 *   window_lse[b]  device fp32 [n_layers][n_heads][L], lse_i = ln sum_j exp(q_i . k_j / sqrt(d)) over the keys
 *                  j <= position of window row i -- what an attention kernel run over the prompt returns as the
 *                  log-sum-exp of its last L query rows.
 * With them A'[i, j] = exp(s_ij - lse_i) (Eq. 12) needs no pass over K for the row sums, so the window scores
 * read K once instead of twice.  Results equal those of taskkv_compress_ex up to the rounding of the supplied
 * values.  window_lse itself is a host array of `batch` device pointers. */
taskkv_status taskkv_compress_lse(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                  const void* const* v, const void* const* window_lse,
                                  void* cache_mem, size_t cache_bytes,
                                  void* workspace_mem, size_t workspace_bytes,
                                  taskkv_stream stream, taskkv_cache** out_cache);

/* Layer at a time, into ONE cache.  Nothing couples the layers of a sequence except the schedules of Eq. 16 /
 * Eq. 17, which are known before any data, and Eq. 16 also fixes how many heads of a layer keep everything, so
 * the place of every layer's segments in the pools is known in advance.  A prefill loop can therefore create the
 * cache first and compress layer r as soon as its K and V exist, then free them:
 *   taskkv_cache_create    plans the whole problem (all layers, all sequences), takes or allocates cache and
 *                          workspace memory exactly as taskkv_compress_ex does, uploads the tables and zeroes the
 *                          state: every unit has length 0 until its layer is compressed.
 *   taskkv_compress_layer  steps a1-a5 for layer `layer` of every sequence:
 *                            q_win[b]  device [n_heads][L][d]       the layer's last L query rows
 *                            k[b],v[b] device [n_kv_heads][N_b][d]  the layer's keys / values
 *                            window_lse[b] device fp32 [n_heads][L] or window_lse == NULL (see taskkv_compress_lse)
 *                          Each layer may be compressed once (ESTATE otherwise), in any order.  Calls for different
 *                          layers work on disjoint parts of the cache and of the workspace, so they may be issued on
 *                          different streams (each ordered after taskkv_cache_create) and then overlap on the GPU;
 *                          host-side the calls on one cache are not re-entrant.  Classes, lengths, retained
 *                          positions, cache rows, segment offsets and work lists are bit for bit those the all-layer
 *                          call produces; once every layer is in, the cache is the same object, and
 *                          taskkv_decode_step and the other decode calls work on it as usual (a layer-range decode
 *                          may already run on layers that are in).
 * Errors: EINVAL (arguments, layer out of range, cache without workspace), ESTATE, ECUDA. */
taskkv_status taskkv_cache_create(const taskkv_params* p, void* cache_mem, size_t cache_bytes,
                                  void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                                  taskkv_cache** out_cache);
taskkv_status taskkv_compress_layer(taskkv_cache* c, int32_t layer, const void* const* q_win,
                                    const void* const* k, const void* const* v, const void* const* window_lse,
                                    taskkv_stream stream);

/* Head sharding (tensor-parallel style): every rank holds some KV heads of every layer.  Window scores, top-t and
 * semantic vectors (Eq. 12-15) are per head; the center of Eq. 8 and the ranking of Sec. IV-A are over ALL heads of a
 * layer; allocation, gather and decode are per head again.  So a rank runs
 *   taskkv_compress_shard_begin   steps a1-a2 for its heads (params with shard_kv_heads > 0; n_heads, n_kv_heads and the
 *                                 q_win / k / v tensors are the rank's own; Eq. 16, Eq. 17 and an n_hetero override
 *                                 count over the model's shard_kv_heads heads),
 *   taskkv_cache_semantic         device pointer to its vectors, fp32 [batch][n_layers][n_kv_heads][d] -- the ranks
 *                                 all-gather these into [batch][n_layers][shard_kv_heads][d] in head order (any
 *                                 collective; into this GPU's own memory),
 *   taskkv_compress_shard_finish  separator over the gathered vectors (every rank computes every head's class and keeps
 *                                 its own), plan and gather for its heads.
 * Which rank the layer's full-cache heads land on is data dependent, so a shard's pools are sized for the most it can
 * get, min(full heads of the layer, n_kv_heads) per (sequence, layer): pool_rows, retained_rows and cache_bytes of
 * taskkv_plan are then upper bounds, and the lengths tell what is used.  Classes, lengths, retained positions, cache
 * rows and decode outputs of a head are those of the unsharded problem.  The decode calls work on a shard's cache as on
 * any other.  finish without begin, or begin's cache used before finish, is ESTATE / undefined lengths of 0. */
taskkv_status taskkv_compress_shard_begin(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                          const void* const* v, const void* const* window_lse,
                                          void* cache_mem, size_t cache_bytes, void* workspace_mem,
                                          size_t workspace_bytes, taskkv_stream stream, taskkv_cache** out_cache);
taskkv_status taskkv_cache_semantic(const taskkv_cache* c, const float** device_ptr, int64_t* n_floats);
taskkv_status taskkv_compress_shard_finish(taskkv_cache* c, const float* sem_all, taskkv_stream stream);

/* Paged cache (block tables), for serving.  Per-head caches of different and growing lengths fragment memory when
 * every batch owns contiguous pools with a reserve per unit; here the K and V rows of every cache live in pages of
 * page_rows rows taken from one pool, each unit has a table of its pages, pages for appended tokens are taken when a
 * unit's last page is full, and destroying a cache returns its pages for the next one.
 *   taskkv_pool_create    a pool of n_pages pages of page_rows rows (a multiple of 64) of head_dim elements of
 *                         `dtype`, for K and for V, in `mem` (device, 256-byte aligned, at least
 *                         taskkv_pool_bytes(...) bytes, owned by the caller) or, with mem == NULL, in memory the
 *                         library allocates.  Layout of that memory: the K pages [n_pages][page_rows][head_dim],
 *                         the V pages likewise from the next multiple of 256 bytes, then the library's list of
 *                         free pages.
 *   taskkv_compress_paged as taskkv_compress_ex, with the compacted rows going to pages of `pool`; cache_mem then
 *                         holds only tables (taskkv_plan_paged gives the sizes and the pages the compression takes).
 *                         max_new_tokens still bounds how far a unit may grow (it sizes the page tables and the
 *                         decode work lists) but reserves no rows.
 * Every other call (append, decode, decode_step, layer ranges, queries, destroy) works on a paged cache as on any
 * other; results are bit for bit those of the contiguous layout.  The library keeps count of the pool's free pages on
 * the host (how many pages a call takes follows from the schedules, not from the data) and refuses a compression or an
 * append that would not fit with EALLOC before anything is launched.  Calls that use one pool -- compressions,
 * appends and decode steps of its caches, and their destruction -- must be ordered with respect to one another by the
 * caller (one stream, or events).  taskkv_pool_destroy on a pool that still has caches only marks it: the last of
 * its caches to be destroyed releases it (caller-supplied pool memory must stay valid until then).
 * The count follows the calls the library sees: an append or a fused step replayed from a captured CUDA graph takes
 * its pages on the device without the count knowing, so replay only calls that append nothing (taskkv_decode_ex) on
 * a paged cache, or none.
 * A paged cache cannot be head-sharded or filled layer by layer (EINVAL).
 * Should the device find the pool empty all the same (calls on one pool that the caller did not order), the
 * row is not stored and the cache's status word gets ESTATE; such a cache is to be destroyed, which returns the pages
 * it verifiably holds and never writes outside the pool's list. */
typedef struct taskkv_pool taskkv_pool;
size_t        taskkv_pool_bytes(int32_t page_rows, int32_t n_pages, int32_t head_dim, int32_t dtype);
taskkv_status taskkv_pool_create(int32_t page_rows, int32_t n_pages, int32_t head_dim, int32_t dtype, void* mem,
                                 size_t bytes, taskkv_stream stream, taskkv_pool** out_pool);
int32_t       taskkv_pool_free_pages(const taskkv_pool* pool);      /* the host's count; -1 for a NULL pool */
void          taskkv_pool_destroy(taskkv_pool* pool);
taskkv_status taskkv_plan_paged(const taskkv_params* p, int32_t page_rows, taskkv_plan_info* out, int64_t* pages_needed);
taskkv_status taskkv_compress_paged(const taskkv_params* p, const void* const* q_win, const void* const* k,
                                    const void* const* v, taskkv_pool* pool, void* cache_mem, size_t cache_bytes,
                                    void* workspace_mem, size_t workspace_bytes, taskkv_stream stream,
                                    taskkv_cache** out_cache);

/* The flat form of the same call: one bf16 sequence, Sec. V-D defaults for
 * everything not listed, library-owned memory, max_new_tokens = 4096. */
taskkv_status taskkv_compress(const void* q_win, const void* k, const void* v,
                              int32_t n_layers, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                              int32_t seq_len, int32_t sink, int32_t recent, int32_t mid_budget,
                              int32_t window, taskkv_stream stream, taskkv_cache** out_cache);

/* As taskkv_compress_ex, but q_win[b], k[b], v[b] are HOST buffers (pinned
 * memory gives asynchronous copies).  Layers are staged through device
 * buffers the library allocates, so the host-to-device copies are part of the
 * call.  Cache memory is library-owned.  The call synchronises the stream and
 * then reads the cache's sticky device status: if a kernel recorded an error
 * (ETIMEOUT) the cache is destroyed, *out_cache is NULL and that code is returned. */
taskkv_status taskkv_compress_host(const taskkv_params* p, const void* const* q_win,
                                   const void* const* k, const void* const* v,
                                   taskkv_stream stream, taskkv_cache** out_cache);

/* Decode-time growth: writes k_new, v_new [batch][n_layers][n_kv_heads][d] at
 * row len_u of every unit and increments len_u.  A unit already at capacity is
 * left unchanged and the cache's sticky status becomes ESTATE. */
taskkv_status taskkv_append(taskkv_cache* c, const void* k_new, const void* v_new, taskkv_stream stream);

/* Decode attention (Eq. 1, one query row per head, no mask) over the ragged
 * cache: q, out [batch][n_layers][n_heads][d] in the cache's dtype, fp32
 * accumulation.  lengths: device int32 [n_units] to attend over a prefix of
 * each segment, or NULL for the cache's own lengths. */
taskkv_status taskkv_decode(const void* q, taskkv_cache* c, const int32_t* lengths, void* out,
                            taskkv_stream stream);

/* The same two calls for layers [layer_begin, layer_begin + layer_count) of every
 * sequence -- what a model's decode loop needs, since layer r's query exists only
 * after layer r-1 has run (Eq. 1 is applied layer by layer).  k_new, v_new are
 * [batch][layer_count][n_kv_heads][d], q and out [batch][layer_count][n_heads][d],
 * lengths (optional) [batch][layer_count][n_kv_heads]; results are identical to the
 * corresponding slices of the all-layer calls.  Calls on one cache share its
 * split-K work buffers: issue them on one stream (or order them yourself).
 * EINVAL if the range leaves [0, n_layers). */
taskkv_status taskkv_append_ex(taskkv_cache* c, const void* k_new, const void* v_new,
                               int32_t layer_begin, int32_t layer_count, taskkv_stream stream);
taskkv_status taskkv_decode_ex(const void* q, taskkv_cache* c, const int32_t* lengths, void* out,
                               int32_t layer_begin, int32_t layer_count, taskkv_stream stream);

/* One decode step in one call: taskkv_append_ex followed by taskkv_decode_ex on the same layers, fused -- the new
 * token's k, v rows are read by the attention kernel straight from k_new, v_new (and stored in the segments by
 * it), and the lengths are raised by its combine pass; outputs, cache rows and lengths afterwards are those of
 * the two separate calls, bit for bit.  A unit already at capacity attends over its existing rows only and
 * the sticky status becomes ESTATE.  taskkv_decode_step covers every layer. */
taskkv_status taskkv_decode_step_ex(const void* q, const void* k_new, const void* v_new, taskkv_cache* c,
                                    void* out, int32_t layer_begin, int32_t layer_count, taskkv_stream stream);
taskkv_status taskkv_decode_step(const void* q, const void* k_new, const void* v_new, taskkv_cache* c,
                                 void* out, taskkv_stream stream);

/* One decode step with HOST buffers: copies q, k_new, v_new in, appends,
 * attends and copies out back (k_new and v_new may both be NULL to skip the
 * append).  Synchronises the stream before returning, and returns the cache's
 * sticky device status if it is not TASKKV_OK (ESTATE: a unit was already at
 * capacity, its row was not appended, `out` is still the attention over the
 * rows it holds; ETIMEOUT: a bounded device-side wait ran out). */
taskkv_status taskkv_decode_host(const void* q, const void* k_new, const void* v_new, taskkv_cache* c,
                                 void* out, taskkv_stream stream);

/* Decode attention without any allocation.  (The paper has no counterpart to
 * this call; it exists for deployment.)  Some callers may not allocate device
 * memory: code running inside a serving engine that has already given all
 * device memory to its own pool, or a latency-critical decode loop in which
 * the device-wide synchronisation of cudaMalloc / cudaFree is unacceptable.
 * This call computes the same result as taskkv_decode over caller-held pools,
 * with its split-K scratch in a fixed 32 MiB device array that is part of the
 * library image (every GPU that loads the library holds it until the process
 * exits).  It calls no cudaMalloc, cudaFree or other allocating routine.
 *   q, out    [n_units * group][head_dim] in `dtype`; unit u serves query heads u*group .. u*group+group-1
 *   k_pool, v_pool   rows of head_dim elements; unit u owns rows seg_off[u] .. seg_off[u] + lengths[u] - 1
 *   seg_off   device int64 [n_units];  lengths  device int32 [n_units]
 *   max_len   host-side upper bound of every lengths[u] (sets the work split); a unit whose length is larger
 *             attends over its first max_len rows only (the length is clamped, never read past)
 * Limits: group in {1,2,4,8}, head_dim in {64,128}, and
 * n_units * group * (head_dim + 2) * 4 bytes must fit the 32 MiB scratch;
 * beyond that the call returns TASKKV_EINVAL (with a line on stderr) and
 * launches nothing.
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call before starting any stream capture.
 * All calls share the one array and it keeps the previous call's contents
 * (every slot a call reads is first rewritten by that call): calls whose
 * kernels may overlap on the GPU - different streams or host threads - race
 * and must be serialised by the caller. */
taskkv_status taskkv_decode_noalloc(const void* q, const void* k_pool, const void* v_pool,
                                    const int64_t* seg_off, const int32_t* lengths, int32_t n_units,
                                    int32_t group, int32_t head_dim, int32_t dtype, int32_t max_len,
                                    void* out, taskkv_stream stream);

/* Synchronising device-to-host reads for tests and reports. */
#define TASKKV_Q_LENGTHS   0   /* int32 [n_units] */
#define TASKKV_Q_CLASSES   1   /* int32 [n_units] */
#define TASKKV_Q_DIST      2   /* float [n_units]: distance to the layer's center */
#define TASKKV_Q_SEMVEC    3   /* float [n_units][d]: semantic vectors v' */
#define TASKKV_Q_OFFSETS   4   /* int64 [n_units+1]: first pool row of each segment */
#define TASKKV_Q_INDICES   5   /* int32 [n_units][index_stride]: retained positions of class-0 units */
#define TASKKV_Q_SCORES    6   /* float, units concatenated: C (valid while the workspace is intact) */
#define TASKKV_Q_TOPT      7   /* int32 [n_units][top_t]: I of Eq. 14, ascending, -1 padded (workspace) */
#define TASKKV_Q_STATUS    8   /* int32 [1]: sticky device status word */
#define TASKKV_Q_KPOOL     9   /* raw K pool bytes */
#define TASKKV_Q_VPOOL    10   /* raw V pool bytes */
#define TASKKV_Q_CAPACITY 11   /* int32 [n_units] */
#define TASKKV_Q_PAGETAB  12   /* int32 [n_units][page_stride]: page ids of each unit's rows, in order (paged caches);
                                  with it TASKKV_Q_KPOOL / TASKKV_Q_VPOOL return the pool's pages */
int64_t       taskkv_cache_query_bytes(const taskkv_cache* c, int32_t what);
taskkv_status taskkv_cache_query(const taskkv_cache* c, int32_t what, void* host_dst, size_t bytes);
taskkv_status taskkv_cache_plan(const taskkv_cache* c, taskkv_plan_info* out);
/* Frees what the library owns of the cache (synchronising the device first if that is device memory).  A paged
 * cache gives its pages back to the pool: the call waits for the device, pushes them onto the pool's free list and
 * waits again, so that the next call on the pool may take them.  NULL is accepted. */
void          taskkv_cache_destroy(taskkv_cache* c);

const char*   taskkv_status_str(taskkv_status s);

/* Eq. 16, f(r) = n*beta - (n*beta - m)/(R-1)*r, rounded half up and clamped to
 * [0, n]; a single layer gives n*beta.  Host only. */
int32_t taskkv_hetero_count(int32_t n, float beta, int32_t m, int32_t R, int32_t r);

/* Eq. 17, k = (B - N*h)/(n - h) - s1 - s2 with h the number of full-cache heads
 * of the layer, the quotient floored, clamped to [0, N - s1 - s2].  Host only. */
int32_t taskkv_mid_budget(double budget_tokens, int32_t N, int32_t h_full, int32_t n,
                          int32_t sink, int32_t recent);

/* Eq. 17 from Eq. 16's head count f = f(r).  literal = 0: h = f plus the promoted closest head (if promote_center
 * and f < n), i.e. the heads that really keep a full cache, so the layer total stays within the budget;
 * literal = 1: h = f, Eq. 17 exactly as printed.  Host only. */
int32_t taskkv_mid_budget_ex(double budget_tokens, int32_t N, int32_t f, int32_t n, int32_t sink, int32_t recent,
                             int32_t promote_center, int32_t literal);

/* Self-test of the bounded device-side waits (no counterpart in the paper).  The tensor-core kernels wait on
 * shared-memory barriers with an iteration limit; when a wait runs out the block raises an abort flag, every other
 * wait of the block returns at once, and the kernel records TASKKV_ETIMEOUT in its status word and exits normally.
 * This call runs that wait, in a one-block kernel with nothing else in flight, on a barrier that nobody completes,
 * with a limit of `max_polls` polls (clamped to [1, 65536]; a few milliseconds at most), then a second wait that
 * must return at once because of the abort flag.  Synchronises `stream`.  Returns TASKKV_ETIMEOUT when the wait
 * gave up as designed (the expected result), TASKKV_OK if it did not, TASKKV_ECUDA on a runtime error;
 * *polls_out (host, optional) receives the polls the first wait made. */
taskkv_status taskkv_selftest_bounded_wait(int32_t max_polls, int32_t* polls_out, taskkv_stream stream);

/* Kernel launches issued by this library in this process so far. */
int64_t taskkv_launch_count(void);

/* Optional per-kernel timing: when enabled every launch is bracketed by CUDA
 * events on its stream.  taskkv_timing_collect synchronises the device, then
 * writes up to `max` records as (kernel id, milliseconds) pairs and clears the
 * log; returns the number written.  Names: taskkv_timing_name(id). */
void        taskkv_timing_enable(int32_t on);
int32_t     taskkv_timing_collect(int32_t* ids, float* ms, int32_t max);
const char* taskkv_timing_name(int32_t id);

#ifdef __cplusplus
}
#endif
#endif  /* TASKKV_H_ */
