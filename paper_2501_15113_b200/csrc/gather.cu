// Data movement of the compacted cache (Sec. IV-B): the retained K and V rows of
// every unit are copied into the unit's pool segment in ascending position
// (full-cache units copy all N rows), and decode-time appends add one row per
// unit.  Rows move as 16-byte vectors.
#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kGatherThreads = 128;   // also the block size of the compensation kernel

// One block copies kGatherRows consecutive segment rows of one unit, K and V.
// Work items are numbered layer-major (gather_off[w], w = (r * B + b) * n_kv + h), so the items of layers
// [layer0, layer0 + n_layers) are the contiguous range [item0, item0 + gridDim.x) and belong to the units
// w0 .. w0 + wn - 1; only those entries of the table are read (later layers may not be planned yet).
// 128 threads and at most 48 registers each: a block then fits beside a resident CTA of the window-score kernel
// (which holds most of an SM's registers and shared memory but leaves HBM bandwidth unused), so that the gather of
// one chunk of layers can run under the window scores of the next.  A block moves its 64 rows in rounds of
// kGatherInFlight 16-byte loads per thread and array, all loads of a round issued before its stores.
constexpr int kGatherInFlight = 4;
template <int ROW_BYTES>
__global__ void __launch_bounds__(kGatherThreads, 10) gather_kernel(DeviceProblem p, int item0, int w0, int wn) {
  constexpr int VPR = ROW_BYTES / 16;                 // vectors (threads) per row
  constexpr int RPP = kGatherThreads / VPR;           // rows per pass
  constexpr int PASSES = kGatherRows / RPP;
  constexpr int ROUND = PASSES < kGatherInFlight ? PASSES : kGatherInFlight;
  static_assert(PASSES % ROUND == 0, "rows per block must be a whole number of rounds");
  __shared__ int s_w;
  grid_dependency_wait();
  const int item = item0 + (int)blockIdx.x;
  if (threadIdx.x < 32) {
    const int wi = w0 + upper_unit_warp(p.gather_off + w0, wn, item, (int)threadIdx.x);
    if (threadIdx.x == 0) s_w = wi;
  }
  __syncthreads();
  const int w = s_w;
  const int u = lm_unit(p, w).u;
  const int len = p.len[u];
  const int N = p.unit_N[u];
  const int r0 = (item - p.gather_off[w]) * kGatherRows;
  const int64_t seg = p.seg_off[u];
  if (p.page_rows == 0 && seg + len > p.pool_rows) return;   // planning overflow, already flagged
  if (r0 >= len) return;                                     // an item between a shard's block end and the next block
  const bool identity = (len == N);
  const int32_t* idx = p.idx + (size_t)u * p.idx_stride;
  const unsigned char* ksrc = static_cast<const unsigned char*>(p.k_ptr[u]);
  const unsigned char* vsrc = static_cast<const unsigned char*>(p.v_ptr[u]);
  // the block's 64 rows are consecutive pool rows (a page holds a multiple of 64 rows), starting at dst0
  const size_t dst0 = pool_row(p, u, seg, r0);
  unsigned char* kdst = static_cast<unsigned char*>(p.k_pool) + dst0 * ROW_BYTES;
  unsigned char* vdst = static_cast<unsigned char*>(p.v_pool) + dst0 * ROW_BYTES;
  const int rr = threadIdx.x / VPR, vc = threadIdx.x % VPR;

  for (int base = 0; base < PASSES; base += ROUND) {
    uint4 kreg[ROUND], vreg[ROUND];
#pragma unroll
    for (int ps = 0; ps < ROUND; ++ps) {
      const int r = r0 + (base + ps) * RPP + rr;
      if (r < len) {
        int src = identity ? r : idx[r];
        src = min(max(src, 0), N - 1);
        kreg[ps] = *reinterpret_cast<const uint4*>(ksrc + (size_t)src * ROW_BYTES + vc * 16);
        vreg[ps] = *reinterpret_cast<const uint4*>(vsrc + (size_t)src * ROW_BYTES + vc * 16);
      }
    }
#pragma unroll
    for (int ps = 0; ps < ROUND; ++ps) {
      const int r = r0 + (base + ps) * RPP + rr;
      if (r < len) {
        *reinterpret_cast<uint4*>(kdst + (size_t)(r - r0) * ROW_BYTES + vc * 16) = kreg[ps];
        *reinterpret_cast<uint4*>(vdst + (size_t)(r - r0) * ROW_BYTES + vc * 16) = vreg[ps];
      }
    }
  }
}

// One warp per unit: the new token's k, v rows go to row len_u of the segment.
template <int ROW_BYTES>
__global__ void __launch_bounds__(256) append_kernel(DeviceProblem p, const unsigned char* k_new,
                                                     const unsigned char* v_new) {
  constexpr int VPR = ROW_BYTES / 16;
  const int vu = blockIdx.x * 8 + (threadIdx.x >> 5);   // view unit: index into k_new, v_new
  const int lane = threadIdx.x & 31;
  if (vu >= p.view_U) return;
  const int u = view_unit(p, vu);
  const int len = p.len[u];
  const int64_t seg = p.seg_off[u];
  bool ok = len < p.cap[u] && (p.page_rows > 0 || seg + len < p.pool_rows);
  if (ok && p.page_rows > 0 && len % p.page_rows == 0) {
    // the row opens a new page: one comes off the pool
    int pg = -1;
    if (lane == 0) {
      const int at = pool_pop(p, 1);
      if (at >= 0) {
        pg = p.pool_free[at];
        p.page_tab[(size_t)u * p.page_stride + len / p.page_rows] = pg;
      }
    }
    pg = __shfl_sync(0xffffffffu, pg, 0);
    ok = pg >= 0;
  }
  __syncwarp();
  if (ok && lane < VPR) {
    const size_t dst = pool_row(p, u, seg, len) * ROW_BYTES + lane * 16;
    const size_t src = (size_t)vu * ROW_BYTES + lane * 16;
    *reinterpret_cast<uint4*>(static_cast<unsigned char*>(p.k_pool) + dst) =
        *reinterpret_cast<const uint4*>(k_new + src);
    *reinterpret_cast<uint4*>(static_cast<unsigned char*>(p.v_pool) + dst) =
        *reinterpret_cast<const uint4*>(v_new + src);
  }
  __syncwarp();
  if (lane == 0) {
    if (ok) p.len[u] = len + 1;
    else set_status(p.status, TASKKV_ESTATE);
  }
}

// "Compressed Cache" of Sec. V-G: rows s1 .. s1 + c - 1 of a non-heterogeneous unit's segment become the
// means of c contiguous groups of the intermediate positions (their first positions are in the index
// table).  One thread per 16-byte column of one compensation row adds the group's rows in position order in
// fp32 and stores the mean in the cache's element type; K and V alike.  Runs after the gather.
template <typename T, int D>
__global__ void __launch_bounds__(kGatherThreads) compensate_kernel(DeviceProblem p, UnitRange ur) {
  constexpr int EPV = 16 / (int)sizeof(T);            // elements per 16-byte vector
  constexpr int VPR = D / EPV;                        // vectors (threads) per row
  constexpr int RPB = kGatherThreads / VPR;           // compensation rows per block
  constexpr int ROW_BYTES = D * (int)sizeof(T);
  const int u = ur.unit(blockIdx.y);
  const int N = p.unit_N[u], len = p.len[u];
  if (len == N) return;                               // the unit kept everything
  const int s1 = p.sink, s2 = p.recent;
  const int c = len - s1 - s2;                        // compensation rows
  const int g = blockIdx.x * RPB + threadIdx.x / VPR;
  if (g >= c) return;
  const int vc = threadIdx.x % VPR;
  const int64_t seg = p.seg_off[u];
  if (p.page_rows == 0 && seg + len > p.pool_rows) return;   // planning overflow, already flagged
  const int32_t* idx = p.idx + (size_t)u * p.idx_stride;
  int j0 = idx[s1 + g];
  int j1 = (g + 1 < c) ? idx[s1 + g + 1] : N - s2;
  j0 = min(max(j0, s1), N - s2);
  j1 = min(max(j1, j0), N - s2);
  const unsigned char* ksrc = static_cast<const unsigned char*>(p.k_ptr[u]) + vc * 16;
  const unsigned char* vsrc = static_cast<const unsigned char*>(p.v_ptr[u]) + vc * 16;
  float ka[EPV], va[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e) { ka[e] = 0.f; va[e] = 0.f; }
  for (int j = j0; j < j1; ++j) {
    float kf[EPV], vf[EPV];
    Vec16<T>::unpack(*reinterpret_cast<const uint4*>(ksrc + (size_t)j * ROW_BYTES), kf);
    Vec16<T>::unpack(*reinterpret_cast<const uint4*>(vsrc + (size_t)j * ROW_BYTES), vf);
#pragma unroll
    for (int e = 0; e < EPV; ++e) { ka[e] += kf[e]; va[e] += vf[e]; }
  }
  const float cnt = (float)max(j1 - j0, 1);
  const size_t drow = pool_row(p, u, seg, s1 + g);
  T* kdst = reinterpret_cast<T*>(static_cast<unsigned char*>(p.k_pool) + drow * ROW_BYTES) + vc * EPV;
  T* vdst = reinterpret_cast<T*>(static_cast<unsigned char*>(p.v_pool) + drow * ROW_BYTES) + vc * EPV;
#pragma unroll
  for (int e = 0; e < EPV; ++e) {
    store_out(kdst + e, ka[e] / cnt);
    store_out(vdst + e, va[e] / cnt);
  }
}

template <typename T, int D>
cudaError_t launch_compensate_typed(const DeviceProblem& p, int max_rows, const UnitRange& ur, cudaStream_t s) {
  constexpr int RPB = kGatherThreads / (D * (int)sizeof(T) / 16);
  const dim3 grid((unsigned)((max_rows + RPB - 1) / RPB), (unsigned)ur.blocks);
  compensate_kernel<T, D><<<grid, kGatherThreads, 0, s>>>(p, ur);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_compensate(const DeviceProblem& p, int dtype, const UnitRange& ur, cudaStream_t s) {
  if (p.max_mid <= 0 || ur.blocks <= 0) return cudaSuccess;
  LaunchScope ls(K_COMPENSATE, s);
  if (dtype == TASKKV_F32)
    return p.d == 64 ? launch_compensate_typed<float, 64>(p, p.max_mid, ur, s)
                     : launch_compensate_typed<float, 128>(p, p.max_mid, ur, s);
  return p.d == 64 ? launch_compensate_typed<__nv_bfloat16, 64>(p, p.max_mid, ur, s)
                   : launch_compensate_typed<__nv_bfloat16, 128>(p, p.max_mid, ur, s);
}

cudaError_t launch_gather(const DeviceProblem& p, int dtype, int batch, int layer0, int n_layers, int64_t item0,
                          int64_t n_items, cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  LaunchScope ls(K_GATHER, s);
  const int row_bytes = p.d * (dtype == TASKKV_F32 ? 4 : 2);
  const unsigned grid = (unsigned)n_items;
  const int first = (int)item0, w0 = layer0 * batch * p.n_kv, wn = n_layers * batch * p.n_kv;
  switch (row_bytes) {
    case 128: return launch_dependent(gather_kernel<128>, grid, (unsigned)kGatherThreads, s, p, first, w0, wn);
    case 256: return launch_dependent(gather_kernel<256>, grid, (unsigned)kGatherThreads, s, p, first, w0, wn);
    case 512: return launch_dependent(gather_kernel<512>, grid, (unsigned)kGatherThreads, s, p, first, w0, wn);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_append(const DeviceProblem& p, int dtype, const void* k_new, const void* v_new,
                          cudaStream_t s) {
  LaunchScope ls(K_APPEND, s);
  const int row_bytes = p.d * (dtype == TASKKV_F32 ? 4 : 2);
  const unsigned grid = (unsigned)((p.view_U + 7) / 8);
  const unsigned char* kn = static_cast<const unsigned char*>(k_new);
  const unsigned char* vn = static_cast<const unsigned char*>(v_new);
  switch (row_bytes) {
    case 128: append_kernel<128><<<grid, 256, 0, s>>>(p, kn, vn); break;
    case 256: append_kernel<256><<<grid, 256, 0, s>>>(p, kn, vn); break;
    case 512: append_kernel<512><<<grid, 256, 0, s>>>(p, kn, vn); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace taskkv
