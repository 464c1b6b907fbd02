// The exact semantic vector of Sec. III-A (Eq. 1-2): v = (sum_i A[i,:] / N) V with the full N x N causal attention
// matrix A of a head -- the quantity that the observation window (Eq. 12-15) approximates.  Quadratic in N: an
// analysis routine (how far is v' from v, do the two rank the heads alike), not part of the compression path.
//
// The column sums come from the tensor-core window-score kernel in prefix mode: the N query rows of a head are cut
// into blocks of 128; block b is a 128-row window over the first 128 (b + 1) keys, whose two passes (row
// normalisers, then scores) give C_b[j] = (1/128) sum_{i in block b} A[i, j].  Then
//   C[j] = 128 / (G N) * sum over the G query heads of the KV head, and over the blocks b >= j / 128, of C_b[j]
//   v    = sum_j C[j] V[j, :]
// with fixed summation orders.  K of a head (N d 2 bytes) is re-read once per block and stays in L2 meanwhile.
#include <algorithm>

#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kBlockRows = 128;        // query rows per prefix window
constexpr int kSliceKeys = 512;        // keys per partial sum of v

// offset of block b's scores inside a head's area: blocks 0 .. b-1 hold 128, 256, ... floats
__host__ __device__ inline int64_t block_off(int64_t b) { return 64 * b * (b + 1); }

__global__ void exact_init_kernel(int32_t* unit_N, int64_t* c_off, int U, int nb) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u > U) return;
  const int head = u / nb, b = u % nb;
  c_off[u] = (int64_t)head * block_off(nb) + block_off(b);
  if (u < U) unit_N[u] = (b + 1) * kBlockRows;
}

// One thread per key j of a KV head: the blocks' scores added in ascending (query head, block) order.
__global__ void __launch_bounds__(256) exact_colsum_kernel(const float* __restrict__ Cb, int nb, int G, int N,
                                                           float* __restrict__ c_full) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int kvh = blockIdx.y;
  if (j >= N) return;
  float s = 0.f;
  for (int g = 0; g < G; ++g) {
    const float* head = Cb + (int64_t)(kvh * G + g) * block_off(nb);
    for (int b = j / kBlockRows; b < nb; ++b) s += head[block_off(b) + j];
  }
  c_full[(int64_t)kvh * N + j] = s * ((float)kBlockRows / ((float)G * (float)N));
}

// partial[kvh][slice][c] = sum over the slice's keys, ascending, of C[j] V[j, c]
template <int D>
__global__ void __launch_bounds__(D) exact_semvec_partial_kernel(const float* __restrict__ c_full,
                                                                 const __nv_bfloat16* __restrict__ V, int N, int slices,
                                                                 float* __restrict__ partial) {
  const int kvh = blockIdx.y, sl = blockIdx.x, c = threadIdx.x;
  const int j0 = sl * kSliceKeys, j1 = min(N, j0 + kSliceKeys);
  const float* w = c_full + (int64_t)kvh * N;
  const __nv_bfloat16* v = V + (int64_t)kvh * N * D + c;
  float acc = 0.f;
  for (int j = j0; j < j1; ++j) acc = fmaf(w[j], __bfloat162float(v[(int64_t)j * D]), acc);
  partial[((int64_t)kvh * slices + sl) * D + c] = acc;
}

template <int D>
__global__ void __launch_bounds__(D) exact_semvec_final_kernel(const float* __restrict__ partial, int slices,
                                                               float* __restrict__ sem) {
  const int kvh = blockIdx.x, c = threadIdx.x;
  float acc = 0.f;
  for (int sl = 0; sl < slices; ++sl) acc += partial[((int64_t)kvh * slices + sl) * D + c];
  sem[(int64_t)kvh * D + c] = acc;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

}  // namespace taskkv

using namespace taskkv;

namespace {

struct ExactLayout {
  size_t o_status, o_unit_N, o_c_off, o_Cb, o_spart, o_stat, o_cfull, o_part, total;
};
// Scratch for batches of hb query heads (a multiple of G).
ExactLayout exact_layout(int64_t hb, int nb, int chunks, int G, int N, int d, int slices, bool own_scores) {
  ExactLayout l;
  const int64_t U = hb * nb;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
  l.o_status = take(64);
  l.o_unit_N = take((size_t)U * 4);
  l.o_c_off = take((size_t)(U + 1) * 8);
  l.o_Cb = take((size_t)hb * block_off(nb) * 4);
  l.o_spart = take((size_t)U * chunks * 2 * kBlockRows * 8);
  l.o_stat = take((size_t)U * 2 * kBlockRows * 4);
  l.o_cfull = take(own_scores ? (size_t)(hb / G) * N * 4 : 0);
  l.o_part = take((size_t)(hb / G) * slices * d * 4);
  l.total = o;
  return l;
}

struct ExactShape {
  int N, d, G, nb, chunks, slices;
  int64_t q_heads;
  bool ok;
};
ExactShape exact_shape(int32_t n_layers, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, int32_t seq_len) {
  ExactShape x = {};
  if (n_layers < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0) return x;
  if (head_dim != 64 && head_dim != 128) return x;
  if (seq_len < 1 || seq_len > (1 << 20)) return x;
  x.N = seq_len;
  x.d = head_dim;
  x.G = n_heads / n_kv_heads;
  x.nb = (x.N + kBlockRows - 1) / kBlockRows;
  x.chunks = (x.nb * kBlockRows + kTcChunk - 1) / kTcChunk;
  x.slices = (x.N + kSliceKeys - 1) / kSliceKeys;
  x.q_heads = (int64_t)n_layers * n_heads;
  x.ok = (int64_t)x.nb * x.G * x.chunks <= (1 << 24);
  return x;
}
// Most query heads per batch: whole KV groups, a work-item count that fits an int, scratch within `budget` bytes
// (0 if not even one group fits).
int64_t exact_heads_per_batch(const ExactShape& x, size_t budget) {
  int64_t hb = x.q_heads;
  while (hb > x.G && hb * x.nb * x.chunks > (1 << 30)) hb -= x.G;
  while (hb > x.G && exact_layout(hb, x.nb, x.chunks, x.G, x.N, x.d, x.slices, true).total > budget)
    hb = std::max<int64_t>(x.G, hb / 2 / x.G * x.G);
  return exact_layout(hb, x.nb, x.chunks, x.G, x.N, x.d, x.slices, true).total <= budget ? hb : 0;
}
constexpr size_t kOwnBudget = (size_t)1536 << 20;   // what the library asks the stream's pool for by itself

}  // namespace

extern "C" size_t taskkv_exact_semantic_bytes(int32_t n_layers, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                              int32_t seq_len) {
  const ExactShape x = exact_shape(n_layers, n_heads, n_kv_heads, head_dim, seq_len);
  if (!x.ok) return 0;
  int64_t hb = exact_heads_per_batch(x, kOwnBudget);
  if (hb == 0) hb = x.G;                              // one KV group is the least a batch can be
  return exact_layout(hb, x.nb, x.chunks, x.G, x.N, x.d, x.slices, true).total;
}

extern "C" taskkv_status taskkv_exact_semantic(const void* q, const void* k, const void* v, int32_t n_layers,
                                               int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, int32_t seq_len,
                                               float* sem_out, float* c_out, void* workspace_mem,
                                               size_t workspace_bytes, taskkv_stream stream) {
  if (!q || !k || !v || !sem_out) return TASKKV_EINVAL;
  const ExactShape x = exact_shape(n_layers, n_heads, n_kv_heads, head_dim, seq_len);
  if (!x.ok) return TASKKV_EINVAL;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v) & 15) return TASKKV_EINVAL;
  if (workspace_mem && ((uintptr_t)workspace_mem & 255)) return TASKKV_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int N = x.N, d = x.d, G = x.G, nb = x.nb, chunks = x.chunks, slices = x.slices;
  const int64_t q_heads = x.q_heads;

  int64_t hb = exact_heads_per_batch(x, workspace_mem ? workspace_bytes : kOwnBudget);
  if (hb == 0 && !workspace_mem) hb = G;
  if (hb == 0) return TASKKV_EALLOC;
  const ExactLayout lay = exact_layout(hb, nb, chunks, G, N, d, slices, true);
  const size_t o_status = lay.o_status, o_unit_N = lay.o_unit_N, o_c_off = lay.o_c_off, o_Cb = lay.o_Cb,
               o_spart = lay.o_spart, o_stat = lay.o_stat, o_cfull = lay.o_cfull, o_part = lay.o_part;
  const int64_t U = hb * nb;
  unsigned char* ws = static_cast<unsigned char*>(workspace_mem);
  if (!ws && cudaMallocAsync(reinterpret_cast<void**>(&ws), lay.total, s) != cudaSuccess) {
    cudaGetLastError();
    return TASKKV_EALLOC;
  }

  DeviceProblem p = {};
  p.U = (int32_t)U;
  p.R = 1;
  p.n_heads = (int32_t)hb;
  p.n_kv = (int32_t)(hb / G);
  p.G = G;
  p.d = d;
  p.L = kBlockRows;
  p.rows = kBlockRows;
  p.rows_pad = kBlockRows;
  p.chunks_max = chunks * 2;
  p.status = reinterpret_cast<int32_t*>(ws + o_status);
  p.unit_N = reinterpret_cast<int32_t*>(ws + o_unit_N);
  p.c_off = reinterpret_cast<int64_t*>(ws + o_c_off);
  p.C = reinterpret_cast<float*>(ws + o_Cb);
  p.stat_part = reinterpret_cast<float*>(ws + o_spart);
  p.stat = reinterpret_cast<float*>(ws + o_stat);

  cudaError_t e = cudaMemsetAsync(ws + o_status, 0, 64, s);
  const size_t es = 2;
  for (int64_t h0 = 0; h0 < q_heads && e == cudaSuccess; h0 += hb) {
    const int64_t hn = std::min<int64_t>(hb, q_heads - h0);          // query heads of this batch (a multiple of G)
    const int64_t kv0 = h0 / G, kvn = hn / G;
    p.U = (int32_t)(hn * nb);
    {
      LaunchScope ls(K_EXACT_SUM, s);
      exact_init_kernel<<<(unsigned)((p.U + 1 + 255) / 256), 256, 0, s>>>(
          reinterpret_cast<int32_t*>(ws + o_unit_N), reinterpret_cast<int64_t*>(ws + o_c_off), p.U, nb);
    }
    const unsigned char* qb = static_cast<const unsigned char*>(q) + (size_t)h0 * N * d * es;
    const unsigned char* kb = static_cast<const unsigned char*>(k) + (size_t)kv0 * N * d * es;
    const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v) + (size_t)kv0 * N * d;
    e = launch_window_prefix(p, qb, kb, (int)hn, G, N, s);
    if (e != cudaSuccess) break;
    float* cf = c_out ? c_out + (size_t)kv0 * N : reinterpret_cast<float*>(ws + o_cfull);
    float* part = reinterpret_cast<float*>(ws + o_part);
    {
      LaunchScope ls(K_EXACT_SUM, s);
      exact_colsum_kernel<<<dim3((unsigned)((N + 255) / 256), (unsigned)kvn), 256, 0, s>>>(p.C, nb, G, N, cf);
    }
    {
      LaunchScope ls(K_EXACT_SUM, s);
      if (d == 64) exact_semvec_partial_kernel<64><<<dim3(slices, (unsigned)kvn), 64, 0, s>>>(cf, vb, N, slices, part);
      else exact_semvec_partial_kernel<128><<<dim3(slices, (unsigned)kvn), 128, 0, s>>>(cf, vb, N, slices, part);
    }
    {
      LaunchScope ls(K_EXACT_SUM, s);
      if (d == 64) exact_semvec_final_kernel<64><<<(unsigned)kvn, 64, 0, s>>>(part, slices, sem_out + (size_t)kv0 * d);
      else exact_semvec_final_kernel<128><<<(unsigned)kvn, 128, 0, s>>>(part, slices, sem_out + (size_t)kv0 * d);
    }
    e = cudaGetLastError();
  }
  int32_t dev_status = 0;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&dev_status, ws + o_status, 4, cudaMemcpyDeviceToHost, s);
  if (!workspace_mem) cudaFreeAsync(ws, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return TASKKV_ECUDA;
  }
  return dev_status;
}
