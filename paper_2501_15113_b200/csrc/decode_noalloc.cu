// taskkv_decode_noalloc: ragged decode attention for callers that must not
// allocate device memory.
//
// The regular decode call keeps its split-K partial results in memory that was
// allocated when the cache was built.  Some callers cannot do that: code that
// runs inside a serving engine which has already handed every byte of device
// memory to its own pool, or code in a latency-critical section where the
// implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.
// For them this file carries the same attention computation with its scratch in
// a fixed, file-scope device array (kScratchBytes, resident on every GPU that
// loads the library until the process exits).  The call allocates nothing and
// frees nothing; the caller passes the query, the K/V pools, the segment
// offsets, the lengths and the output.
//
// Work split: every unit is cut into the same number of splits (chosen on the
// host from max_len and the scratch size); split s of unit u covers rows
// [s * rps, min(len_u, (s + 1) * rps)).  Every split writes its partial, also an
// empty one, so nothing left in the array by an earlier call is ever read.
// The array is shared by all calls: two calls whose kernels overlap on the GPU
// (different streams, or different host threads) race on it.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace taskkv {
namespace {

constexpr size_t kScratchBytes = 32u << 20;   // 32 MiB per GPU
constexpr int kMaxDevices = 64;
constexpr int kNaThreads = 128;
constexpr int kNaWarps = kNaThreads / 32;
constexpr int kNaUnroll = 4;
constexpr int kNaMinRows = 256;               // rows per split aimed for

// In host code this name is only a stand-in; the device address comes from
// cudaGetSymbolAddress (see scratch_for_current_device).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_na_mu;
void* g_na_ptr[kMaxDevices] = {nullptr};

// Looks up, once per device and with that device current, where the scratch
// array lives on the device.
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_na_mu);
  if (!g_na_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_na_ptr[dev] = ptr;
  }
  *out = g_na_ptr[dev];
  return cudaSuccess;
}

struct NaArgs {
  const void* q;
  const unsigned char* k_pool;
  const unsigned char* v_pool;
  const int64_t* seg_off;
  const int32_t* lengths;
  void* out;
  float* part_acc;     // [n_units * splits][G][D]   (inside the static scratch)
  float* part_ml;      // [n_units * splits][G][2]
  int32_t n_units, splits, rows_per_split;
  int32_t max_len;     // lengths above it are clamped to it
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(kNaThreads) na_attn_kernel(NaArgs a) {
  constexpr int EPL = 16 / (int)sizeof(T);
  constexpr int LPR = D / EPL;
  constexpr int RPW = 32 / LPR;
  constexpr int NSG = kNaWarps * RPW;
  constexpr int ROW_BYTES = D * (int)sizeof(T);

  __shared__ float sm_m[NSG][G];
  __shared__ float sm_l[NSG][G];
  __shared__ __align__(16) float sm_acc[NSG][G][D];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sg = lane / LPR, sl = lane % LPR;
  const int gsg = warp * RPW + sg;
  const int total = a.n_units * a.splits;
  const float scale2 = kLog2e * rsqrtf((float)D);
  const T* q = static_cast<const T*>(a.q);

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    __syncthreads();
    const int u = item / a.splits, sp = item % a.splits;
    const int len = min(max(a.lengths[u], 0), a.max_len);
    const int rbeg = min(len, sp * a.rows_per_split);
    const int rend = min(len, rbeg + a.rows_per_split);
    const int64_t seg = a.seg_off[u];
    const unsigned char* kp = a.k_pool + (size_t)seg * ROW_BYTES + sl * 16;
    const unsigned char* vp = a.v_pool + (size_t)seg * ROW_BYTES + sl * 16;

    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      Vec16<T>::unpack(*reinterpret_cast<const uint4*>(q + ((size_t)u * G + g) * D + sl * EPL), qf[g]);
#pragma unroll
      for (int e = 0; e < EPL; ++e) qf[g][e] *= scale2;
    }
    float m[G], l[G], acc[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      m[g] = -INFINITY;
      l[g] = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
    }
    for (int base = rbeg; base < rend; base += NSG * kNaUnroll) {
      const int r0 = base + gsg;
      uint4 kraw[kNaUnroll], vraw[kNaUnroll];
#pragma unroll
      for (int i = 0; i < kNaUnroll; ++i) {
        const int r = r0 + i * NSG;
        kraw[i] = make_uint4(0, 0, 0, 0);
        vraw[i] = make_uint4(0, 0, 0, 0);
        if (r < rend) {
          kraw[i] = *reinterpret_cast<const uint4*>(kp + (size_t)r * ROW_BYTES);
          vraw[i] = *reinterpret_cast<const uint4*>(vp + (size_t)r * ROW_BYTES);
        }
      }
      float s[kNaUnroll][G];
#pragma unroll
      for (int i = 0; i < kNaUnroll; ++i) {
        float kf[EPL];
        Vec16<T>::unpack(kraw[i], kf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float d0 = 0.f;
#pragma unroll
          for (int e = 0; e < EPL; ++e) d0 = fmaf(qf[g][e], kf[e], d0);
#pragma unroll
          for (int o = LPR / 2; o > 0; o >>= 1) d0 += __shfl_xor_sync(0xffffffffu, d0, o);
          s[i][g] = (r0 + i * NSG < rend) ? d0 : -INFINITY;
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float mn = m[g];
#pragma unroll
        for (int i = 0; i < kNaUnroll; ++i) mn = fmaxf(mn, s[i][g]);
        const float mu = (mn == -INFINITY) ? 0.f : mn;
        const float corr = exp2f(m[g] - mu);
        l[g] *= corr;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[g][e] *= corr;
        m[g] = mn;
#pragma unroll
        for (int i = 0; i < kNaUnroll; ++i) {
          const float pw = exp2f(s[i][g] - mu);
          l[g] += pw;
          float vf[EPL];
          Vec16<T>::unpack(vraw[i], vf);
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(pw, vf[e], acc[g][e]);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (sl == 0) { sm_m[gsg][g] = m[g]; sm_l[gsg][g] = l[g]; }
#pragma unroll
      for (int e = 0; e < EPL; ++e) sm_acc[gsg][g][sl * EPL + e] = acc[g][e];
    }
    __syncthreads();
    // always written, also for an empty split: (max = -inf, sum = 0, acc = 0)
    for (int i = tid; i < G * D; i += kNaThreads) {
      const int g = i / D, dd = i % D;
      float M = -INFINITY;
#pragma unroll
      for (int x = 0; x < NSG; ++x) M = fmaxf(M, sm_m[x][g]);
      float av = 0.f, ll = 0.f;
#pragma unroll
      for (int x = 0; x < NSG; ++x) {
        const float mx = sm_m[x][g];
        const float w = (mx == -INFINITY) ? 0.f : exp2f(mx - M);
        av = fmaf(w, sm_acc[x][g][dd], av);
        ll = fmaf(w, sm_l[x][g], ll);
      }
      a.part_acc[((size_t)item * G + g) * D + dd] = av;
      if (dd == 0) {
        a.part_ml[((size_t)item * G + g) * 2 + 0] = M;
        a.part_ml[((size_t)item * G + g) * 2 + 1] = ll;
      }
    }
  }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(256) na_combine_kernel(NaArgs a) {
  constexpr int EPL = D / 32;
  const int w = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= a.n_units * G) return;
  const int u = w / G, g = w % G;
  const int i0 = u * a.splits, i1 = i0 + a.splits;
  float M = -INFINITY;
  for (int i = i0 + lane; i < i1; i += 32) M = fmaxf(M, a.part_ml[((size_t)i * G + g) * 2]);
  M = warp_max(M);
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  float L = 0.f;
  for (int i = i0; i < i1; ++i) {
    const float mi = a.part_ml[((size_t)i * G + g) * 2];
    if (mi == -INFINITY) continue;
    const float wgt = exp2f(mi - M);
    L = fmaf(wgt, a.part_ml[((size_t)i * G + g) * 2 + 1], L);
    const float* pa = a.part_acc + ((size_t)i * G + g) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(wgt, pa[e], acc[e]);
  }
  const float inv = L > 0.f ? 1.0f / L : 0.f;
  T* o = static_cast<T*>(a.out) + ((size_t)u * G + g) * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) store_out(o + e, acc[e] * inv);
}

template <typename T, int D, int G>
cudaError_t na_launch(const NaArgs& a, cudaStream_t s) {
  const int64_t total = (int64_t)a.n_units * a.splits;
  const unsigned grid = (unsigned)(total < 148 * 8 ? total : 148 * 8);
  {
    LaunchScope ls(K_DECODE_ATTN, s);
    na_attn_kernel<T, D, G><<<grid, kNaThreads, 0, s>>>(a);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;      // no combine over partials that were never written
  {
    LaunchScope ls(K_DECODE_COMBINE, s);
    na_combine_kernel<T, D, G><<<(unsigned)((a.n_units * G + 7) / 8), 256, 0, s>>>(a);
  }
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t na_group(const NaArgs& a, int G, cudaStream_t s) {
  switch (G) {
    case 1: return na_launch<T, D, 1>(a, s);
    case 2: return na_launch<T, D, 2>(a, s);
    case 4: return na_launch<T, D, 4>(a, s);
    case 8: return na_launch<T, D, 8>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace
}  // namespace taskkv

extern "C" taskkv_status taskkv_decode_noalloc(const void* q, const void* k_pool, const void* v_pool,
                                               const int64_t* seg_off, const int32_t* lengths,
                                               int32_t n_units, int32_t group, int32_t head_dim,
                                               int32_t dtype, int32_t max_len, void* out,
                                               taskkv_stream stream) {
  using namespace taskkv;
  if (!q || !k_pool || !v_pool || !seg_off || !lengths || !out) return TASKKV_EINVAL;
  if ((((uintptr_t)q | (uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)out) & 15) != 0) return TASKKV_EINVAL;
  if (n_units < 1 || max_len < 1) return TASKKV_EINVAL;
  if (group != 1 && group != 2 && group != 4 && group != 8) return TASKKV_EINVAL;
  if (head_dim != 64 && head_dim != 128) return TASKKV_EINVAL;
  if (dtype != TASKKV_F32 && dtype != TASKKV_BF16) return TASKKV_EINVAL;

  // scratch per work item: G * D accumulators + G * (max, sum)
  const size_t acc_bytes = (size_t)group * head_dim * sizeof(float);
  const size_t ml_bytes = (size_t)group * 2 * sizeof(float);
  const size_t item_bytes = acc_bytes + ml_bytes;
  const size_t max_items = (kScratchBytes - 256) / item_bytes;
  if ((size_t)n_units > max_items) {
    std::fprintf(stderr,
                 "taskkv_decode_noalloc: %d units x %d heads x %d dims need more than the fixed %zu-byte scratch "
                 "(at most %zu units at this shape)\n", n_units, group, head_dim, kScratchBytes, max_items);
    return TASKKV_EINVAL;
  }
  int64_t splits = ((int64_t)max_len + kNaMinRows - 1) / kNaMinRows;
  if (splits > (int64_t)(max_items / (size_t)n_units)) splits = (int64_t)(max_items / (size_t)n_units);
  if (splits < 1) splits = 1;
  const int64_t rps = ((int64_t)max_len + splits - 1) / splits;

  void* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) {
    cudaGetLastError();
    return TASKKV_ECUDA;
  }
  NaArgs a;
  a.q = q;
  a.k_pool = static_cast<const unsigned char*>(k_pool);
  a.v_pool = static_cast<const unsigned char*>(v_pool);
  a.seg_off = seg_off;
  a.lengths = lengths;
  a.out = out;
  a.n_units = n_units;
  a.splits = (int32_t)splits;
  a.rows_per_split = (int32_t)rps;
  a.max_len = max_len;
  const size_t items = (size_t)n_units * (size_t)splits;
  a.part_acc = static_cast<float*>(scratch);
  a.part_ml = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) +
                                       (items * acc_bytes + 255) / 256 * 256);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (dtype == TASKKV_F32)
    e = head_dim == 64 ? na_group<float, 64>(a, group, s) : na_group<float, 128>(a, group, s);
  else
    e = head_dim == 64 ? na_group<__nv_bfloat16, 64>(a, group, s) : na_group<__nv_bfloat16, 128>(a, group, s);
  return e == cudaSuccess ? TASKKV_OK : TASKKV_ECUDA;
}
