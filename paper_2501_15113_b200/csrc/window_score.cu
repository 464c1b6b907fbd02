// Observation-window scores (Eq. 12, Eq. 13): for every unit
//   S = Q_win K^T / sqrt(d), causal mask on the last L keys, row softmax,
//   C[j] = mean over the unit's G*L window rows of the normalised weights.
//
// Generic two-pass path on the CUDA cores (fp32 accumulate), used for fp32
// inputs and as the reference implementation for bf16:
//   pass 1  per (unit, 1024-key chunk): row maxima and exp-sums  -> partial stats
//   reduce  per unit: combine chunks -> (row max, 1 / row sum)
//   pass 2  per (unit, chunk): recompute S, C[j] = sum_i exp(s_ij - max_i) / Z_i / rows
// Scores are kept in log2 units (scaled by log2(e)/sqrt(d)) so exp is one ex2.
#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kTile = 128;      // keys per tile, one per thread
constexpr int kRowBlock = 16;   // window rows accumulated in registers at a time

template <typename T, int D>
struct WinSmem {
  static constexpr int kRowBytes = D * (int)sizeof(T) + 16;  // +16: conflict-free 16-byte row reads
};

template <typename T, int D, int PASS>
__global__ void __launch_bounds__(kTile) window_pass_kernel(DeviceProblem p, UnitRange ur) {
  const int u = ur.unit(blockIdx.y);
  const int N = p.unit_N[u];
  const int key0 = blockIdx.x * kScoreChunk;
  if (key0 >= N) return;
  const int key_end = min(N, key0 + kScoreChunk);
  const int rows = p.rows, rows_pad = p.rows_pad, L = p.L;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  extern __shared__ __align__(16) unsigned char smem[];
  float* Qs = reinterpret_cast<float*>(smem);                       // [rows_pad][D]
  unsigned char* Ks = smem + (size_t)rows_pad * D * sizeof(float);  // [kTile][kRowBytes]
  float2* st = reinterpret_cast<float2*>(Ks + kTile * WinSmem<T, D>::kRowBytes);  // [rows_pad][4]

  // Q rows of the unit's G heads: [rows][d] contiguous, converted to fp32 once.
  const T* q = static_cast<const T*>(p.q_ptr[u]);
  for (int i = tid; i < rows_pad * D; i += kTile) Qs[i] = (i < rows * D) ? to_float(q[i]) : 0.f;
  for (int i = tid; i < rows_pad * 4; i += kTile) {
    if (PASS == 1) {
      st[i] = make_float2(-INFINITY, 0.f);
    } else if (i < rows_pad) {
      // pass 2: st[row] = (row max, 1/Z)
      st[i] = (i < rows) ? reinterpret_cast<const float2*>(p.stat)[(size_t)u * rows_pad + i]
                         : make_float2(0.f, 0.f);
    }
  }

  const float scale2 = kLog2e * rsqrtf((float)D);
  constexpr int VN = Vec16<T>::N;
  constexpr int VPR = D / VN;  // 16-byte vectors per key row
  const unsigned char* kbase = static_cast<const unsigned char*>(p.k_ptr[u]);
  const unsigned char* krow = Ks + tid * WinSmem<T, D>::kRowBytes;

  for (int t0 = key0; t0 < key_end; t0 += kTile) {
    __syncthreads();  // previous tile consumed (and Q/state initialised on the first trip)
    for (int v = tid; v < kTile * VPR; v += kTile) {
      const int r = v / VPR, c = v % VPR;
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (t0 + r < N)
        raw = *reinterpret_cast<const uint4*>(kbase + ((size_t)(t0 + r) * D) * sizeof(T) + (size_t)c * 16);
      *reinterpret_cast<uint4*>(Ks + r * WinSmem<T, D>::kRowBytes + c * 16) = raw;
    }
    __syncthreads();

    const int j = t0 + tid;       // this thread's key
    float csum = 0.f;
    for (int rb = 0; rb < rows_pad; rb += kRowBlock) {
      float acc[kRowBlock];
#pragma unroll
      for (int i = 0; i < kRowBlock; ++i) acc[i] = 0.f;
#pragma unroll 2
      for (int dd = 0; dd < D; dd += VN) {
        float kf[VN];
        Vec16<T>::unpack(*reinterpret_cast<const uint4*>(krow + dd * sizeof(T)), kf);
#pragma unroll
        for (int i = 0; i < kRowBlock; ++i) {
          const float4* qp = reinterpret_cast<const float4*>(Qs + (rb + i) * D + dd);
#pragma unroll
          for (int h = 0; h < VN / 4; ++h) {
            const float4 qv = qp[h];
            acc[i] = fmaf(qv.x, kf[4 * h + 0], acc[i]);
            acc[i] = fmaf(qv.y, kf[4 * h + 1], acc[i]);
            acc[i] = fmaf(qv.z, kf[4 * h + 2], acc[i]);
            acc[i] = fmaf(qv.w, kf[4 * h + 3], acc[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kRowBlock; ++i) {
        const int row = rb + i;
        // window row (row % L) sits at position N - L + (row % L)
        const bool visible = (row < rows) && (j < N) && (j <= N - L + (row % L));
        const float s2 = acc[i] * scale2;
        if (PASS == 1) {
          const float sv = visible ? s2 : -INFINITY;
          const float m = warp_max(sv);
          const float e = (visible && m > -INFINITY) ? exp2f(sv - m) : 0.f;
          const float z = warp_sum(e);
          if (lane == 0 && row < rows && m > -INFINITY) {
            float2 o = st[row * 4 + warp];
            const float M = fmaxf(o.x, m);
            o.y = o.y * exp2f(o.x - M) + z * exp2f(m - M);
            o.x = M;
            st[row * 4 + warp] = o;
          }
        } else {
          if (visible) {
            const float2 ms = st[row];
            csum += exp2f(s2 - ms.x) * ms.y;
          }
        }
      }
    }
    if (PASS == 2 && j < N) p.C[p.c_off[u] + j] = csum * (1.0f / (float)rows);
  }

  if (PASS == 1) {
    __syncthreads();
    for (int row = tid; row < rows_pad; row += kTile) {
      float M = -INFINITY;
      for (int w = 0; w < 4; ++w) M = fmaxf(M, st[row * 4 + w].x);
      float z = 0.f;
      for (int w = 0; w < 4; ++w) {
        const float2 o = st[row * 4 + w];
        if (o.x > -INFINITY) z += o.y * exp2f(o.x - M);
      }
      reinterpret_cast<float2*>(p.stat_part)[((size_t)u * p.chunks_max + blockIdx.x) * rows_pad + row] =
          make_float2(M, z);
    }
  }
}

// Combine the chunk partials of one unit: (max, sum) -> (max, 1/sum) per window row.
__global__ void window_reduce_kernel(DeviceProblem p, UnitRange ur) {
  const int u = ur.unit(blockIdx.x);
  const int row = threadIdx.x;
  if (row >= p.rows_pad) return;
  const int N = p.unit_N[u];
  const int chunks = (N + kScoreChunk - 1) / kScoreChunk;
  const float2* part = reinterpret_cast<const float2*>(p.stat_part) + (size_t)u * p.chunks_max * p.rows_pad;
  float M = -INFINITY;
  for (int c = 0; c < chunks; ++c) M = fmaxf(M, part[(size_t)c * p.rows_pad + row].x);
  float z = 0.f;
  for (int c = 0; c < chunks; ++c) {
    const float2 o = part[(size_t)c * p.rows_pad + row];
    if (o.x > -INFINITY) z += o.y * exp2f(o.x - M);
  }
  float2 out = make_float2(0.f, 0.f);
  if (row < p.rows && z > 0.f) out = make_float2(M, 1.0f / z);
  reinterpret_cast<float2*>(p.stat)[(size_t)u * p.rows_pad + row] = out;
}

// Caller-supplied normalisers lse_i = ln sum_j exp(s_ij) of the window rows, in place of pass 1.  A unit's G*L rows
// are contiguous in [R][n][L].  Tensor-core path: one offset per row, lse * log2(e) + log2(rows); here: the pair
// (reference, 1 / sum relative to it) = (lse * log2(e), 1).
__global__ void lse_to_stat_kernel(DeviceProblem p, int u0, const float* __restrict__ lse, int tc_format) {
  const int lu = blockIdx.x, row = threadIdx.x;
  if (row >= p.rows) return;
  const float v = lse[(size_t)lu * p.rows + row] * kLog2e;
  const size_t u = (size_t)(u0 + lu);
  if (tc_format) p.stat[u * (2 * p.rows_pad) + row] = v + log2f((float)p.rows);
  else reinterpret_cast<float2*>(p.stat)[u * p.rows_pad + row] = make_float2(v, 1.0f);
}

template <typename T, int D>
cudaError_t launch_generic(const DeviceProblem& p, int max_N, const WindowHostInfo& h, cudaStream_t s, int layer0,
                           int n_layers) {
  const size_t smem = (size_t)p.rows_pad * D * sizeof(float) + (size_t)kTile * WinSmem<T, D>::kRowBytes +
                      (size_t)p.rows_pad * 4 * sizeof(float2);
  cudaError_t e;
  e = cudaFuncSetAttribute(window_pass_kernel<T, D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(window_pass_kernel<T, D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const UnitRange ur = layer_range(p, h.batch, layer0, n_layers);
  const dim3 grid((max_N + kScoreChunk - 1) / kScoreChunk, ur.blocks);
  if (h.lse) {
    const int per_seq = p.R * p.n_kv;
    const size_t lse_skip = (size_t)(layer0 - h.base_layer) * p.n_heads * p.L;
    for (int b = 0; b < h.batch; ++b) {
      e = launch_lse_to_stat(p, b * per_seq + ur.first, ur.count, static_cast<const float*>(h.lse[b]) + lse_skip, false, s);
      if (e != cudaSuccess) return e;
    }
  } else {
    {
      LaunchScope ls(K_WINDOW_STATS, s);
      window_pass_kernel<T, D, 1><<<grid, kTile, smem, s>>>(p, ur);
    }
    {
      LaunchScope ls(K_WINDOW_REDUCE, s);
      window_reduce_kernel<<<ur.blocks, p.rows_pad, 0, s>>>(p, ur);
    }
  }
  {
    LaunchScope ls(K_WINDOW_SCORES, s);
    window_pass_kernel<T, D, 2><<<grid, kTile, smem, s>>>(p, ur);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_lse_to_stat(const DeviceProblem& p, int u0, int n_units, const float* lse, bool tensor_core_format,
                               cudaStream_t s) {
  LaunchScope ls(K_WINDOW_REDUCE, s);
  lse_to_stat_kernel<<<n_units, 128, 0, s>>>(p, u0, lse, tensor_core_format ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_window_scores(const DeviceProblem& p, int dtype, int max_N, const WindowHostInfo& h,
                                 cudaStream_t s, int layer0, int n_layers) {
  if (n_layers < 0) { layer0 = 0; n_layers = p.R; }
  // bf16 with 32 / 64 / 128 window rows runs on the tensor cores; everything else here
  if (window_tc_supported(p, dtype)) return launch_window_scores_tc(p, h, s, layer0, n_layers);
  if (dtype == TASKKV_F32) {
    return p.d == 64 ? launch_generic<float, 64>(p, max_N, h, s, layer0, n_layers)
                     : launch_generic<float, 128>(p, max_N, h, s, layer0, n_layers);
  }
  return p.d == 64 ? launch_generic<__nv_bfloat16, 64>(p, max_N, h, s, layer0, n_layers)
                   : launch_generic<__nv_bfloat16, 128>(p, max_N, h, s, layer0, n_layers);
}

}  // namespace taskkv
