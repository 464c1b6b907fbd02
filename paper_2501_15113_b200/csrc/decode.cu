// Decode attention over the ragged per-head cache (Eq. 1, one query row per
// head, no mask): o_a = softmax(q_a K_u^T / sqrt(d)) V_u over the len_u rows of
// the KV head's segment, for the G query heads that share it.
//
// Split-K: a unit's rows are cut into work items of kDecodeChunk (512) rows, numbered
// by an exclusive scan over the units (so a 32768-row full head and a 772-row
// pruned head load the SMs alike).  Each item produces an un-normalised partial
// (running max, sum, weighted V) per head with an online softmax in fp32; one
// combine pass merges a unit's partials.  K/V rows are read once, as 16-byte
// vectors, by all G heads.
#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kUnroll = 4;

template <typename T, int D, int G>
__global__ void __launch_bounds__(kAttnThreads) decode_attn_kernel(DeviceProblem p, const T* __restrict__ q,
                                                                   const int32_t* __restrict__ lengths) {
  constexpr int EPL = 16 / (int)sizeof(T);          // elements per lane (one 16-byte vector)
  constexpr int LPR = D / EPL;                      // lanes per row
  constexpr int RPW = 32 / LPR;                     // rows per warp instruction
  constexpr int NSG = kAttnWarps * RPW;             // row sub-groups per block
  constexpr int ROW_BYTES = D * (int)sizeof(T);

  __shared__ float sm_m[NSG][G];
  __shared__ float sm_l[NSG][G];
  __shared__ __align__(16) float sm_acc[NSG][G][D];
  __shared__ int s_unit;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sg = lane / LPR, sl = lane % LPR;
  const int gsg = warp * RPW + sg;
  const int total = p.dec_off[p.U];
  const float scale2 = kLog2e * rsqrtf((float)D);

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    __syncthreads();                                // previous item's shared state consumed
    if (tid == 0) s_unit = upper_unit(p.dec_off, p.U, item);
    __syncthreads();
    const int u = s_unit;
    int len = p.len[u];
    if (lengths) len = min(max(lengths[u], 0), len);
    const int rbeg = (item - p.dec_off[u]) * kDecodeChunk;
    const int rend = min(len, rbeg + kDecodeChunk);
    const int64_t seg = p.seg_off[u];
    const unsigned char* kp = static_cast<const unsigned char*>(p.k_pool) + (size_t)seg * ROW_BYTES + sl * 16;
    const unsigned char* vp = static_cast<const unsigned char*>(p.v_pool) + (size_t)seg * ROW_BYTES + sl * 16;

    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)u * G + g) * D + sl * EPL);
      Vec16<T>::unpack(raw, qf[g]);
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

    for (int base = rbeg; base < rend; base += NSG * kUnroll) {   // warp-uniform trip count
      const int r0 = base + gsg;
      uint4 kraw[kUnroll], vraw[kUnroll];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int r = r0 + i * NSG;
        if (r < rend) {
          kraw[i] = *reinterpret_cast<const uint4*>(kp + (size_t)r * ROW_BYTES);
          vraw[i] = *reinterpret_cast<const uint4*>(vp + (size_t)r * ROW_BYTES);
        } else {
          kraw[i] = make_uint4(0, 0, 0, 0);
          vraw[i] = make_uint4(0, 0, 0, 0);
        }
      }
      float s[kUnroll][G];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        float kf[EPL];
        Vec16<T>::unpack(kraw[i], kf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float d0 = 0.f;
#pragma unroll
          for (int e = 0; e < EPL; ++e) d0 = fmaf(qf[g][e], kf[e], d0);
          s[i][g] = d0;
        }
      }
#pragma unroll
      for (int i = 0; i < kUnroll; ++i)
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float v = s[i][g];
#pragma unroll
          for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          s[i][g] = (r0 + i * NSG < rend) ? v : -INFINITY;
        }
      float pw[kUnroll][G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float mn = m[g];
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) mn = fmaxf(mn, s[i][g]);
        const float mu = (mn == -INFINITY) ? 0.f : mn;
        const float corr = exp2f(m[g] - mu);
        float ps = 0.f;
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
          pw[i][g] = exp2f(s[i][g] - mu);
          ps += pw[i][g];
        }
        l[g] = l[g] * corr + ps;
        m[g] = mn;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[g][e] *= corr;
      }
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        float vf[EPL];
        Vec16<T>::unpack(vraw[i], vf);
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(pw[i][g], vf[e], acc[g][e]);
      }
    }

    // merge the block's sub-groups
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (sl == 0) { sm_m[gsg][g] = m[g]; sm_l[gsg][g] = l[g]; }
#pragma unroll
      for (int e = 0; e < EPL; ++e) sm_acc[gsg][g][sl * EPL + e] = acc[g][e];
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += kAttnThreads) {
      const int g = i / D, dd = i % D;
      float M = -INFINITY;
#pragma unroll
      for (int x = 0; x < NSG; ++x) M = fmaxf(M, sm_m[x][g]);
      float a = 0.f, ll = 0.f;
#pragma unroll
      for (int x = 0; x < NSG; ++x) {
        const float mx = sm_m[x][g];
        const float w = (mx == -INFINITY) ? 0.f : exp2f(mx - M);
        a = fmaf(w, sm_acc[x][g][dd], a);
        ll = fmaf(w, sm_l[x][g], ll);
      }
      p.part_acc[((size_t)item * G + g) * D + dd] = a;
      if (dd == 0) {
        p.part_ml[((size_t)item * G + g) * 2 + 0] = M;
        p.part_ml[((size_t)item * G + g) * 2 + 1] = ll;
      }
    }
  }
}

// One block per (unit, query head of the group): merge the unit's partials.  First the block finds
// the largest running maximum, then each warp accumulates every fourth partial against it (independent
// loads, fixed order), and the four warps are summed in shared memory.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kAttnThreads) decode_combine_kernel(DeviceProblem p, T* __restrict__ out) {
  constexpr int EPL = D / 32;
  __shared__ float s_max[kAttnWarps];
  __shared__ float s_l[kAttnWarps];
  __shared__ float s_acc[kAttnWarps][D];
  const int u = blockIdx.x / G, g = blockIdx.x % G;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int i0 = p.dec_off[u], i1 = p.dec_off[u + 1];
  float M = -INFINITY;
  for (int i = i0 + tid; i < i1; i += kAttnThreads) M = fmaxf(M, p.part_ml[((size_t)i * G + g) * 2]);
  M = warp_max(M);
  if (lane == 0) s_max[warp] = M;
  __syncthreads();
  M = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  float L = 0.f;
#pragma unroll 4
  for (int i = i0 + warp; i < i1; i += kAttnWarps) {
    const float mi = p.part_ml[((size_t)i * G + g) * 2];
    const float li = p.part_ml[((size_t)i * G + g) * 2 + 1];
    const float wgt = (mi == -INFINITY) ? 0.f : exp2f(mi - M);
    L = fmaf(wgt, li, L);
    const float* pa = p.part_acc + ((size_t)i * G + g) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(wgt, pa[e], acc[e]);
  }
#pragma unroll
  for (int e = 0; e < EPL; ++e) s_acc[warp][lane * EPL + e] = acc[e];
  if (lane == 0) s_l[warp] = L;
  __syncthreads();
  if (tid < D) {
    const float Lt = (s_l[0] + s_l[1]) + (s_l[2] + s_l[3]);
    const float a = (s_acc[0][tid] + s_acc[1][tid]) + (s_acc[2][tid] + s_acc[3][tid]);
    store_out(out + ((size_t)u * G + g) * D + tid, Lt > 0.f ? a / Lt : 0.f);
  }
}

template <typename T, int D, int G>
cudaError_t launch_typed(const DeviceProblem& p, const void* q, const int32_t* lengths, void* out,
                         cudaStream_t s) {
  // persistent blocks: 16 per SM (measured best on B200 with 512-row items)
  int64_t grid = p.max_items < 148 * 16 ? p.max_items : 148 * 16;
  if (grid < 1) grid = 1;
  {
    LaunchScope ls(K_DECODE_ATTN, s);
    decode_attn_kernel<T, D, G><<<(unsigned)grid, kAttnThreads, 0, s>>>(p, static_cast<const T*>(q), lengths);
  }
  {
    LaunchScope ls(K_DECODE_COMBINE, s);
    decode_combine_kernel<T, D, G><<<(unsigned)(p.U * G), kAttnThreads, 0, s>>>(p, static_cast<T*>(out));
  }
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_group(const DeviceProblem& p, const void* q, const int32_t* lengths, void* out,
                         cudaStream_t s) {
  switch (p.G) {
    case 1: return launch_typed<T, D, 1>(p, q, lengths, out, s);
    case 2: return launch_typed<T, D, 2>(p, q, lengths, out, s);
    case 4: return launch_typed<T, D, 4>(p, q, lengths, out, s);
    case 8: return launch_typed<T, D, 8>(p, q, lengths, out, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_decode(const DeviceProblem& p, int dtype, const void* q, const int32_t* lengths, void* out,
                          cudaStream_t s) {
  cudaError_t e = launch_decode_plan(p, lengths, s);
  if (e != cudaSuccess) return e;
  if (dtype == TASKKV_F32)
    return p.d == 64 ? launch_group<float, 64>(p, q, lengths, out, s) : launch_group<float, 128>(p, q, lengths, out, s);
  return p.d == 64 ? launch_group<__nv_bfloat16, 64>(p, q, lengths, out, s)
                   : launch_group<__nv_bfloat16, 128>(p, q, lengths, out, s);
}

}  // namespace taskkv
