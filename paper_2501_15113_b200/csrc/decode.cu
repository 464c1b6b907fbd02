// Decode attention over the ragged per-head cache (Eq. 1, one query row per
// head, no mask): o_a = softmax(q_a K_u^T / sqrt(d)) V_u over the len_u rows of
// the KV head's segment, for the G query heads that share it.
//
// Split-K: a unit's rows are cut into work items of kDecodeChunk (512) rows, numbered once at
// compression for every unit at its capacity (so a 32768-row full head and a 772-row pruned head
// load the SMs alike; items beyond a segment's current length are skipped).  Each item produces an un-normalised partial
// (running max, sum, weighted V) per head with an online softmax in fp32; one
// combine pass merges a unit's partials.  K/V rows are read once, as 16-byte
// vectors, by all G heads.
#include <type_traits>

#include "common.cuh"

namespace taskkv {

namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kUnroll = 4;

// PAGED (both attention kernels): the rows of a unit live in pages of the shared pool; the rows one loop iteration
// touches never cross a page (a page holds a multiple of 64 rows).  A work item's 512 rows lie in at most 8 pages:
// every lane reads one of their table entries when the item starts (lane i and i + 8, ... hold the i-th), and an
// iteration gets its page by a shuffle, so no table load sits between an iteration and its row loads.
struct ItemPages {
  int first;   // table index of the item's first page
  int mine;    // page held by this lane
};
__device__ __forceinline__ ItemPages item_pages(const DeviceProblem& p, int u, int rbeg, int lane) {
  ItemPages ip;
  ip.first = rbeg / p.page_rows;
  const int pi = ip.first + (lane & 7);
  ip.mine = pi < p.page_stride ? p.page_tab[(size_t)u * p.page_stride + pi] : 0;
  return ip;
}
// Walks the item's rows in steps of at most one page: where() gives the pool row of the current row minus that row's
// index (for all lanes of a converged warp), advance() moves on.  One division per item instead of one per step.
struct PageWalk {
  int pi;    // page of the current row, counted from the item's first
  int rem;   // its row within that page
  __device__ __forceinline__ void start(const DeviceProblem& p, const ItemPages& ip, int r) {
    pi = r / p.page_rows - ip.first;
    rem = r % p.page_rows;
  }
  __device__ __forceinline__ size_t where(const DeviceProblem& p, const ItemPages& ip, int r) const {
    const int pg = __shfl_sync(0xffffffffu, ip.mine, pi);
    return (size_t)((int64_t)pg * p.page_rows + rem - r);
  }
  __device__ __forceinline__ void advance(const DeviceProblem& p, int step) {
    rem += step;
    if (rem >= p.page_rows) {
      rem -= p.page_rows;
      ++pi;
    }
  }
};
template <typename T, int D, int G, bool PAGED>
__global__ void __launch_bounds__(kAttnThreads) decode_attn_kernel(DeviceProblem p, const T* __restrict__ q,
                                                                   const int32_t* __restrict__ lengths,
                                                                   const unsigned char* __restrict__ k_new,
                                                                   const unsigned char* __restrict__ v_new,
                                                                   T* __restrict__ out, int early) {
  constexpr int EPL = 16 / (int)sizeof(T);          // elements per lane (one 16-byte vector)
  constexpr int LPR = D / EPL;                      // lanes per row
  constexpr int RPW = 32 / LPR;                     // rows per warp instruction
  constexpr int NSG = kAttnWarps * RPW;             // row sub-groups per block
  constexpr int ROW_BYTES = D * (int)sizeof(T);

  __shared__ float sm_m[NSG][G];
  __shared__ float sm_l[NSG][G];
  __shared__ __align__(16) float sm_acc[NSG][G][D];
  __shared__ int s_unit, s_rbeg;
  __shared__ int s_direct;     // >= 0: the item is its unit's only one, the output goes to view unit s_direct

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sg = lane / LPR, sl = lane % LPR;
  const int gsg = warp * RPW + sg;
  // the view's layers are a contiguous range of layer-major indices, hence of work items
  const int w0 = p.view_l0 * lm_batch(p) * p.n_kv;
  // (from the host's table of block starts: it does not depend on which layers have been compressed so far)
  const int item0 = p.dec_base[p.view_l0 * lm_batch(p)], item1 = p.dec_base[(p.view_l0 + p.view_nl) * lm_batch(p)];
  const float scale2 = kLog2e * rsqrtf((float)D);

  // The table of work items is written when the cache is planned, not by the kernel before this one in the
  // stream: the block's first item is looked up before the wait, under that kernel's tail.
  int wi_first = 0;
  if (warp == 0 && item0 + (int)blockIdx.x < item1)
    wi_first = w0 + upper_unit_warp(p.dec_off + w0, p.view_U, item0 + (int)blockIdx.x, lane);
  // `early` (set by the host when the kernel before this one in the stream cannot be one that writes these units'
  // lengths or page tables: see launch_decode): the first item's unit data is read before the wait as well, and the
  // wait comes just before the block first touches what the caller's kernels produce (q, the new token's rows) or
  // writes anything.  (A block all of whose items are beyond their segments' lengths leaves without waiting.)
  bool waited = false;
  auto wait_once = [&]() {
    if (!waited) {
      grid_dependency_wait();
      grid_launch_dependents();
      waited = true;
    }
  };
  if (!early) wait_once();
  for (int item = item0 + blockIdx.x; item < item1; item += gridDim.x) {
    __syncthreads();                                // previous item's shared state consumed
    if (warp == 0) {
      const int wi = item == item0 + (int)blockIdx.x ? wi_first
                                                     : w0 + upper_unit_warp(p.dec_off + w0, p.view_U, item, lane);
      if (lane == 0) {
        s_unit = wi;
        s_rbeg = (item - p.dec_off[wi]) * kDecodeChunk;
      }
    }
    __syncthreads();
    const int w = s_unit;
    const LmUnit lu = lm_unit(p, w);
    const int vu = lu.v;                            // view unit: index into q and lengths
    const int u = lu.u;                             // unit: index into the cache
    int len = p.len[u];
    // fused step: the new token's row sits at index len; it is read from k_new / v_new and the item that holds
    // it also stores it in the segment (the length itself is raised by the combine pass)
    const int new_r = (k_new != nullptr && len < p.cap[u]) ? len : -1;
    if (new_r >= 0) ++len;
    if (lengths) len = min(max(lengths[vu], 0), len);
    const int rbeg = s_rbeg;
    if (rbeg >= len) continue;                      // an item of the reserve beyond the segment's length
    const int rend = min(len, rbeg + kDecodeChunk);
    if (tid == 0) s_direct = len <= kDecodeChunk ? vu : -1;     // read back after the row loop (no register held)
    const int64_t seg = p.seg_off[u];
    const unsigned char* kn_row = k_new + (size_t)vu * ROW_BYTES;
    const unsigned char* vn_row = v_new + (size_t)vu * ROW_BYTES;
    wait_once();
    if (new_r >= rbeg && new_r < rend) {
      bool have_page = true;
      if (PAGED && new_r % p.page_rows == 0) {
        // the appended row opens a new page: one comes off the pool (only this block touches the unit's new row)
        if (tid == 0) {
          const int at = pool_pop(p, 1);
          if (at >= 0) p.page_tab[(size_t)u * p.page_stride + new_r / p.page_rows] = p.pool_free[at];
          s_unit = at;                              // (the unit index has been read by everybody)
        }
        __syncthreads();
        have_page = s_unit >= 0;                    // an empty pool: status ESTATE, the row is not stored
      }
      if (have_page && tid < ROW_BYTES / 16) {
        const size_t drow = pool_row(p, u, seg, new_r);
        unsigned char* kd = static_cast<unsigned char*>(p.k_pool) + drow * ROW_BYTES + tid * 16;
        unsigned char* vd = static_cast<unsigned char*>(p.v_pool) + drow * ROW_BYTES + tid * 16;
        *reinterpret_cast<uint4*>(kd) = *reinterpret_cast<const uint4*>(kn_row + tid * 16);
        *reinterpret_cast<uint4*>(vd) = *reinterpret_cast<const uint4*>(vn_row + tid * 16);
      }
    }
    ItemPages ip{0, 0};
    if (PAGED) ip = item_pages(p, u, rbeg, lane);
    const unsigned char* kp = static_cast<const unsigned char*>(p.k_pool) + (PAGED ? 0 : (size_t)seg * ROW_BYTES) + sl * 16;
    const unsigned char* vp = static_cast<const unsigned char*>(p.v_pool) + (PAGED ? 0 : (size_t)seg * ROW_BYTES) + sl * 16;

    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)vu * G + g) * D + sl * EPL);
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

    // two copies of the row loop: only the item that holds the new token's row pays for telling it apart
    auto rows_loop = [&](auto has_new) {
    PageWalk pw{0, 0};
    if (PAGED) pw.start(p, ip, rbeg);
    for (int base = rbeg; base < rend; base += NSG * kUnroll) {   // warp-uniform trip count
      const int r0 = base + gsg;
      // pool row of row `base` minus base: adding a row index of this iteration gives its pool row
      size_t rowoff = 0;
      if (PAGED) {
        rowoff = pw.where(p, ip, base);
        pw.advance(p, NSG * kUnroll);
      }
      uint4 kraw[kUnroll], vraw[kUnroll];
      // one 64-bit address per array and iteration; the unrolled loads differ by compile-time offsets
      const unsigned char* kb = kp + (rowoff + (size_t)r0) * ROW_BYTES;
      const unsigned char* vb = vp + (rowoff + (size_t)r0) * ROW_BYTES;
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int r = r0 + i * NSG;
        if (r < rend) {
          kraw[i] = *reinterpret_cast<const uint4*>((decltype(has_new)::value && r == new_r) ? kn_row + sl * 16
                                                                                             : kb + i * NSG * ROW_BYTES);
          vraw[i] = *reinterpret_cast<const uint4*>((decltype(has_new)::value && r == new_r) ? vn_row + sl * 16
                                                                                             : vb + i * NSG * ROW_BYTES);
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

    };
    if (new_r >= rbeg && new_r < rend) rows_loop(std::true_type{}); else rows_loop(std::false_type{});

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
      if (s_direct >= 0) {
        // the unit's only item: this is Eq. 1 over the whole segment (what the combine pass would make of one
        // partial, bit for bit); the combine pass skips such units
        store_out(out + ((size_t)s_direct * G + g) * D + dd, ll > 0.f ? a / ll : 0.f);
        continue;
      }
      p.part_acc[((size_t)item * G + g) * D + dd] = a;
      if (dd == 0) {
        p.part_ml[((size_t)item * G + g) * 2 + 0] = M;
        p.part_ml[((size_t)item * G + g) * 2 + 1] = ll;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Grouped-query variant for bf16 (G >= 2 query heads per KV head): with several heads per row the
// scalar kernel above runs out of issue slots long before HBM, so the two contractions go through
// warp-level mma (m16n8k16, bf16 x bf16 -> fp32) on operands taken straight from 16-byte global
// loads -- no shared-memory staging; the fragment layouts are met by permuting the contraction
// index instead:
//   S^T[head, row] = Q K^T   A = Q (heads on the 16 M rows, rows >= G zero), B = 8 cache rows.  Lane
//       (g = lane/4, t = lane%4) owns cache row g and loads its 16-byte pieces i*4 + t; the two
//       halves of piece i are the lane's operand words of k-chunks 2i and 2i+1.  Q is loaded with the
//       same rule, so both sides agree on which d sits in which k slot.
//   O^T[d, head] += V^T P^T   the accumulator fragment of S^T (head g, rows 2t, 2t+1) is already the
//       B fragment of P^T; the A fragment needs pairs of consecutive rows at one d, built with one
//       byte-permute from the lane's loads of rows 2t, 2t+1, 2t+8, 2t+9 (piece g of each 128-byte
//       line).  Accumulator row (m-block mb, half hf) of lane g stands for d = pd(mb, hf, g).
// P is rounded to bf16 for the second product (fp32 accumulation); the normaliser is summed in fp32.
// Each warp walks 16-row blocks of the work item with its own running (max, sum, O^T); the four
// warps are merged like the sub-groups of the scalar kernel and the partial goes to the same slots.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t word_of(const uint4& v, int i) {
  return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

template <int D, int G, bool PAGED>
__global__ void __launch_bounds__(kAttnThreads, 4) decode_attn_mma_kernel(DeviceProblem p,
                                                                       const __nv_bfloat16* __restrict__ q,
                                                                       const int32_t* __restrict__ lengths,
                                                                       const unsigned char* __restrict__ k_new,
                                                                       const unsigned char* __restrict__ v_new,
                                                                       __nv_bfloat16* __restrict__ out, int early) {
  constexpr int ROW_BYTES = D * 2;
  constexpr int KC = D / 16;            // k-chunks of the first product
  constexpr int KP = D / 32;            // 16-byte pieces of a K row per lane
  constexpr int MB = D / 16;            // m-blocks (16 d each) of the second product
  constexpr int VP = D / 64;            // 16-byte pieces of a V row per lane
  constexpr int kBlk = 16;              // cache rows per warp iteration

  __shared__ float sm_m[kAttnWarps][G];
  __shared__ float sm_l[kAttnWarps][G];
  __shared__ __align__(16) float sm_acc[kAttnWarps][G][D];
  __shared__ int s_unit, s_rbeg;
  __shared__ int s_direct;     // >= 0: the item is its unit's only one, the output goes to view unit s_direct

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  // the view's layers are a contiguous range of layer-major indices, hence of work items
  const int w0 = p.view_l0 * lm_batch(p) * p.n_kv;
  // (from the host's table of block starts: it does not depend on which layers have been compressed so far)
  const int item0 = p.dec_base[p.view_l0 * lm_batch(p)], item1 = p.dec_base[(p.view_l0 + p.view_nl) * lm_batch(p)];
  const float scale2 = kLog2e * rsqrtf((float)D);
  // d of accumulator row (mb, hf) of this lane's two output rows: e = hf * MB + mb, piece e / 8, element e % 8
  auto pd = [&](int mb, int hf, int gg) { const int e = hf * MB + mb; return (e >> 3) * 64 + gg * 8 + (e & 7); };

  // The table of work items is written when the cache is planned, not by the kernel before this one in the
  // stream: the block's first item is looked up before the wait, under that kernel's tail.
  int wi_first = 0;
  if (warp == 0 && item0 + (int)blockIdx.x < item1)
    wi_first = w0 + upper_unit_warp(p.dec_off + w0, p.view_U, item0 + (int)blockIdx.x, lane);
  // `early` (set by the host when the kernel before this one in the stream cannot be one that writes these units'
  // lengths or page tables: see launch_decode): the first item's unit data is read before the wait as well, and the
  // wait comes just before the block first touches what the caller's kernels produce (q, the new token's rows) or
  // writes anything.  (A block all of whose items are beyond their segments' lengths leaves without waiting.)
  bool waited = false;
  auto wait_once = [&]() {
    if (!waited) {
      grid_dependency_wait();
      grid_launch_dependents();
      waited = true;
    }
  };
  if (!early) wait_once();
  for (int item = item0 + blockIdx.x; item < item1; item += gridDim.x) {
    __syncthreads();
    if (warp == 0) {
      const int wi = item == item0 + (int)blockIdx.x ? wi_first
                                                     : w0 + upper_unit_warp(p.dec_off + w0, p.view_U, item, lane);
      if (lane == 0) {
        s_unit = wi;
        s_rbeg = (item - p.dec_off[wi]) * kDecodeChunk;
      }
    }
    __syncthreads();
    const int w = s_unit;
    const LmUnit lu = lm_unit(p, w);
    const int vu = lu.v;                            // view unit: index into q and lengths
    const int u = lu.u;                             // unit: index into the cache
    int len = p.len[u];
    // fused step: the new token's row sits at index len; it is read from k_new / v_new and the item that holds
    // it also stores it in the segment (the length itself is raised by the combine pass)
    const int new_r = (k_new != nullptr && len < p.cap[u]) ? len : -1;
    if (new_r >= 0) ++len;
    if (lengths) len = min(max(lengths[vu], 0), len);
    const int rbeg = s_rbeg;
    if (rbeg >= len) continue;                      // an item of the reserve beyond the segment's length
    const int rend = min(len, rbeg + kDecodeChunk);
    if (tid == 0) s_direct = len <= kDecodeChunk ? vu : -1;     // read back after the row loop (no register held)
    const int64_t seg = p.seg_off[u];
    const unsigned char* kn_row = k_new + (size_t)vu * ROW_BYTES;
    const unsigned char* vn_row = v_new + (size_t)vu * ROW_BYTES;
    wait_once();
    if (new_r >= rbeg && new_r < rend) {
      bool have_page = true;
      if (PAGED && new_r % p.page_rows == 0) {
        // the appended row opens a new page: one comes off the pool (only this block touches the unit's new row)
        if (tid == 0) {
          const int at = pool_pop(p, 1);
          if (at >= 0) p.page_tab[(size_t)u * p.page_stride + new_r / p.page_rows] = p.pool_free[at];
          s_unit = at;                              // (the unit index has been read by everybody)
        }
        __syncthreads();
        have_page = s_unit >= 0;                    // an empty pool: status ESTATE, the row is not stored
      }
      if (have_page && tid < ROW_BYTES / 16) {
        const size_t drow = pool_row(p, u, seg, new_r);
        unsigned char* kd = static_cast<unsigned char*>(p.k_pool) + drow * ROW_BYTES + tid * 16;
        unsigned char* vd = static_cast<unsigned char*>(p.v_pool) + drow * ROW_BYTES + tid * 16;
        *reinterpret_cast<uint4*>(kd) = *reinterpret_cast<const uint4*>(kn_row + tid * 16);
        *reinterpret_cast<uint4*>(vd) = *reinterpret_cast<const uint4*>(vn_row + tid * 16);
      }
    }
    ItemPages ip{0, 0};
    if (PAGED) ip = item_pages(p, u, rbeg, lane);
    const unsigned char* kp = static_cast<const unsigned char*>(p.k_pool);
    const unsigned char* vp = static_cast<const unsigned char*>(p.v_pool);

    // Q fragments: head g on M row g
    uint32_t qa[KC][2];
#pragma unroll
    for (int i = 0; i < KP; ++i) {
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (g < G) raw = *reinterpret_cast<const uint4*>(q + ((size_t)vu * G + g) * D + (i * 4 + t) * 8);
      qa[2 * i][0] = raw.x; qa[2 * i][1] = raw.y;
      qa[2 * i + 1][0] = raw.z; qa[2 * i + 1][1] = raw.w;
    }
    float m_run = -INFINITY, l_run = 0.f;   // head g (this lane's share of the sum)
    float o[MB][4];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[mb][e] = 0.f;

    // byte offset of this lane's first K vector (row g, piece t) and V vector (row 2t, piece g) within a block
    const int klane = g * ROW_BYTES + t * 16, vlane = 2 * t * ROW_BYTES + g * 16;
    // two copies of the row loop: only the item that holds the new token's row pays for telling it apart
    auto rows_loop = [&](auto has_new) {
    PageWalk pw{0, 0};
    if (PAGED) pw.start(p, ip, rbeg + warp * kBlk);
    // kb, vb: this lane's first K and V vector of the current 16-row block; the unrolled loads differ from them by
    // compile-time offsets.  Contiguous layout: row r of the unit is pool row seg + r, the pointers step from block
    // to block; paged: they are set from the block's page.
    const unsigned char* kb = kp + ((size_t)seg + (size_t)(rbeg + warp * kBlk)) * ROW_BYTES + klane;
    const unsigned char* vb = vp + ((size_t)seg + (size_t)(rbeg + warp * kBlk)) * ROW_BYTES + vlane;
    for (int blk = rbeg + warp * kBlk; blk < rend; blk += kAttnWarps * kBlk) {   // warp-uniform
      if (PAGED) {
        // pool row of row `blk` minus blk: adding a row index of this 16-row block gives its pool row
        const size_t rowoff = pw.where(p, ip, blk);
        pw.advance(p, kAttnWarps * kBlk);
        kb = kp + (rowoff + (size_t)blk) * ROW_BYTES + klane;
        vb = vp + (rowoff + (size_t)blk) * ROW_BYTES + vlane;
      }
      uint4 kraw[2][KP], vraw[4][VP];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int r = blk + 8 * j + g;
#pragma unroll
        for (int i = 0; i < KP; ++i)
          kraw[j][i] = r < rend ? *reinterpret_cast<const uint4*>((decltype(has_new)::value && r == new_r)
                                                                      ? kn_row + (i * 4 + t) * 16
                                                                      : kb + j * 8 * ROW_BYTES + i * 64)
                                : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int r = blk + 2 * t + (x & 1) + 8 * (x >> 1);
#pragma unroll
        for (int i = 0; i < VP; ++i)
          vraw[x][i] = r < rend ? *reinterpret_cast<const uint4*>((decltype(has_new)::value && r == new_r)
                                                                      ? vn_row + i * 128 + g * 16
                                                                      : vb + ((x & 1) + 8 * (x >> 1)) * ROW_BYTES + i * 128)
                                : make_uint4(0, 0, 0, 0);
      }
      // S^T for the two 8-row halves of the block
      float sc[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) sc[j][e] = 0.f;
#pragma unroll
        for (int i = 0; i < KP; ++i) {
          mma_bf16_16816(sc[j], qa[2 * i][0], 0u, qa[2 * i][1], 0u, kraw[j][i].x, kraw[j][i].y);
          mma_bf16_16816(sc[j], qa[2 * i + 1][0], 0u, qa[2 * i + 1][1], 0u, kraw[j][i].z, kraw[j][i].w);
        }
      }
      // online softmax for head g over rows blk + 8j + 2t + {0, 1}
      float tv[4];
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int r = blk + 8 * j + 2 * t + e;
          tv[2 * j + e] = r < rend ? sc[j][e] * scale2 : -INFINITY;
        }
      float mx = fmaxf(fmaxf(tv[0], tv[1]), fmaxf(tv[2], tv[3]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mn = fmaxf(m_run, mx);
      const float mu = (mn == -INFINITY) ? 0.f : mn;
      const float corr = exp2f(m_run - mu);
      float pw[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) pw[e] = exp2f(tv[e] - mu);
      l_run = l_run * corr + ((pw[0] + pw[1]) + (pw[2] + pw[3]));
      m_run = mn;
      // rescale O^T: its columns are heads 2t, 2t+1, whose factors live in lanes 8t and 8t + 4
      const float ca = __shfl_sync(0xffffffffu, corr, 8 * t);
      const float cb = __shfl_sync(0xffffffffu, corr, 8 * t + 4);
      if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          o[mb][0] *= ca; o[mb][1] *= cb; o[mb][2] *= ca; o[mb][3] *= cb;
        }
      }
      const uint32_t pb0 = pack_bf16(pw[0], pw[1]);   // rows 2t, 2t+1
      const uint32_t pb1 = pack_bf16(pw[2], pw[3]);   // rows 2t+8, 2t+9
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) {
        uint32_t a[4];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int e = hf * MB + mb, pc = e >> 3, wi = (e & 7) >> 1;
          const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
          a[hf] = __byte_perm(word_of(vraw[0][pc], wi), word_of(vraw[1][pc], wi), sel);       // rows 2t, 2t+1
          a[2 + hf] = __byte_perm(word_of(vraw[2][pc], wi), word_of(vraw[3][pc], wi), sel);   // rows 2t+8, 2t+9
        }
        mma_bf16_16816(o[mb], a[0], a[1], a[2], a[3], pb0, pb1);
      }
      if (!PAGED) {
        kb += kAttnWarps * kBlk * ROW_BYTES;
        vb += kAttnWarps * kBlk * ROW_BYTES;
      }
    }

    };
    if (new_r >= rbeg && new_r < rend) rows_loop(std::true_type{}); else rows_loop(std::false_type{});

    // merge the four warps (same partial format as the scalar kernel)
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (t == 0 && g < G) { sm_m[warp][g] = m_run; sm_l[warp][g] = l_run; }
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int head = 2 * t + (e & 1);
        if (head < G) sm_acc[warp][head][pd(mb, e >> 1, g)] = o[mb][e];
      }
    __syncthreads();
    for (int i = tid; i < G * D; i += kAttnThreads) {
      const int hh = i / D, dd = i % D;
      float M = -INFINITY;
#pragma unroll
      for (int x = 0; x < kAttnWarps; ++x) M = fmaxf(M, sm_m[x][hh]);
      float a = 0.f, ll = 0.f;
#pragma unroll
      for (int x = 0; x < kAttnWarps; ++x) {
        const float mx = sm_m[x][hh];
        const float w = (mx == -INFINITY) ? 0.f : exp2f(mx - M);
        a = fmaf(w, sm_acc[x][hh][dd], a);
        ll = fmaf(w, sm_l[x][hh], ll);
      }
      if (s_direct >= 0) {
        // the unit's only item: Eq. 1 over the whole segment, as in the scalar kernel
        store_out(out + ((size_t)s_direct * G + hh) * D + dd, ll > 0.f ? a / ll : 0.f);
        continue;
      }
      p.part_acc[((size_t)item * G + hh) * D + dd] = a;
      if (dd == 0) {
        p.part_ml[((size_t)item * G + hh) * 2 + 0] = M;
        p.part_ml[((size_t)item * G + hh) * 2 + 1] = ll;
      }
    }
  }
}

// One block per (view unit, query head of the group): merge the unit's partials.  First the block finds
// the largest running maximum, then each warp accumulates every fourth partial against it (independent
// loads, fixed order), and the four warps are summed in shared memory.
constexpr int kCombineThreads = 256;
constexpr int kCombineWarps = kCombineThreads / 32;
constexpr int kCombineStage = 1024;     // partial results weighted per round (one round up to 524288 rows)

// One block per (view unit, query head of the group).  The weights exp2(m_i - M) of the unit's partial results
// are computed once, by all threads, into shared memory; the accumulation loop then has nothing but independent
// 16-byte loads in it (a long unit has over a hundred partials and one block: its latency is the kernel's).
// PRE: partial outputs a warp loads ahead of the weights (8: 64 registers, four blocks per SM (the lean one: six), for grids that are
// resident at once anyway -- it takes two round trips to L2 off the merge; 0: the lean variant for many thousands of
// blocks, most of them with nothing to merge).
template <typename T, int D, int G, int PRE>
__global__ void __launch_bounds__(kCombineThreads, PRE > 0 ? 4 : 6) decode_combine_kernel(DeviceProblem p,
                                                                         const int32_t* __restrict__ lengths,
                                                                         int fused_step, T* __restrict__ out) {
  constexpr int EPL = D / 32;
  __shared__ float s_red[kCombineWarps];
  __shared__ float s_l[kCombineWarps];
  __shared__ float s_w[kCombineStage];
  __shared__ __align__(16) float s_acc[kCombineWarps][D];
  // Lengths, capacities and the item table are not written by the attention kernel before this one: they are read
  // before the wait, under that kernel's tail (the lengths were last written by this kernel's previous launch or by
  // an append, both complete before the attention kernel let this one start).
  const int u = blockIdx.x / G, g = blockIdx.x % G;     // u: view unit
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = view_unit(p, u);
  int len = p.len[unit];
  const bool grown = fused_step && len < p.cap[unit];   // the attention pass appends the new token's row
  const int len_next = len + (grown ? 1 : 0);
  len = len_next;
  if (lengths) len = min(max(lengths[u], 0), len);
  // the unit's items that hold rows (the table also numbers the reserve for appended tokens)
  const int i0 = p.dec_off[lm_index(p, unit)], i1 = i0 + (len + kDecodeChunk - 1) / kDecodeChunk;
  grid_dependency_wait();
  grid_launch_dependents();
  if (i1 - i0 != 1) {                                   // a unit of one item has its output from the attention kernel
  const float2* ml = reinterpret_cast<const float2*>(p.part_ml);
  const int n = i1 - i0;
  // Issued together, right after the wait: this thread's (max, sum) pair and this warp's first kPre partial outputs
  // (they do not depend on the weights), so that the merge costs two round trips to L2 instead of four.
  constexpr int kPre = PRE;
  using Vec = typename std::conditional<EPL == 4, float4, float2>::type;
  Vec pre[kPre > 0 ? kPre : 1];
#pragma unroll
  for (int q = 0; q < kPre; ++q) {
    const int j = warp + q * kCombineWarps;
    if (j < n) pre[q] = *reinterpret_cast<const Vec*>(p.part_acc + ((size_t)(i0 + j) * G + g) * D + lane * EPL);
  }
  const float2 v0 = tid < n ? ml[(size_t)(i0 + tid) * G + g] : make_float2(-INFINITY, 0.f);
  float M = v0.x;
  for (int i = i0 + tid + kCombineThreads; i < i1; i += kCombineThreads) M = fmaxf(M, ml[(size_t)i * G + g].x);
  M = warp_max(M);
  if (lane == 0) s_red[warp] = M;
  __syncthreads();
  M = s_red[0];
#pragma unroll
  for (int w = 1; w < kCombineWarps; ++w) M = fmaxf(M, s_red[w]);
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  float L = 0.f;
  auto add = [&](float wgt, const Vec& t) {
    if constexpr (EPL == 4) {
      acc[0] = fmaf(wgt, t.x, acc[0]); acc[1] = fmaf(wgt, t.y, acc[1]);
      acc[2] = fmaf(wgt, t.z, acc[2]); acc[3] = fmaf(wgt, t.w, acc[3]);
    } else {
      acc[0] = fmaf(wgt, t.x, acc[0]); acc[1] = fmaf(wgt, t.y, acc[1]);
    }
  };
  for (int c0 = i0; c0 < i1; c0 += kCombineStage) {
    const int cn = min(kCombineStage, i1 - c0);
    __syncthreads();                                    // the previous round's weights have been used
    for (int j = tid; j < cn; j += kCombineThreads) {
      const float2 v = (c0 == i0 && j == tid) ? v0 : ml[(size_t)(c0 + j) * G + g];
      const float wgt = (v.x == -INFINITY) ? 0.f : exp2f(v.x - M);
      s_w[j] = wgt;
      L = fmaf(wgt, v.y, L);
    }
    __syncthreads();
    int j = warp;                                       // every warp adds its partials in ascending order
    if (c0 == i0) {
#pragma unroll
      for (int q = 0; q < kPre; ++q, j += kCombineWarps)
        if (j < cn) add(s_w[j], pre[q]);
    }
#pragma unroll 8
    for (; j < cn; j += kCombineWarps)
      add(s_w[j], *reinterpret_cast<const Vec*>(p.part_acc + ((size_t)(c0 + j) * G + g) * D + lane * EPL));
  }
  L = warp_sum(L);
#pragma unroll
  for (int e = 0; e < EPL; ++e) s_acc[warp][lane * EPL + e] = acc[e];
  if (lane == 0) s_l[warp] = L;
  __syncthreads();
  if (tid < D) {
    float Lt = 0.f, a = 0.f;
#pragma unroll
    for (int w = 0; w < kCombineWarps; ++w) {
      Lt += s_l[w];
      a += s_acc[w][tid];
    }
    store_out(out + ((size_t)u * G + g) * D + tid, Lt > 0.f ? a / Lt : 0.f);
  }
  }
  // fused step: the last of the unit's G blocks (each has read the old length by now) raises the length
  if (fused_step && tid == 0) {
    if (atomicAdd(&p.step_cnt[unit], 1) == G - 1) {
      p.step_cnt[unit] = 0;
      // (a recorded device error -- a paged cache whose pool ran dry under this very step -- freezes the lengths:
      // no row is counted whose page may not exist)
      if (grown) { if (p.page_rows == 0 || *p.status == 0) p.len[unit] = len_next; }
      else set_status(p.status, TASKKV_ESTATE);
    }
  }
}

template <typename T, int D, int G>
cudaError_t launch_typed(const DeviceProblem& p, const void* q, const int32_t* lengths, const void* k_new,
                         const void* v_new, void* out, cudaStream_t s, int early) {
  const unsigned char* kn = static_cast<const unsigned char*>(k_new);
  const unsigned char* vn = static_cast<const unsigned char*>(v_new);
  // persistent blocks: 16 per SM (measured best on B200 with 512-row items)
  int64_t grid = p.max_items < 148 * 16 ? p.max_items : 148 * 16;
  if (grid < 1) grid = 1;
  cudaError_t e;
  {
    LaunchScope ls(K_DECODE_ATTN, s);
    if (p.page_rows > 0) {
      if constexpr (sizeof(T) == 2)
        e = launch_dependent(decode_attn_mma_kernel<D, G, true>, (unsigned)grid, kAttnThreads, s, p, static_cast<const T*>(q), lengths, kn, vn, static_cast<T*>(out), early);
      else
        e = launch_dependent(decode_attn_kernel<T, D, G, true>, (unsigned)grid, kAttnThreads, s, p, static_cast<const T*>(q), lengths, kn, vn, static_cast<T*>(out), early);
    } else {
      if constexpr (sizeof(T) == 2)
        e = launch_dependent(decode_attn_mma_kernel<D, G, false>, (unsigned)grid, kAttnThreads, s, p, static_cast<const T*>(q), lengths, kn, vn, static_cast<T*>(out), early);
      else
        e = launch_dependent(decode_attn_kernel<T, D, G, false>, (unsigned)grid, kAttnThreads, s, p, static_cast<const T*>(q), lengths, kn, vn, static_cast<T*>(out), early);
    }
  }
  if (e != cudaSuccess) return e;
  {
    LaunchScope ls(K_DECODE_COMBINE, s);
    // up to 16 blocks per SM: the variant that loads ahead (its blocks are resident within a few waves)
    if ((int64_t)p.view_U * G <= 148 * 16)
      e = launch_dependent(decode_combine_kernel<T, D, G, 8>, (unsigned)(p.view_U * G), kCombineThreads, s, p, lengths,
                           k_new != nullptr ? 1 : 0, static_cast<T*>(out));
    else
      e = launch_dependent(decode_combine_kernel<T, D, G, 0>, (unsigned)(p.view_U * G), kCombineThreads, s, p, lengths,
                           k_new != nullptr ? 1 : 0, static_cast<T*>(out));
  }
  return e;
}

template <typename T, int D>
cudaError_t launch_group(const DeviceProblem& p, const void* q, const int32_t* lengths, const void* k_new,
                         const void* v_new, void* out, cudaStream_t s, int early) {
  switch (p.G) {
    case 1: return launch_typed<T, D, 1>(p, q, lengths, k_new, v_new, out, s, early);
    case 2: return launch_typed<T, D, 2>(p, q, lengths, k_new, v_new, out, s, early);
    case 4: return launch_typed<T, D, 4>(p, q, lengths, k_new, v_new, out, s, early);
    case 8: return launch_typed<T, D, 8>(p, q, lengths, k_new, v_new, out, s, early);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_decode(const DeviceProblem& p, int dtype, const void* q, const int32_t* lengths,
                          const void* k_new, const void* v_new, void* out, cudaStream_t s, bool early_unit_data) {
  // Reading lengths and page tables before the dependency wait is sound only if the kernel before this one in the
  // stream does not write them for these units; a caller's array of lengths is never read early.
  const int early = (early_unit_data && lengths == nullptr) ? 1 : 0;
  if (dtype == TASKKV_F32)
    return p.d == 64 ? launch_group<float, 64>(p, q, lengths, k_new, v_new, out, s, early)
                     : launch_group<float, 128>(p, q, lengths, k_new, v_new, out, s, early);
  return p.d == 64 ? launch_group<__nv_bfloat16, 64>(p, q, lengths, k_new, v_new, out, s, early)
                   : launch_group<__nv_bfloat16, 128>(p, q, lengths, k_new, v_new, out, s, early);
}

}  // namespace taskkv
