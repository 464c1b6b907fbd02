// Observation-window scores (Eq. 12, Eq. 13) with K read once: the raw scores of a whole unit stay in
// tensor memory between the two steps of the softmax.  For bf16 inputs with G*L = 32 window rows and
// sequences of up to 16 x 2048 keys.
//
// Eq. 13 sums the rows of the window's softmax, so every row's normaliser (over all N keys) is needed before
// any column can be finished.  The two-launch kernel of window_score_tc.cu reads K a second time for that.
// Here a thread-block cluster of T CTAs (T = 1, 2, 4, 8 or 16, the smallest that holds the sequence) owns one unit
// at a time; CTA c takes the c-th slice of the unit's 128-key tiles (at most 16 of them) and keeps
// S^T[key, row] = K Q^T of every tile in its own 32 columns of TMEM: 16 tiles x 32 columns x 128 lanes = all 512
// columns.  Per unit:
//   step 1  as each tile's MMAs complete, an epilogue warp replaces its scores in place (tcgen05.ld, ex2,
//           tcgen05.st) by e = exp2(s - c_row) and adds them into per-thread row sums (a TMEM lane is a key;
//           c_row is the score of one visible key of the warp, so the sum holds a term equal to 1 and loses
//           nothing that matters to underflow; should a term come near the top of the fp32 range, or should
//           the warp's reference key fall into the causally masked tail, the warp walks its tiles again with
//           its exact row maxima); masked scores become 0;
//   exchange  the warps' partial (c, sum) pairs are merged per CTA and sent to every CTA of the cluster
//           through distributed shared memory (st.async completing bytes on the receiver's mbarrier);
//   step 2  every warp folds the T pairs of each row into the row's offset, turns it into one weight per row,
//           w = exp2(c_row - offset_row), walks its tiles in TMEM again and writes C[key] = sum_rows e w
//           (no second exponential); each tile's columns are then handed back to the MMA issuer for the
//           next unit.
// K tiles of the next unit keep streaming into the shared-memory ring during exchange and step 2.
// Warp roles: 0 TMA producer, 1 MMA issuer, 2-9 epilogue (two groups of four, alternating tiles).
// Every wait inside the pipeline is bounded; after a time-out the CTA stops, its cluster peers run into
// their own limits, and all of them meet at the closing cluster barrier, so no CTA exits while a peer may
// still write into its shared memory.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace taskkv {

using namespace tc;

namespace {

constexpr int kTile = 128;          // keys per tile (UMMA M)
constexpr int kRows = 32;           // window rows = UMMA N = TMEM columns of one tile
constexpr int kSlots = 16;          // tiles a CTA holds in TMEM
constexpr int kStages = 6;          // K tiles in flight per CTA
constexpr int kEpiWarps = 8;
constexpr int kThreads = 320;
constexpr int kMaxTeam = 16;        // largest cluster
constexpr int kMaxSeq = 8;          // sequences per launch
constexpr uint32_t kTmemCols = 512;

struct ResMaps {
  CUtensorMap k[kMaxSeq];   // [units * N][d] of each sequence
  CUtensorMap q[kMaxSeq];   // [units * 32][d]
};
struct ResArgs {
  int n_seq;                // sequences in this launch
  int n_items;              // (sequence, unit) pairs
  int steps;                // items of the busiest cluster
  int u0[kMaxSeq];          // first unit of each sequence
  int N[kMaxSeq];           // sequence length
  int tiles[kMaxSeq];       // 128-key tiles per unit
  int item_off[kMaxSeq + 1];
};

struct Item {
  int seq, lu, t0, nt;
  bool valid;
};
// Item k of this CTA's cluster and the CTA's slice of its tiles.
__device__ __forceinline__ Item decode_item(const ResArgs& a, int k, int cluster, int n_clusters, int rank, int team) {
  Item it;
  const int i = cluster + k * n_clusters;
  it.valid = i < a.n_items;
  it.seq = 0;
#pragma unroll
  for (int s = 1; s < kMaxSeq; ++s)
    if (s < a.n_seq && i >= a.item_off[s]) it.seq = s;
  it.lu = it.valid ? i - a.item_off[it.seq] : 0;
  const int tiles = a.tiles[it.seq];
  it.t0 = rank * tiles / team;
  it.nt = it.valid ? (rank + 1) * tiles / team - it.t0 : 0;
  return it;
}

struct ResLayout {
  int tile_bytes, q_block_bytes;
  int off_q, off_part, off_x, off_ref, off_off, off_mod, off_bars;
  int total;
};
inline ResLayout make_layout(int D) {
  ResLayout l;
  const int KB = D / 64;
  l.tile_bytes = KB * kTile * 128;
  l.q_block_bytes = KB * kRows * 128;
  l.off_q = kStages * l.tile_bytes;
  l.off_part = l.off_q + 2 * l.q_block_bytes;
  l.off_x = l.off_part + 2 * kEpiWarps * kRows * (int)sizeof(float2);
  l.off_ref = l.off_x + 2 * kMaxTeam * kRows * (int)sizeof(float2);
  l.off_off = l.off_ref + kEpiWarps * kRows * (int)sizeof(float);
  l.off_mod = l.off_off + kEpiWarps * kRows * (int)sizeof(float);
  l.off_bars = l.off_mod + kRows * (int)sizeof(int);
  l.total = l.off_bars + 512 + 1024;
  return l;
}

enum : int {
  B_FULL = 0, B_EMPTY = 6, B_QFULL = 12, B_QEMPTY = 14, B_TFULL = 16, B_TEMPTY = 32, B_PART = 48, B_X = 50,
  B_COUNT = 52
};

// Reduction of 32 per-lane values across the 32 lanes of a warp: on return v[0] of lane i holds
// op over all lanes of their v[i].  31 shuffles; the order of the operations is fixed.
template <typename Op>
__device__ __forceinline__ void warp_transpose_reduce(float (&v)[32], int lane, Op op) {
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const bool up = (lane & s) != 0;
#pragma unroll
    for (int i = 0; i < s; ++i) {
      const float send = up ? v[i] : v[i + s];
      const float keep = up ? v[i + s] : v[i];
      v[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, s));
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
window_res_kernel(const __grid_constant__ ResMaps maps, DeviceProblem p, const __grid_constant__ ResArgs a,
                  ResLayout lay) {
  constexpr int KB = D / 64;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* sK = smem;                                          // [stages][KB][128 keys][128 B]
  unsigned char* sQ = smem + lay.off_q;                              // [2][KB][32 rows][128 B]
  float2* sPart = reinterpret_cast<float2*>(smem + lay.off_part);    // [2][8 warps][32 rows]  (c, sum)
  float2* sX = reinterpret_cast<float2*>(smem + lay.off_x);          // [2][16 CTAs][32 rows]  (c, sum)
  float* sRef = reinterpret_cast<float*>(smem + lay.off_ref);        // [8 warps][32 rows]  the warp's c
  float* sOff = reinterpret_cast<float*>(smem + lay.off_off);        // [8 warps][32 rows]  the rows' weights
  int* sMod = reinterpret_cast<int*>(smem + lay.off_mod);            // [32 rows]  row % L
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + lay.off_bars);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = p.L;
  const int team = (int)cluster_nctarank();
  const int rank = (int)cluster_ctarank();
  const int cluster = (int)blockIdx.x / team;
  const int n_clusters = (int)gridDim.x / team;
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(BAR(B_FULL + i), 1); mbar_init(BAR(B_EMPTY + i), 1); }
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(BAR(B_TFULL + i), 1);
      mbar_init(BAR(B_TEMPTY + i), 4);     // the four warps of the group that reads the tile
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(B_QFULL + i), 1);
      mbar_init(BAR(B_QEMPTY + i), 1);
      mbar_init(BAR(B_PART + i), kEpiWarps);
      mbar_init(BAR(B_X + i), 1);          // the local arrive that states the byte count; peers complete bytes
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid >= 32 && tid < 64) sMod[tid - 32] = (tid - 32) % L;
  if (warp == 1) {
    tc_alloc(smem_u32(s_tmem), kTmemCols);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // no peer may send to this CTA's barriers before they exist
  cluster_sync_all();
  const uint32_t tmem_base = *s_tmem;
  const float scale2 = kLog2e * rsqrtf((float)D);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0, qb = 0;
    uint32_t phase = 0, qphase[2] = {0, 0};
    bool ok = true;
    for (int k = 0; k < a.steps && ok; ++k) {
      const Item it = decode_item(a, k, cluster, n_clusters, rank, team);
      if (it.nt == 0) continue;
      const int N = a.N[it.seq];
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QEMPTY + qb), qphase[qb] ^ 1, s_abort));
      if (!ok) break;
      if (elect_one()) {
        mbar_expect_tx(BAR(B_QFULL + qb), (uint32_t)lay.q_block_bytes);
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d(smem_u32(sQ + (size_t)qb * lay.q_block_bytes + (size_t)kb * kRows * 128), &maps.q[it.seq],
                      kb * 64, it.lu * kRows, BAR(B_QFULL + qb));
      }
      __syncwarp();
      qphase[qb] ^= 1;
      qb ^= 1;
      for (int t = 0; t < it.nt; ++t) {
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_EMPTY + stage), phase ^ 1, s_abort));
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(BAR(B_FULL + stage), (uint32_t)lay.tile_bytes);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
            tma_load_2d(smem_u32(sK + (size_t)stage * lay.tile_bytes + (size_t)kb * kTile * 128), &maps.k[it.seq],
                        kb * 64, it.lu * N + (it.t0 + t) * kTile, BAR(B_FULL + stage));
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    // every tcgen05.commit aimed at this CTA's barriers must have arrived before the CTA exits
    for (int i = 0; i < kStages && ok; ++i) {
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_EMPTY + stage), phase ^ 1, s_abort));
      if (++stage == kStages) { stage = 0; phase ^= 1; }
    }
    for (int i = 0; i < 2 && ok; ++i, qb ^= 1)
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QEMPTY + qb), qphase[qb] ^ 1, s_abort));
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer: tile t of a unit goes to TMEM
    // columns [32 t, 32 t + 32); the columns are free again when the tile's step 2 is done
    int stage = 0, qb = 0;
    uint32_t sphase = 0, qphase[2] = {0, 0};
    uint32_t tphase = 0;                       // bit t: phase of TEMPTY[t] this warp has consumed
    const uint32_t idesc = instr_desc(128, kRows);
    const uint64_t desc_hi = smem_desc(0);
    bool ok = true;
    for (int k = 0; k < a.steps && ok; ++k) {
      const Item it = decode_item(a, k, cluster, n_clusters, rank, team);
      if (it.nt == 0) continue;
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QFULL + qb), qphase[qb], s_abort));
      if (!ok) break;
      qphase[qb] ^= 1;
      const uint32_t q_lo = smem_u32(sQ + (size_t)qb * lay.q_block_bytes) >> 4;
      for (int t = 0; t < it.nt; ++t) {
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_FULL + stage), sphase, s_abort) &&
                                         mbar_wait(BAR(B_TEMPTY + t), ((tphase >> t) & 1u) ^ 1u, s_abort));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(t * kRows);
        const uint32_t k_lo = smem_u32(sK + (size_t)stage * lay.tile_bytes) >> 4;
        if (elect_one()) {
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t ad = desc_hi | (uint64_t)(k_lo + (uint32_t)((kb * kTile * 128 + kk * 32) >> 4));
              const uint64_t bd = desc_hi | (uint64_t)(q_lo + (uint32_t)((kb * kRows * 128 + kk * 32) >> 4));
              tc_mma(d_tmem, ad, bd, idesc, (kb | kk) ? 1u : 0u);
            }
          tc_commit(BAR(B_EMPTY + stage));
          tc_commit(BAR(B_TFULL + t));
        }
        __syncwarp();
        tphase ^= 1u << t;
        if (++stage == kStages) { stage = 0; sphase ^= 1; }
      }
      if (!ok) break;
      if (elect_one()) tc_commit(BAR(B_QEMPTY + qb));
      __syncwarp();
      qb ^= 1;
    }
  } else {
    // ------------------------------------------------------------ epilogue: warps 2-5 take the even tiles of
    // the slice, warps 6-9 the odd ones; a TMEM lane is a key, a column a window row
    const int ew = warp - 2;                        // 0..7
    const int grp = ew >> 2;
    const int quad = warp & 3;                      // TMEM lane quadrant this warp may access
    float* myRef = sRef + ew * kRows;
    float* myW = sOff + ew * kRows;
    uint32_t fphase = 0;                            // bit t: phase of TFULL[t] to wait for
    int nu = 0;                                     // units this CTA has been through
    bool ok = true;
    for (int k = 0; k < a.steps && ok; ++k) {
      const Item it = decode_item(a, k, cluster, n_clusters, rank, team);
      if (!it.valid) continue;
      const int u = a.u0[it.seq] + it.lu;
      const int N = a.N[it.seq];
      const int buf = nu & 1;
      const uint32_t uphase = (uint32_t)((nu >> 1) & 1);
      const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
      auto key_of = [&](int t) { return (it.t0 + t) * kTile + quad * 32 + lane; };   // this thread's key in tile t
      // bit i: window row i may see this thread's key of tile t (Eq. 12: key <= N - L + i % L, and a key at all)
      auto in_tail = [&](int t) { return (it.t0 + t) * kTile + kTile - 1 > N - L; };   // some key masked for some row
      auto visible_rows = [&](int t) -> uint32_t {
        if (!in_tail(t)) return 0xffffffffu;
        const int j = key_of(t);
        uint32_t vm = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) vm |= (uint32_t)(j < N && j <= N - L + sMod[i]) << i;
        return vm;
      };

      // ---- step 1: every score becomes e = exp2(s - c_row) in place; per-thread row sums of e.
      // c_row is the score of the warp's first key in its first tile (lane 0 broadcasts its 32 values).
      float z[32], cs[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) { z[i] = 0.f; cs[i] = 0.f; }
      const bool mine = grp < it.nt;                // this warp has at least one tile
      int t_raw = -1;                               // first tile left as raw scores: the exact walk below is needed
      bool have_ref = false;
      for (int t = grp; t < it.nt; t += 2) {
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_TFULL + t), (fphase >> t) & 1u, s_abort));
        if (!ok) break;
        tc_fence_after();
        if (t_raw >= 0) continue;                   // only wait for the rest
        if (!have_ref && in_tail(t)) {
          t_raw = t;                                // the reference key must be visible to every row
          continue;
        }
        const uint32_t vm = visible_rows(t);
        uint32_t r[32];
        tc_ld32(lane_addr + (uint32_t)(t * kRows), r);
        tc_wait_ld();
        if (!have_ref) {
          have_ref = true;
          if (lane == 0) {
#pragma unroll
            for (int i = 0; i < 32; ++i) myRef[i] = __uint_as_float(r[i]) * scale2;
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 c4 = *reinterpret_cast<const float4*>(myRef + i);
            cs[i] = c4.x; cs[i + 1] = c4.y; cs[i + 2] = c4.z; cs[i + 3] = c4.w;
          }
        }
        float mx[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float e = ex2(fmaf(__uint_as_float(r[i]), scale2, -cs[i]));
          e = (vm >> i) & 1u ? e : 0.f;
          mx[i & 3] = fmaxf(mx[i & 3], e);
          z[i] += e;
          r[i] = __float_as_uint(e);
        }
        // a term near the top of the fp32 range (or a NaN): the sums over keys, lanes, warps and CTAs would not hold
        const bool big = !(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) < 1.0e30f);
        if (__any_sync(0xffffffffu, big)) {
          t_raw = t;
          continue;
        }
        tc_st32(lane_addr + (uint32_t)(t * kRows), r);
      }
      if (!ok) break;
      if (t_raw >= 0) {
        // Exact walk (rare: a key more than 2^100 above the warp's reference in some row, or a reference tile in the
        // masked tail).  Tiles before t_raw hold e relative to cs, the others raw scores.  First the rows' maxima over
        // the warp's visible keys, then every tile is (re)written relative to them.
        tc_wait_st();
        float m[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) m[i] = -INFINITY;
        for (int t = grp; t < it.nt; t += 2) {
          const uint32_t vm = visible_rows(t);
          const bool raw = t >= t_raw;
          uint32_t r[32];
          tc_ld32(lane_addr + (uint32_t)(t * kRows), r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float x = __uint_as_float(r[i]);
            const float v = raw ? x * scale2 : cs[i] + lg2(x);      // lg2(0) = -inf: a masked or vanished term
            if ((vm >> i) & 1u) m[i] = fmaxf(m[i], v);
          }
        }
        warp_transpose_reduce(m, lane, [](float x, float y) { return fmaxf(x, y); });
        __syncwarp();
        myRef[lane] = m[0];                         // -inf: no key of this warp is visible to the row
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float c = myRef[i];
          const float c_new = c > -INFINITY ? c : 0.f;
          m[i] = ex2(cs[i] - c_new);                // factor for the tiles that already hold e (at most 1)
          cs[i] = c_new;
          z[i] = 0.f;
        }
        for (int t = grp; t < it.nt; t += 2) {
          const uint32_t vm = visible_rows(t);
          const bool raw = t >= t_raw;
          uint32_t r[32];
          tc_ld32(lane_addr + (uint32_t)(t * kRows), r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float x = __uint_as_float(r[i]);
            float e = raw ? ex2(fmaf(x, scale2, -cs[i])) : x * m[i];
            e = (vm >> i) & 1u ? e : 0.f;
            z[i] += e;
            r[i] = __float_as_uint(e);
          }
          tc_st32(lane_addr + (uint32_t)(t * kRows), r);
        }
      } else if (!mine) {
        __syncwarp();
        myRef[lane] = -INFINITY;                    // no tile: nothing to contribute
        __syncwarp();
      }
      // lane i <- the warp's sum of row i
      warp_transpose_reduce(z, lane, [](float x, float y) { return x + y; });
      const float my_c = myRef[lane];
      sPart[(buf * kEpiWarps + ew) * kRows + lane] = make_float2(my_c, z[0]);
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_PART + buf));

      // ---- exchange: warp 2 merges the CTA's eight partials and sends the pair of each row to every CTA
      if (ew == 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_PART + buf), uphase, s_abort));
        if (!ok) break;
        float M = -INFINITY, Z = 0.f;
#pragma unroll
        for (int w = 0; w < kEpiWarps; ++w) M = fmaxf(M, sPart[(buf * kEpiWarps + w) * kRows + lane].x);
#pragma unroll
        for (int w = 0; w < kEpiWarps; ++w) {
          const float2 o = sPart[(buf * kEpiWarps + w) * kRows + lane];
          if (o.x > -INFINITY) Z += o.y * ex2(o.x - M);
        }
        if (lane == 0) mbar_expect_tx(BAR(B_X + buf), (uint32_t)(team * kRows * (int)sizeof(float2)));
        const uint64_t word = (uint64_t)__float_as_uint(M) | ((uint64_t)__float_as_uint(Z) << 32);
        const uint32_t slot = smem_u32(sX + (buf * kMaxTeam + rank) * kRows + lane);
        for (int r = 0; r < team; ++r) st_async_b64(mapa(slot, (uint32_t)r), word, mapa(BAR(B_X + buf), (uint32_t)r));
      }
      ok = __all_sync(0xffffffffu, mbar_wait_cluster(BAR(B_X + buf), uphase, s_abort));
      if (!ok) break;
      {
        // lane = row: the T pairs -> the row's offset max + log2(sum) + log2(rows); a stored e of this warp then
        // weighs exp2(c - offset) in C
        float M = -INFINITY, Z = 0.f;
        for (int r = 0; r < team; ++r) M = fmaxf(M, sX[(buf * kMaxTeam + r) * kRows + lane].x);
        for (int r = 0; r < team; ++r) {
          const float2 o = sX[(buf * kMaxTeam + r) * kRows + lane];
          if (o.x > -INFINITY) Z += o.y * ex2(o.x - M);
        }
        const float off = M + lg2(Z) + 5.f;         // log2(32 rows)
        __syncwarp();
        myW[lane] = (Z > 0.f && my_c > -INFINITY) ? ex2(my_c - off) : 0.f;
        __syncwarp();
      }

      // ---- step 2: C[key] = sum over rows of e * weight; the tile's columns go back to the issuer
      tc_wait_st();
      for (int t = grp; t < it.nt; t += 2) {
        uint32_t r[32];
        tc_ld32(lane_addr + (uint32_t)(t * kRows), r);
        tc_wait_ld();
        float c4[4] = {0.f, 0.f, 0.f, 0.f};
        const float4* w4 = reinterpret_cast<const float4*>(myW);
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 w = w4[i >> 2];
          c4[0] = fmaf(__uint_as_float(r[i]), w.x, c4[0]);
          c4[1] = fmaf(__uint_as_float(r[i + 1]), w.y, c4[1]);
          c4[2] = fmaf(__uint_as_float(r[i + 2]), w.z, c4[2]);
          c4[3] = fmaf(__uint_as_float(r[i + 3]), w.w, c4[3]);
        }
        const int j = key_of(t);
        if (j < N) p.C[p.c_off[u] + j] = (c4[0] + c4[1]) + (c4[2] + c4[3]);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_TEMPTY + t));
      }
      for (int t = grp; t < it.nt; t += 2) fphase ^= 1u << t;
      ++nu;
    }
  }

  // ---------------------------------------------------------------- teardown
  if (*s_abort)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, kTmemCols);
  }
  if (tid == 0 && *s_abort) set_status(p.status, TASKKV_ETIMEOUT);
}

// Clusters of `team` CTAs of this kernel that the device runs at once (0: the cluster size is not available).
template <int D>
int max_clusters(int team, int smem) {
  static int cached[kMaxTeam + 1] = {0};
  static bool known[kMaxTeam + 1] = {false};
  if (known[team]) return cached[team];
  known[team] = true;
  int n = 0;
  if (cudaFuncSetAttribute(window_res_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess &&
      cudaFuncSetAttribute(window_res_kernel<D>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(team, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = team;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, window_res_kernel<D>, &cfg) != cudaSuccess) n = 0;
  }
  cudaGetLastError();
  cached[team] = n;
  return n;
}

inline int team_for(int max_tiles) {
  int team = 1;
  while (team * kSlots < max_tiles) team *= 2;
  return team;
}

inline int seq_team(int N) { return team_for((N + kTile - 1) / kTile); }

// One launch per cluster size in use and per eight sequences of it: a sequence is handled by the smallest cluster
// that holds it, so that short sequences of a ragged batch do not leave most CTAs of a large cluster without a tile.
template <int D>
cudaError_t launch_res_d(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0, int n_layers) {
  const ResLayout lay = make_layout(D);
  const int per_seq_all = p.R * p.n_kv;
  const int first = layer0 * p.n_kv;               // the launch covers units [first, first + per_seq) of every sequence
  const int per_seq = n_layers * p.n_kv;
  if (per_seq <= 0) return cudaSuccess;
  for (int team = 1; team <= kMaxTeam; team *= 2) {
    int b_next = 0;
    for (;;) {
      int seqs[kMaxSeq], nb = 0;
      while (b_next < h.batch && nb < kMaxSeq) {
        if (seq_team(h.seq_lens[b_next]) == team) seqs[nb++] = b_next;
        ++b_next;
      }
      if (nb == 0) break;
      const int n_cl = max_clusters<D>(team, lay.total);
      if (n_cl <= 0) return cudaErrorInvalidConfiguration;
      ResMaps maps;
      ResArgs a;
      a.n_seq = nb;
      a.item_off[0] = 0;
      for (int i = 0; i < kMaxSeq; ++i) {
        const int b = seqs[i < nb ? i : 0];                   // unused slots repeat the first sequence
        const int N = h.seq_lens[b];
        if (i >= nb) {
          maps.k[i] = maps.k[0];
          maps.q[i] = maps.q[0];
        } else {
          // h.k[b], h.q[b] point at layer h.base_layer
          const size_t skip = (size_t)(first - h.base_layer * p.n_kv);
          const char* kb = static_cast<const char*>(h.k[b]) + skip * (size_t)N * D * sizeof(__nv_bfloat16);
          const char* qb = static_cast<const char*>(h.q[b]) + skip * kRows * D * sizeof(__nv_bfloat16);
          if (!make_tensor_map_2d(&maps.k[i], kb, D, (uint64_t)per_seq * (uint64_t)N, kTile)) return cudaErrorUnknown;
          if (!make_tensor_map_2d(&maps.q[i], qb, D, (uint64_t)per_seq * (uint64_t)kRows, kRows))
            return cudaErrorUnknown;
        }
        a.u0[i] = b * per_seq_all + first;
        a.N[i] = N;
        a.tiles[i] = (N + kTile - 1) / kTile;
        a.item_off[i + 1] = a.item_off[i] + (i < nb ? per_seq : 0);
      }
      a.n_items = a.item_off[nb];
      const int clusters = a.n_items < n_cl ? a.n_items : n_cl;
      a.steps = (a.n_items + clusters - 1) / clusters;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(clusters * team, 1, 1);
      cfg.blockDim = dim3(kThreads, 1, 1);
      cfg.dynamicSmemBytes = lay.total;
      cfg.stream = s;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = team;
      attr.val.clusterDim.y = 1;
      attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      cudaError_t e;
      {
        LaunchScope ls(K_WINDOW_TC, s);
        e = cudaLaunchKernelEx(&cfg, window_res_kernel<D>, maps, p, a, lay);
      }
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

}  // namespace

// Whether the single-read kernel takes this problem: 32 window rows, every sequence within 16 CTAs x 16 tiles, and a
// device that co-schedules enough clusters of every size in use to fill three quarters of its SMs.
bool window_res_supported(const DeviceProblem& p, const WindowHostInfo& h) {
  if (p.rows != kRows || p.L > kRows || h.lse != nullptr) return false;
  int dev = 0, n_sm = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  const int smem = make_layout(p.d).total;
  bool checked[kMaxTeam + 1] = {false};
  for (int b = 0; b < h.batch; ++b) {
    const int tiles = (h.seq_lens[b] + kTile - 1) / kTile;
    if (tiles > kMaxTeam * kSlots) return false;
    const int team = team_for(tiles);
    if (checked[team]) continue;
    checked[team] = true;
    const int n_cl = p.d == 64 ? max_clusters<64>(team, smem) : max_clusters<128>(team, smem);
    if (n_cl * team * 4 < n_sm * 3) return false;
  }
  return true;
}

cudaError_t launch_window_scores_res(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0,
                                     int n_layers) {
  if (n_layers < 0) { layer0 = 0; n_layers = p.R; }
  return p.d == 64 ? launch_res_d<64>(p, h, s, layer0, n_layers) : launch_res_d<128>(p, h, s, layer0, n_layers);
}

}  // namespace taskkv
