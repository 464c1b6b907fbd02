// Observation-window scores (Eq. 12, Eq. 13) on the 5th-generation tensor cores,
// for bf16 inputs with G*L in {32, 64, 128} window rows.
//
// The contraction S = Q_win K^T is 2*G*L*d flop per key (32-128 flop per byte of
// K): too much for the CUDA cores next to an HBM-rate K stream, little for
// tcgen05.  Each CTA is a persistent, warp-specialised pipeline:
//   warp 0        TMA producer: K tiles of 128 keys (and the unit's Q rows) into
//                 128-byte-swizzled shared memory, completion on mbarriers
//   warps 1, 6    tcgen05.mma issuers, alternating tiles; accumulators in TMEM (four of
//                 them); tcgen05.commit frees the smem stage and hands the accumulator over
//   warps 2-5, 7-10  two epilogue groups, alternating tiles: tcgen05.ld, softmax arithmetic
//                 in fp32 registers
// (A third epilogue group, with one accumulator per group and a single issuer so that every accumulator
// keeps one issuer and one reader, was measured at the same speed with 128 rows and is not used.)
// Two passes (two launches), as Eq. 13 needs every row's normaliser before rows can be summed:
//   pass 1 (row statistics)  every epilogue warp keeps a running (max, exp-sum) per window row
//     over the keys it sees in a work item and stores it as the warp's own partial; a small
//     kernel folds the partials of a unit.  With up to 64 rows D[key, row] = K Q^T is used (a
//     TMEM lane is a key) and the warp's 32x32 block is transposed through shared memory;
//     with 128 rows the operands are swapped, D[row, key], and a lane owns a row outright.
//   pass 2 (scores)  D[key, row] = K Q^T: a TMEM lane is a key, so
//     C[key] = sum_rows exp2(s - max_row) / Z_row is a sum inside one thread.
// No warp ever waits for another epilogue warp.  Scores are kept in log2 units (scale
// log2(e)/sqrt(d)); exp is one ex2.approx.  Every wait is bounded: on time-out the CTA records
// TASKKV_ETIMEOUT, stops issuing work, releases its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace taskkv {

using namespace tc;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      cudaGetLastError();
  }
  return fn;
}

// 2-D bf16 tensor [rows_total][d], box of 64 elements x box_rows rows, 128-byte swizzle.
bool make_tensor_map_2d(CUtensorMap* map, const void* base, int d, uint64_t rows_total, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows_total};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

constexpr int kTile = 128;          // keys per tile (UMMA M in pass 2, key sub-tiles in pass 1)
constexpr int kMaxStages = 6;       // K tiles in flight per CTA (the count is fitted to shared memory)
constexpr int kEpiWarps = 8;        // two groups of four epilogue warps, alternating tiles
static_assert(kEpiWarps == kTcParts, "one partial-statistic slot per epilogue warp");
constexpr int kThreads = 352;       // warp 0 producer; 1, 6 MMA issuers; 2-5 and 7-10 epilogue groups
constexpr uint32_t kTmemCols = 512; // four accumulators of up to 128 columns

// Work items of one launch (one pass over up to kMaxSeq sequences): (sequence, unit, chunk of chunk_keys keys),
// numbered sequence-major, then unit-major: i = item_off[s] + unit * chunks[s] + chunk.  CTA c of a grid of g
// CTAs takes the items c, c + g, c + 2g, ...  Short sequences share a launch so that every SM has work.
constexpr int kMaxSeq = 8;
struct TcMaps {
  CUtensorMap k[kMaxSeq];   // [units * N][d] of each sequence
  CUtensorMap q[kMaxSeq];   // [units * rows][d]
};
struct TcArgs {
  int pass;                 // 1 = row statistics, 2 = scores
  int n_seq;                // sequences in this launch
  int n_local;              // units per sequence (layers * kv heads)
  int chunk_keys;           // keys per work item (multiple of 128)
  int steps;                // items of the busiest CTA
  // Prefix mode (the column sums of the full causal attention matrix, Eq. 1-2 of Sec. III-A): unit lu stands for the
  // 128 query rows [128 b, 128 b + 128) of query head lu / prefix_blocks, b = lu % prefix_blocks, as a window
  // over the first 128 (b + 1) keys of that head's KV head.  0: every unit has its own N keys and rows.
  int prefix_blocks;
  int group;                // query heads per KV head (prefix mode)
  int u0[kMaxSeq];          // first unit of each sequence
  int N[kMaxSeq];           // sequence length
  int chunks[kMaxSeq];      // work items per unit
  int item_off[kMaxSeq + 1];
};

struct Item {
  int seq, lu, ch;
  int N;                    // keys of the unit
  int krow0, qrow0;         // first row of the unit in the K and Q tensor maps
  bool valid;
};
__device__ __forceinline__ Item decode_item(const TcArgs& a, int k, int rows) {
  Item it;
  const int i = (int)blockIdx.x + k * (int)gridDim.x;
  it.valid = i < a.item_off[a.n_seq];
  it.seq = 0;
#pragma unroll
  for (int s = 1; s < kMaxSeq; ++s)
    if (s < a.n_seq && i >= a.item_off[s]) it.seq = s;
  const int local = it.valid ? i - a.item_off[it.seq] : 0;
  it.lu = local / a.chunks[it.seq];
  it.ch = local % a.chunks[it.seq];
  const int N = a.N[it.seq];
  if (a.prefix_blocks > 0) {
    const int head = it.lu / a.prefix_blocks, b = it.lu % a.prefix_blocks;
    it.N = (b + 1) * kTile;                 // may run past the sequence end: those rows and keys are neutralised
    it.krow0 = (head / a.group) * N;
    it.qrow0 = head * N + b * kTile;
    it.valid = it.valid && it.ch * a.chunk_keys < it.N;
  } else {
    it.N = N;
    it.krow0 = it.lu * N;
    it.qrow0 = it.lu * rows;
  }
  return it;
}

// Shared-memory plan, made on the host: the Q blocks and the per-warp areas scale with the number of
// window rows; what is left of the 227 KB goes to K stages (an even count, so that each stage is always
// consumed by the same issuer).
struct TcLayout {
  int stages;
  int tile_bytes, q_block_bytes;
  int off_q, off_stat, off_trans, off_bars;
  int total;
};

inline TcLayout make_layout(int D, int rows) {
  TcLayout l;
  const int KB = D / 64;
  l.tile_bytes = KB * kTile * 128;
  l.q_block_bytes = KB * rows * 128;
  const int stat = kEpiWarps * rows * (int)sizeof(float2);
  // with 128 rows pass 1 puts the window rows on the TMEM lanes and needs no transposition
  const int trans = rows == 128 ? 0 : kEpiWarps * 32 * 33 * (int)sizeof(float);
  const int bars = 512;
  const int budget = 232448 - 1024;     // dynamic shared memory of one CTA minus the alignment slack
  int stages = (budget - 2 * l.q_block_bytes - stat - trans - bars) / l.tile_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  l.stages = stages & ~1;
  l.off_q = l.stages * l.tile_bytes;
  l.off_stat = l.off_q + 2 * l.q_block_bytes;
  l.off_trans = l.off_stat + stat;
  l.off_bars = l.off_trans + trans;
  l.total = l.off_bars + bars + 1024;
  return l;
}

// barrier slots
enum : int {
  B_FULL = 0, B_EMPTY = 8, B_QFULL = 16, B_QEMPTY = 18, B_TFULL = 20, B_TEMPTY = 24, B_COUNT = 28
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
window_tc_kernel(const __grid_constant__ TcMaps maps, DeviceProblem p, const __grid_constant__ TcArgs a,
                 TcLayout lay) {
  constexpr int KB = D / 64;
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment: the swizzle pattern is a function of the address bits
  // (offset added to the array itself: a round trip through an integer would turn every access below into a
  // generic-address load or store)
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* sK = smem;                                         // [stages][KB][128 keys][128 B]
  unsigned char* sQ = smem + lay.off_q;                             // [2][KB][rows][128 B]
  float2* sStat = reinterpret_cast<float2*>(smem + lay.off_stat);   // [8 warps][rows]
  float* sTrans = reinterpret_cast<float*>(smem + lay.off_trans);   // [8 warps][32][33]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + lay.off_bars);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rows = p.rows;                  // 32, 64 or 128
  const int L = p.L;
  const int S = lay.stages;
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };

  if (tid == 0) {
    for (int i = 0; i < kMaxStages; ++i) { mbar_init(BAR(B_FULL + i), 1); mbar_init(BAR(B_EMPTY + i), 1); }
    for (int i = 0; i < 4; ++i) {
      mbar_init(BAR(B_TFULL + i), 1);
      mbar_init(BAR(B_TEMPTY + i), 4);     // the four warps of the group that reads the accumulator
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(B_QFULL + i), 1);
      mbar_init(BAR(B_QEMPTY + i), 2);     // both issuers release a Q block
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tc_alloc(smem_u32(s_tmem), kTmemCols);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const float scale2 = kLog2e * rsqrtf((float)D);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (whole warp, one lane issues)
    {
      int stage = 0, qb = 0;
      uint32_t phase = 0, qphase[2] = {0, 0};
      bool ok = true;
      for (int k = 0; k < a.steps && ok; ++k) {
        const Item it = decode_item(a, k, rows);
        if (!it.valid) continue;
        const int N = it.N;
        const int key0 = it.ch * a.chunk_keys;
        const int ntiles = (min(N, key0 + a.chunk_keys) - key0 + kTile - 1) / kTile;
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QEMPTY + qb), qphase[qb] ^ 1, s_abort));
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(BAR(B_QFULL + qb), (uint32_t)lay.q_block_bytes);
          for (int kb = 0; kb < KB; ++kb)
            tma_load_2d(smem_u32(sQ + (size_t)qb * lay.q_block_bytes + (size_t)kb * rows * 128), &maps.q[it.seq],
                        kb * 64, it.qrow0, BAR(B_QFULL + qb));
        }
        __syncwarp();
        qphase[qb] ^= 1;
        qb ^= 1;
        for (int t = 0; t < ntiles; ++t) {
          ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_EMPTY + stage), phase ^ 1, s_abort));
          if (!ok) break;
          if (elect_one()) {
            mbar_expect_tx(BAR(B_FULL + stage), (uint32_t)lay.tile_bytes);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
              tma_load_2d(smem_u32(sK + (size_t)stage * lay.tile_bytes + (size_t)kb * kTile * 128), &maps.k[it.seq],
                          kb * 64, it.krow0 + key0 + t * kTile, BAR(B_FULL + stage));
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1; }
        }
      }
      // Drain: every tcgen05.commit aimed at this CTA's barriers must have arrived before the CTA exits,
      // or it would land on the barriers of the next CTA that is given this shared memory.
      for (int i = 0; i < S && ok; ++i) {
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_EMPTY + stage), phase ^ 1, s_abort));
        if (++stage == S) { stage = 0; phase ^= 1; }
      }
      for (int i = 0; i < 2 && ok; ++i, qb ^= 1)
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QEMPTY + qb), qphase[qb] ^ 1, s_abort));
    }
  } else if (warp == 1 || warp == 6) {
    // ------------------------------------------------------------ MMA issuers: D[key, row] = K Q^T, both passes.
    // Two elected threads: the issue -> commit -> hand-over chain of one tile overlaps with the other's.
    // Tiles are numbered n = 0, 1, ... per CTA across items: issuer n & 1, smem stage n % stages, TMEM
    // accumulator n & 3 (read by epilogue group n & 1).
    // The per-tile bookkeeping is kept to counters that step by two (this issuer's tiles), and the
    // descriptors to one add on a precomputed low word: a lone warp issues an instruction only every few cycles.
    {
      const int me = warp == 1 ? 0 : 1;
      int qb = 0, tiles_before = 0;
      int stage = me, acc = me;                 // S is even: own stages me, me + 2, ...; accumulators me, me + 2
      uint32_t sphase = 0, aphase = 0;
      uint32_t qphase[2] = {0, 0};
      const uint32_t idesc = instr_desc(128, rows);
      const uint64_t desc_hi = smem_desc(0);    // everything but the start address
      bool ok = true;
      for (int k = 0; k < a.steps && ok; ++k) {
        const Item it = decode_item(a, k, rows);
        if (!it.valid) continue;
        const int N = it.N;
        const int key0 = it.ch * a.chunk_keys;
        const int ntiles = (min(N, key0 + a.chunk_keys) - key0 + kTile - 1) / kTile;
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QFULL + qb), qphase[qb], s_abort));
        if (!ok) break;
        qphase[qb] ^= 1;
        const uint32_t q_lo = smem_u32(sQ + (size_t)qb * lay.q_block_bytes) >> 4;
        const bool swap = a.pass == 1 && rows == 128;   // D[row, key] instead of D[key, row]
        for (int t = (me ^ tiles_before) & 1; t < ntiles; t += 2) {
          ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_FULL + stage), sphase, s_abort) &&
                                           mbar_wait(BAR(B_TEMPTY + acc), aphase ^ 1, s_abort));
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * 128u;
          const uint32_t k_lo = smem_u32(sK + (size_t)stage * lay.tile_bytes) >> 4;
          if (elect_one()) {
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint64_t ad = desc_hi | (uint64_t)(k_lo + (uint32_t)((kb * kTile * 128 + k * 32) >> 4));
                const uint64_t bd = desc_hi | (uint64_t)(q_lo + (uint32_t)((kb * rows * 128 + k * 32) >> 4));
                if (swap) tc_mma(d_tmem, bd, ad, idesc, (kb | k) ? 1u : 0u);
                else tc_mma(d_tmem, ad, bd, idesc, (kb | k) ? 1u : 0u);
              }
            tc_commit(BAR(B_EMPTY + stage));   // smem stage free once these MMAs have read it
            tc_commit(BAR(B_TFULL + acc));     // accumulator ready for the epilogue
          }
          __syncwarp();
          stage += 2;
          if (stage >= S) { stage -= S; sphase ^= 1; }
          acc ^= 2;
          if (acc == me) aphase ^= 1;
        }
        if (!ok) break;
        tiles_before += ntiles;
        if (elect_one()) tc_commit(BAR(B_QEMPTY + qb));   // this issuer is done with the Q block
        __syncwarp();
        qb ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: two groups of 4 warps (2-5 take
    // even tiles, 7-10 odd tiles); a TMEM lane is a key
    const int ew = warp < 6 ? warp - 2 : warp - 3;  // 0..7
    const int grp = ew >> 2;
    const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
    float* myStat = reinterpret_cast<float*>(sStat) + ew * rows;
    float* myT = sTrans + ew * (32 * 33);
    int n = 0;
    bool ok = true;
    // pass 2: the rows' offsets max + log2(sum) + log2(rows) of a unit (one subtraction then turns a raw score
    // into its share of C), lane i holding rows i, i + 32, ...; loaded one item ahead
    const float* stat_g = p.stat;
    float pre[4];
    auto fetch_stats = [&](int k) {
      const Item nx = decode_item(a, k, rows);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        pre[q] = (nx.valid && q * 32 + lane < rows) ? stat_g[(size_t)(a.u0[nx.seq] + nx.lu) * (2 * p.rows_pad) + q * 32 + lane]
                                                    : 0.f;
    };
    if (a.pass == 2) fetch_stats(0);
    for (int k = 0; k < a.steps && ok; ++k) {
      const Item it = decode_item(a, k, rows);
      if (!it.valid) {
        if (a.pass == 2) fetch_stats(k + 1);   // (prefix mode skips items in mid-run: keep the prefetch one ahead)
        continue;
      }
      const int u = a.u0[it.seq] + it.lu;
      const int N = it.N;
      const int key0 = it.ch * a.chunk_keys;
      const int ntiles = (min(N, key0 + a.chunk_keys) - key0 + kTile - 1) / kTile;
      // pass 1 state: after the transposition lane = window row (rg * 32 + lane); raw (unscaled) maxima
      float m_run[4], z_run[4];
#pragma unroll
      for (int rg = 0; rg < 4; ++rg) { m_run[rg] = -INFINITY; z_run[rg] = 0.f; }
      if (a.pass == 2) {
        __syncwarp();                       // the previous item's readers of myStat are done
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (q * 32 + lane < rows) myStat[q * 32 + lane] = pre[q];
        __syncwarp();
        fetch_stats(k + 1);                 // in flight while this item's tiles are worked on
      }
      // Which of the item's tiles this group takes depends on how many tiles the CTA has seen before (n): with n even
      // at the item's start it is the even ones.  The partial statistics below are filed under that parity, not under
      // the group, so that a slot always holds the same tiles (and keys) whatever else the CTA worked on before:
      // results do not depend on how a problem is cut into launches.
      const int par = grp ^ (n & 1);                 // parity, within the item, of the tiles this warp takes
      for (int t = 0; t < ntiles; ++t, ++n) {
        if ((n & 1) != grp) continue;
        const int acc = n & 3;
        const uint32_t accphase = (uint32_t)((n >> 2) & 1);
        ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_TFULL + acc), accphase, s_abort));
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)acc * 128u;
        const int tbase = key0 + t * kTile;
        const bool tail = (tbase + kTile - 1 > N - L);   // some key of the tile is masked for some row
        if (a.pass == 1 && rows == 128) {
          // a TMEM lane is a window row (quad * 32 + lane), the 128 columns are the keys of the tile
          const int pos = N - L + ((quad * 32 + lane) % L);   // last key this window row may see
#pragma unroll
          for (int cg = 0; cg < 2; ++cg) {               // 64 keys per TMEM load
            uint32_t r[64];
            tc_ld64(taddr + (uint32_t)(cg * 64), r);
            tc_wait_ld();
            float x[64];
            if (!tail) {
#pragma unroll
              for (int k = 0; k < 64; ++k) x[k] = __uint_as_float(r[k]);
            } else {
#pragma unroll
              for (int k = 0; k < 64; ++k) {
                const int j = tbase + cg * 64 + k;
                x[k] = (j <= pos && j < N) ? __uint_as_float(r[k]) : -INFINITY;
              }
            }
            float cm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int k = 0; k < 64; ++k) cm4[k & 3] = fmaxf(cm4[k & 3], x[k]);
            const float cm = fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3]));
            if (cm > m_run[0]) {
              z_run[0] *= ex2((m_run[0] - cm) * scale2);
              m_run[0] = cm;
            }
            if (m_run[0] > -INFINITY) {
              const float ms = -m_run[0] * scale2;
              float zs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int k = 0; k < 64; ++k) zs[k & 3] += ex2(fmaf(x[k], scale2, ms));
              z_run[0] += (zs[0] + zs[1]) + (zs[2] + zs[3]);
            }
          }
        } else if (a.pass == 1) {
          const int jw = tbase + quad * 32;              // first key of this warp's 32 lanes
#pragma unroll
          for (int rg = 0; rg < 4; ++rg) {
            if (rg * 32 < rows) {
              uint32_t r[32];
              tc_ld32(taddr + (uint32_t)(rg * 32), r);
              tc_wait_ld();
              // transpose the warp's [32 keys][32 rows] block through shared memory
#pragma unroll
              for (int c = 0; c < 32; ++c) myT[lane * 33 + c] = __uint_as_float(r[c]);
              __syncwarp();
              float x[32];
              if (!tail) {
#pragma unroll
                for (int k = 0; k < 32; ++k) x[k] = myT[k * 33 + lane];
              } else {
                const int pos = N - L + ((rg * 32 + lane) % L);   // last key this window row may see
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                  const int j = jw + k;
                  x[k] = (j <= pos && j < N) ? myT[k * 33 + lane] : -INFINITY;
                }
              }
              __syncwarp();
              // four interleaved chains: a single running max / sum would serialise on the ALU latency
              float cm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
              for (int k = 0; k < 32; ++k) cm4[k & 3] = fmaxf(cm4[k & 3], x[k]);
              const float cm = fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3]));
              if (cm > m_run[rg]) {
                z_run[rg] *= ex2((m_run[rg] - cm) * scale2);
                m_run[rg] = cm;
              }
              if (m_run[rg] > -INFINITY) {
                const float ms = -m_run[rg] * scale2;
                float zs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int k = 0; k < 32; ++k) zs[k & 3] += ex2(fmaf(x[k], scale2, ms));
                z_run[rg] += (zs[0] + zs[1]) + (zs[2] + zs[3]);
              }
            }
          }
        } else {
          const int j = tbase + quad * 32 + lane;   // this thread's key
          float cs[4] = {0.f, 0.f, 0.f, 0.f};   // four interleaved chains (FMA latency)
          if (rows >= 64 && !tail) {
            // 64 columns per TMEM load: half the load / wait round trips of the 32-column walk below
            for (int c0 = 0; c0 < rows; c0 += 64) {
              uint32_t r[64];
              tc_ld64(taddr + (uint32_t)c0, r);
              tc_wait_ld();
              const float4* st4 = reinterpret_cast<const float4*>(myStat + c0);   // four rows per 16-byte load
#pragma unroll
              for (int c = 0; c < 64; c += 4) {
                const float4 off = st4[c >> 2];
                cs[0] += ex2(fmaf(__uint_as_float(r[c]), scale2, -off.x));
                cs[1] += ex2(fmaf(__uint_as_float(r[c + 1]), scale2, -off.y));
                cs[2] += ex2(fmaf(__uint_as_float(r[c + 2]), scale2, -off.z));
                cs[3] += ex2(fmaf(__uint_as_float(r[c + 3]), scale2, -off.w));
              }
            }
          } else
          for (int c0 = 0; c0 < rows; c0 += 32) {
            uint32_t r[32];
            tc_ld32(taddr + (uint32_t)c0, r);
            tc_wait_ld();
            if (!tail) {
              const float4* st4 = reinterpret_cast<const float4*>(myStat + c0);   // four rows per 16-byte load
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                const float4 off = st4[c >> 2];
                cs[0] += ex2(fmaf(__uint_as_float(r[c]), scale2, -off.x));
                cs[1] += ex2(fmaf(__uint_as_float(r[c + 1]), scale2, -off.y));
                cs[2] += ex2(fmaf(__uint_as_float(r[c + 2]), scale2, -off.z));
                cs[3] += ex2(fmaf(__uint_as_float(r[c + 3]), scale2, -off.w));
              }
            } else {
              // window row c0 + c sees keys up to N - L + (c0 + c) % L.  The residue is counted along (one
              // division per 32 rows): a division per element made this tile cost fourteen ordinary ones
              int res = c0 % L;
              const int need = j - (N - L);         // the row's residue must reach this for key j to be visible
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const float off = myStat[c0 + c];
                const bool vis = (j < N) && (need <= res);
                if (vis) cs[c & 3] += ex2(fmaf(__uint_as_float(r[c]), scale2, -off));
                res = (res + 1 == L) ? 0 : res + 1;
              }
            }
          }
          const float csum = (cs[0] + cs[1]) + (cs[2] + cs[3]);
          if (j < N) p.C[p.c_off[u] + j] = csum;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_TEMPTY + acc));
      }
      if (!ok) break;
      if (a.pass == 1) {
        // the warp's partial of this item: slot (chunk, part), part = (tile parity, lane quadrant); with 128 rows a
        // quadrant is a set of rows, so there part = tile parity
        float2* slot = reinterpret_cast<float2*>(p.stat_part) +
                       ((size_t)u * p.chunks_max + (size_t)it.ch * (rows == 128 ? 2 : kTcParts)) * p.rows_pad;
        if (rows == 128) {
          slot[(size_t)par * p.rows_pad + quad * 32 + lane] = make_float2(m_run[0] * scale2, z_run[0]);
        } else {
#pragma unroll
          for (int rg = 0; rg < 4; ++rg)
            if (rg * 32 < rows)
              slot[(size_t)(par * 4 + quad) * p.rows_pad + rg * 32 + lane] = make_float2(m_run[rg] * scale2, z_run[rg]);
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  // after a time-out give copies and MMAs still in flight a bounded time to land before the memory is released
  if (*s_abort)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, kTmemCols);
  }
  if (tid == 0 && *s_abort) set_status(p.status, TASKKV_ETIMEOUT);
}

// Folds the partial statistics of one unit: slots (item, warp) of pass 1 -> one offset per row.
// One block per unit, one thread per row: the thread walks the unit's slots in order (a fixed order whatever the
// launch), its neighbours reading the neighbouring rows of the same slot (coalesced); four slots are loaded ahead of
// the dependent max / sum updates.
__global__ void __launch_bounds__(128) window_tc_reduce_kernel(DeviceProblem p, UnitRange ur, int chunk_keys,
                                                               int parts, int n_real) {
  const int u = ur.unit(blockIdx.x);
  const int slots = (p.unit_N[u] + chunk_keys - 1) / chunk_keys * parts;
  const float2* part = reinterpret_cast<const float2*>(p.stat_part) + (size_t)u * p.chunks_max * p.rows_pad;
  const int row = threadIdx.x;
  if (row >= p.rows) return;
  float M = -INFINITY, z = 0.f;
  auto fold = [&](const float2 o) {
    if (o.x > -INFINITY) {
      const float Mn = fmaxf(M, o.x);
      z = z * exp2f(M - Mn) + o.y * exp2f(o.x - Mn);
      M = Mn;
    }
  };
  int c = 0;
  for (; c + 4 <= slots; c += 4) {
    float2 o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = part[(size_t)(c + i) * p.rows_pad + row];
#pragma unroll
    for (int i = 0; i < 4; ++i) fold(o[i]);
  }
  for (; c < slots; ++c) fold(part[(size_t)c * p.rows_pad + row]);
  // one offset per row: score * scale - (max + log2(sum) + log2(rows)) is log2 of the row's share of C
  // prefix mode (n_real > 0): a query row at or beyond the end of the sequence does not exist; an infinite
  // offset takes it out of every column sum
  const bool absent = n_real > 0 && p.unit_N[u] - p.rows + row >= n_real;
  p.stat[(size_t)u * (2 * p.rows_pad) + row] = (z > 0.f && !absent) ? M + log2f(z) + log2f((float)p.rows) : INFINITY;
}

// Keys per work item.  Every item costs a Q load and, in pass 2, a statistics load, so long items are
// better as long as the CTAs still get a dozen items each; short inputs keep 2048-key items.
inline int pick_chunk(int64_t units_times_keys, int n_sm) {
  const int big = 2 * kTcChunk;
  return units_times_keys / big >= (int64_t)12 * n_sm ? big : kTcChunk;
}

template <int D>
cudaError_t launch_tc_d(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0, int n_layers) {
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  const TcLayout lay = make_layout(D, p.rows);
  if (lay.stages < 2) return cudaErrorInvalidValue;
  const int smem = lay.total;
  cudaError_t e = cudaFuncSetAttribute(window_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  const int per_seq_all = p.R * p.n_kv;
  const int first = layer0 * p.n_kv;               // the launch covers units [first, first + per_seq) of every sequence
  const int per_seq = n_layers * p.n_kv;
  const int skip = (layer0 - h.base_layer) * p.n_kv;   // units between what h.q / h.k point at and the first one
  if (per_seq <= 0) return cudaSuccess;
  const int parts = p.rows == 128 ? 2 : kTcParts;
  // up to kMaxSeq sequences per pair of launches
  for (int b0 = 0; b0 < h.batch; b0 += kMaxSeq) {
    const int nb = h.batch - b0 < kMaxSeq ? h.batch - b0 : kMaxSeq;
    TcMaps maps;
    TcArgs a;
    int64_t keys = 0;
    for (int i = 0; i < nb; ++i) keys += (int64_t)per_seq * h.seq_lens[b0 + i];
    a.n_seq = nb;
    a.n_local = per_seq;
    a.prefix_blocks = 0;
    a.group = 1;
    a.chunk_keys = pick_chunk(keys, n_sm);
    a.item_off[0] = 0;
    for (int i = 0; i < kMaxSeq; ++i) {
      const int b = b0 + (i < nb ? i : 0);                  // unused slots repeat the first sequence
      const int N = h.seq_lens[b];
      if (i >= nb) {
        maps.k[i] = maps.k[0];
        maps.q[i] = maps.q[0];
      } else {
        const char* kb = static_cast<const char*>(h.k[b]) + (size_t)skip * (size_t)N * D * sizeof(__nv_bfloat16);
        const char* qb = static_cast<const char*>(h.q[b]) + (size_t)skip * p.rows * D * sizeof(__nv_bfloat16);
        if (!make_tensor_map_2d(&maps.k[i], kb, D, (uint64_t)per_seq * (uint64_t)N, kTile)) return cudaErrorUnknown;
        if (!make_tensor_map_2d(&maps.q[i], qb, D, (uint64_t)per_seq * (uint64_t)p.rows, p.rows))
          return cudaErrorUnknown;
      }
      a.u0[i] = b * per_seq_all + first;
      a.N[i] = N;
      a.chunks[i] = (N + a.chunk_keys - 1) / a.chunk_keys;
      a.item_off[i + 1] = a.item_off[i] + (i < nb ? per_seq * a.chunks[i] : 0);
    }
    const int n1 = a.item_off[nb];
    const int grid = n1 < n_sm ? n1 : n_sm;
    a.steps = (n1 + grid - 1) / grid;
    if (h.lse) {
      // the caller already has the rows' normalisers: no pass 1
      const size_t lse_skip = (size_t)(layer0 - h.base_layer) * p.n_heads * p.L;
      for (int i = 0; i < nb; ++i) {
        e = launch_lse_to_stat(p, (b0 + i) * per_seq_all + first, per_seq,
                               static_cast<const float*>(h.lse[b0 + i]) + lse_skip, true, s);
        if (e != cudaSuccess) return e;
      }
    } else {
      a.pass = 1;
      {
        LaunchScope ls(K_WINDOW_TC, s);
        window_tc_kernel<D><<<grid, kThreads, smem, s>>>(maps, p, a, lay);
      }
      {
        LaunchScope ls(K_WINDOW_REDUCE, s);
        const UnitRange ur{b0 * per_seq_all + first, per_seq, per_seq_all, nb * per_seq};
        window_tc_reduce_kernel<<<nb * per_seq, 128, 0, s>>>(p, ur, a.chunk_keys, parts, 0);
      }
    }
    a.pass = 2;
    {
      LaunchScope ls(K_WINDOW_TC, s);
      window_tc_kernel<D><<<grid, kThreads, smem, s>>>(maps, p, a, lay);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Prefix mode: p describes heads * blocks virtual units of 128 window rows (rows = L = 128; unit_N, c_off, stat,
// stat_part sized for them); q is [heads][N][d], k is [heads / group][N][d].
template <int D>
cudaError_t launch_prefix_d(const DeviceProblem& p, const void* q, const void* k, int heads, int group, int N,
                            cudaStream_t s) {
  int dev = 0, n_sm = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (n_sm <= 0) n_sm = 148;
  const TcLayout lay = make_layout(D, p.rows);
  if (lay.stages < 2) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(window_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, lay.total);
  if (e != cudaSuccess) return e;
  const int blocks = (N + kTile - 1) / kTile;
  TcMaps maps;
  TcArgs a;
  a.n_seq = 1;
  a.n_local = heads * blocks;
  a.prefix_blocks = blocks;
  a.group = group;
  a.chunk_keys = kTcChunk;
  a.item_off[0] = 0;
  for (int i = 0; i < kMaxSeq; ++i) {
    if (i > 0) {
      maps.k[i] = maps.k[0];
      maps.q[i] = maps.q[0];
    } else {
      if (!make_tensor_map_2d(&maps.k[i], k, D, (uint64_t)(heads / group) * (uint64_t)N, kTile)) return cudaErrorUnknown;
      if (!make_tensor_map_2d(&maps.q[i], q, D, (uint64_t)heads * (uint64_t)N, p.rows)) return cudaErrorUnknown;
    }
    a.u0[i] = 0;
    a.N[i] = N;
    a.chunks[i] = (blocks * kTile + a.chunk_keys - 1) / a.chunk_keys;
    a.item_off[i + 1] = a.item_off[i] + (i == 0 ? a.n_local * a.chunks[i] : 0);
  }
  const int n1 = a.item_off[1];
  const int grid = n1 < n_sm ? n1 : n_sm;
  a.steps = (n1 + grid - 1) / grid;
  a.pass = 1;
  {
    LaunchScope ls(K_WINDOW_TC, s);
    window_tc_kernel<D><<<grid, kThreads, lay.total, s>>>(maps, p, a, lay);
  }
  {
    LaunchScope ls(K_WINDOW_REDUCE, s);
    const UnitRange ur{0, a.n_local, a.n_local, a.n_local};
    window_tc_reduce_kernel<<<a.n_local, 128, 0, s>>>(p, ur, a.chunk_keys, 2, N);
  }
  a.pass = 2;
  {
    LaunchScope ls(K_WINDOW_TC, s);
    window_tc_kernel<D><<<grid, kThreads, lay.total, s>>>(maps, p, a, lay);
  }
  return cudaGetLastError();
}

}  // namespace

bool window_tc_supported(const DeviceProblem& p, int dtype) {
  return dtype == TASKKV_BF16 && (p.rows == 32 || p.rows == 64 || p.rows == 128) && p.L <= p.rows &&
         encode_fn() != nullptr;
}

cudaError_t launch_window_prefix(const DeviceProblem& p, const void* q, const void* k, int heads, int group, int N,
                                 cudaStream_t s) {
  return p.d == 64 ? launch_prefix_d<64>(p, q, k, heads, group, N, s) : launch_prefix_d<128>(p, q, k, heads, group, N, s);
}

cudaError_t launch_window_scores_tc(const DeviceProblem& p, const WindowHostInfo& h, cudaStream_t s, int layer0,
                                    int n_layers) {
  if (n_layers < 0) { layer0 = 0; n_layers = p.R; }
  // 32 window rows and sequences short enough for a unit's scores to stay in tensor memory: K is read once
  if (window_res_supported(p, h)) return launch_window_scores_res(p, h, s, layer0, n_layers);
  return p.d == 64 ? launch_tc_d<64>(p, h, s, layer0, n_layers) : launch_tc_d<128>(p, h, s, layer0, n_layers);
}

}  // namespace taskkv
