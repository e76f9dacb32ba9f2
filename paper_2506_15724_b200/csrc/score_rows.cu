// Stage 1, tensor-core path for wide windows (Eq. 7 with the softmax of Eq. 5): bf16 inputs with 64 < g * w <= 256
// window rows per KV head (grouped-query attention with many query heads per KV head), and the single-pass form of
// stage 1 (log-sum-exps supplied by the caller) for every bf16 shape with g * w <= 256.
//
// With that many rows the work per key byte is dominated by the exponentials (g * w of them per key and pass), not
// by HBM: the special-function unit delivers 16 exp2 per clock and SM, which for 256 rows is 2048 clocks per 128-key
// tile against ~1400 clocks for reading the tile from HBM. The kernels are therefore built around keeping that unit
// busy.
//   pass 1  window rows on M (one or two blocks of 128 rows), the 128 keys of a tile on N: an epilogue thread owns
//           ONE window row (a TMEM lane) and a share of the tile's columns and keeps a running (max, sum of exp2) of
//           its row in registers, carried from tile to tile for as long as the CTA stays with the unit; one (max,
//           sum) pair per row, column share and run goes to the workspace
//   merge   per (unit, row): all pairs -> the row's log-sum-exp (a separate small kernel)
//   pass 2  the tile turned back (128 keys on M, the window rows on N): a thread owns one key and a quarter of the
//           window rows, and psi(i) = sum over rows of exp2(s - lse) is an in-thread sum over columns of its TMEM lane.
//           The shift by the row's log-sum-exp is part of the contraction: one more 16-deep step multiplies a
//           constant column of ones on the key side with -lse / scale (as three bf16 terms) on the row side, so the
//           accumulator arrives shifted and the epilogue reads no per-row operand (with the log-sum-exps as
//           shared-memory broadcasts the loads competed with the tensor core's operand reads and cost a fifth of
//           the pass). The four warps that share a key add their partial sums up through shared memory in a
//           fixed order.
// In both passes all 16 epilogue warps work on the same tile while the MMAs of the next tile fill the other half of
// the TMEM; the TMEM load of a warp's next 16 columns is in flight while it works on the present ones.
// K is streamed twice. The passes are separate launches and no CTA ever waits for another CTA. The work is the list
// of all 128-key tiles in (sequence, layer, KV head, tile) order; a CTA takes a contiguous range of it, the same
// number of tiles to within one for every CTA whatever the lengths in the batch. The part of a unit inside a CTA's
// range is a run: queries and log-sum-exps are loaded once per run, and pass 1 leaves one pair per run, so a unit's
// statistics come in as many pieces as CTAs share it (two or three for long sequences). Warp roles: warp 0 TMA
// producer, warp 1 MMA issuer and TMEM owner, warps 2-17 epilogue; TMEM lane quarter = warp % 4 throughout. Every wait is bounded: on expiry the kernel records MADAKV_ETIMEOUT, drains and returns.
#include "tc_common.cuh"

namespace madakv {
namespace {

constexpr int kRowThreads = 576;  // 2 + 16 warps
constexpr int kMaxSeqScan = 1024; // batches up to this size get the exact (ragged-aware) tile partition
constexpr int kFoldTiles = 16;    // pass 1 moves a row's sum to its second level every this many tiles

struct RowParams {
  const int32_t* seq_len;
  float* psi;        // [units, n_max]
  float2* part;      // ws: [units, smax, cparts, rs] (max, sum) of every row over a column share of one CTA's run
  const float* lse2; // ws: [units, rs] NEGATED log2-domain log-sum-exp, padding rows hold kEmptyMax (pass 2)
  int32_t* status;   // ws header
  int B, units, L, Hq, Hkv, g, w, R, n_max, causal, rs, mblocks, cparts, n16;  // n16: R rounded up to 16
  int smax;          // runs (CTAs) a unit's tiles can be spread over at most: wide_max_runs()
  int grid;          // CTAs of the two passes (the merge kernel needs the partition)
  float scale2;
};

template <int D, int PASS>
struct RowSmem {
  // pass 2 gives up one K stage for the operands of its extra contraction step (see the MMA issuer)
  static constexpr int kStages = (D == 128 ? 4 : 8) - (PASS == 2 ? (D == 128 ? 1 : 2) : 0);
  static constexpr int kKBlocks = D / 64;
  static constexpr int kStageBytes = kTileKeys * D * 2;
  static constexpr int kQBytes = 256 * D * 2;  // up to two blocks of 128 rows
  static constexpr int kKOff = 0;
  static constexpr int kQOff = kStages * kStageBytes;
  static constexpr int kOnesOff = kQOff + kQBytes;                          // pass 2: [128 keys][64] bf16, 1 in columns 0-2
  static constexpr int kShiftOff = kOnesOff + (PASS == 2 ? 128 * 128 : 0);  // pass 2: [256 rows][64] bf16, columns 0-2
  static constexpr int kBarOff = kShiftOff + (PASS == 2 ? 256 * 128 : 0);
  // full[kStages], empty[kStages], qfull, qempty, tfull[2], tempty[2], drain, xfull[8], xempty[8]
  static constexpr int kNumBars = 2 * kStages + 2 + 4 + 1 + 16;
  static constexpr int kMiscOff = (kBarOff + kNumBars * 8 + 15) / 16 * 16;
  static constexpr int kColOff = kMiscOff + 48;            // window position (row % w) of every row [256]
  static constexpr int kXchOff = kColOff + 256 * 4;        // pass 2: partial psi of column shares 1-3 [2][3][128]
  static constexpr int kTotal = kXchOff + 6 * 128 * 4;
  static constexpr int kAlloc = kTotal + 1024;
  static_assert(kQOff % 1024 == 0 && kOnesOff % 1024 == 0 && kShiftOff % 1024 == 0 && kBarOff % 8 == 0, "alignment");
  static_assert(kAlloc <= 227 * 1024, "shared memory");
};

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kIdescRows = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

// exp2 of 8 packed pairs, summed
__device__ __forceinline__ uint64_t exp2_sum16(const uint64_t (&x)[8]) {
  uint64_t e[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float lo, hi;
    unpack2(x[i], lo, hi);
    e[i] = pack2(ex2(lo), ex2(hi));
  }
  return add2(add2(add2(e[0], e[1]), add2(e[2], e[3])), add2(add2(e[4], e[5]), add2(e[6], e[7])));
}

__device__ __forceinline__ float sum4(const uint64_t (&a)[4]) {
  float lo, hi;
  unpack2(add2(add2(a[0], a[1]), add2(a[2], a[3])), lo, hi);
  return lo + hi;
}
__device__ __forceinline__ float block_max16(const uint32_t (&r)[16]) {
  const float a0 = max3f(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
  const float a1 = max3f(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
  const float a2 = max3f(__uint_as_float(r[6]), __uint_as_float(r[7]), __uint_as_float(r[8]));
  const float a3 = max3f(__uint_as_float(r[9]), __uint_as_float(r[10]), __uint_as_float(r[11]));
  const float a4 = max3f(__uint_as_float(r[12]), __uint_as_float(r[13]), __uint_as_float(r[14]));
  return max3f(max3f(a0, a1, a2), a3, fmaxf(a4, __uint_as_float(r[15])));
}

// A tile's NB blocks of 16 accumulator columns of this thread's TMEM lane, none of them masked, as a software
// pipeline over steps of 8 columns: the exponentials of step s are queued on the special-function unit, then the
// results of step s - 1 are added up and the inputs of step s + 1 prepared, so that a warp on its own keeps the unit
// supplied (with the steps one after the other a lone warp kept it half busy, and at the end of every tile the
// last warps of a scheduler are on their own). The TMEM load of block j + 1 is in flight during block j.
//
// Pass 2: acc += exp2(scale2 * column); the accumulator already holds q.k - lse / scale.
template <int NB>
__device__ __forceinline__ void psi_tile(uint32_t taddr, uint64_t sc2, uint64_t (&acc)[4]) {
  uint32_t r[2][16];
  uint64_t x[2][4], e[2][4];
  tmem_ld16_issue(taddr, r[0]);
  tmem_ld_wait16(r[0]);
  if (NB > 1) tmem_ld16_issue(taddr + 16, r[1]);
#pragma unroll
  for (int i = 0; i < 4; ++i) x[0][i] = mul2(pack2u(r[0][2 * i], r[0][2 * i + 1]), sc2);
#pragma unroll
  for (int s = 0; s < 2 * NB; ++s) {
    const int cur = s & 1, nxt = cur ^ 1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float lo, hi;
      unpack2(x[cur][i], lo, hi);
      e[cur][i] = pack2(ex2(lo), ex2(hi));
    }
    if (s > 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] = add2(acc[i], e[nxt][i]);
    }
    if (s + 1 < 2 * NB) {
      const int blk = (s + 1) >> 1, half = (s + 1) & 1, b = blk & 1;
      if (half == 0) {
        tmem_ld_wait16(r[b]);
        if (blk + 1 < NB) tmem_ld16_issue(taddr + (blk + 1) * 16, r[b ^ 1]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) x[nxt][i] = mul2(pack2u(r[b][8 * half + 2 * i], r[b][8 * half + 2 * i + 1]), sc2);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) acc[i] = add2(acc[i], e[(2 * NB - 1) & 1][i]);
}

// Pass 1: the row's running maximum m (log2 domain) is checked once per block; it rarely grows once a few hundred
// keys have been seen, so the rescaling sits behind a warp-uniform branch. acc holds the sum of exp2(scale2 * s - m)
// of the item at hand, z_run that of the run's earlier items.
template <int NB>
__device__ __forceinline__ void stat_tile(uint32_t taddr, float scale2, uint64_t sc2, float& m, uint64_t (&acc)[4],
                                          float& z_run) {
  uint32_t r[2][16];
  uint64_t x[2][4], e[2][4];
  auto grow = [&](float bm) {
    const float mn = fmaxf(m, bm);
    const float f = ex2(m - mn);
    const uint64_t f2 = pack2(f, f);
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = mul2(acc[i], f2);
    z_run *= f;
    m = mn;
  };
  tmem_ld16_issue(taddr, r[0]);
  tmem_ld_wait16(r[0]);
  if (NB > 1) tmem_ld16_issue(taddr + 16, r[1]);
  {
    const float bm = block_max16(r[0]) * scale2;
    if (__any_sync(0xffffffffu, bm > m)) grow(bm);
  }
  uint64_t nm2 = pack2(-m, -m);
#pragma unroll
  for (int i = 0; i < 4; ++i) x[0][i] = fma2(pack2u(r[0][2 * i], r[0][2 * i + 1]), sc2, nm2);
#pragma unroll
  for (int s = 0; s < 2 * NB; ++s) {
    const int cur = s & 1, nxt = cur ^ 1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float lo, hi;
      unpack2(x[cur][i], lo, hi);
      e[cur][i] = pack2(ex2(lo), ex2(hi));
    }
    if (s > 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] = add2(acc[i], e[nxt][i]);
    }
    if (s + 1 < 2 * NB) {
      const int blk = (s + 1) >> 1, half = (s + 1) & 1, b = blk & 1;
      if (half == 0) {
        tmem_ld_wait16(r[b]);
        if (blk + 1 < NB) tmem_ld16_issue(taddr + (blk + 1) * 16, r[b ^ 1]);
        const float bm = block_max16(r[b]) * scale2;
        if (__any_sync(0xffffffffu, bm > m)) {
          // the exponentials just queued were taken against the old maximum: they go in before the rescaling
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            acc[i] = add2(acc[i], e[cur][i]);
            e[cur][i] = 0ull;
          }
          grow(bm);
          nm2 = pack2(-m, -m);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) x[nxt][i] = fma2(pack2u(r[b][8 * half + 2 * i], r[b][8 * half + 2 * i + 1]), sc2, nm2);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) acc[i] = add2(acc[i], e[(2 * NB - 1) & 1][i]);
}

// The CTA's share of the work: a contiguous range of the 128-key tiles of all units, in (sequence, layer, KV head,
// tile) order, cut at tile granularity (every CTA gets the same number of tiles to within one, whatever the batch's
// length mix). The part of one unit inside a CTA's range is a run: the queries are loaded once per run, and pass 1
// leaves one (max, sum) pair per run, row and column share. Sequence b has L * Hkv * tiles_of(b) tiles.
struct TileCursor {
  int b;        // sequence
  int r;        // index among the tiles of sequence b
  int tb;       // tiles per unit of sequence b
  int per_b;    // tiles of sequence b
  int left;     // tiles of the range still to do
  int done;     // tiles of the range already done
};
struct Run {
  int u, b, n;  // unit, its sequence and that sequence's length
  int t0, cnt;  // first tile of the run within the unit, tiles in the run (what the partition counts)
  int tiles;    // tiles of the run that hold keys (fewer than cnt only in the uniform partition of very large batches)
};

__device__ __forceinline__ int tiles_of(const RowParams& p, int b, bool exact) {
  return ((exact ? clamped_len(p.seq_len, b, p.n_max) : p.n_max) + kTileKeys - 1) / kTileKeys;
}
__device__ __forceinline__ void cursor_settle(const RowParams& p, TileCursor& c, bool exact) {
  // move on to the next sequence that has tiles
  while (c.left > 0 && c.r >= c.per_b) {
    c.r -= c.per_b;
    ++c.b;
    if (c.b >= p.B) {
      c.left = 0;
      break;
    }
    c.tb = tiles_of(p, c.b, exact);
    c.per_b = p.L * p.Hkv * c.tb;
  }
}
__device__ __forceinline__ Run cursor_run(const RowParams& p, const TileCursor& c) {
  Run r;
  const int ub = c.r / c.tb;
  r.t0 = c.r - ub * c.tb;
  r.cnt = min(c.tb - r.t0, c.left);
  r.b = c.b;
  r.u = c.b * p.L * p.Hkv + ub;
  r.n = clamped_len(p.seq_len, c.b, p.n_max);
  const int real = (r.n + kTileKeys - 1) / kTileKeys;  // tiles of the unit that hold keys
  r.tiles = max(0, min(r.t0 + r.cnt, real) - r.t0);
  return r;
}
__device__ __forceinline__ void cursor_advance(const RowParams& p, TileCursor& c, const Run& r, bool exact) {
  c.r += r.cnt;
  c.left -= r.cnt;
  c.done += r.cnt;
  cursor_settle(p, c, exact);
}
// The CTA whose range [total * c / grid, total * (c + 1) / grid) holds tile x of the global order.
__device__ __forceinline__ int cta_of(long long total, int grid, long long x) {
  int c = (int)(x * grid / total);
  while (c + 1 < grid && total * (c + 1) / grid <= x) ++c;
  while (c > 0 && total * c / grid > x) --c;
  return c;
}

template <int D, int PASS>
__global__ void __launch_bounds__(kRowThreads, 1)  // 96 registers: warps are allocated four at a time (18 -> 20)
score_rows_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q, RowParams p) {
  using SL = RowSmem<D, PASS>;
  constexpr int kStages = SL::kStages;
  constexpr int kKBlocks = SL::kKBlocks;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* k_s = smem + SL::kKOff;
  uint8_t* q_s = smem + SL::kQOff;
  uint8_t* ones_s = smem + SL::kOnesOff;
  uint8_t* shift_s = smem + SL::kShiftOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBarOff);
  uint64_t* full = bars;               // [kStages] TMA -> MMA
  uint64_t* empty = bars + kStages;    // [kStages] MMA -> TMA
  uint64_t* qfull = empty + kStages;   // [1]       TMA -> MMA (queries of the unit; in pass 2 also its shift rows)
  uint64_t* qempty = qfull + 1;        // [1]       MMA -> TMA
  uint64_t* tfull = qempty + 1;        // [2]       MMA -> epilogue
  uint64_t* tempty = tfull + 2;        // [2]       epilogue -> MMA
  uint64_t* drain = tempty + 2;        // [1]
  uint64_t* xfull = drain + 1;         // [2][4]    pass 2: column shares 1-3 -> share 0, per buffer and lane quarter
  uint64_t* xempty = xfull + 8;        // [2][4]    pass 2: share 0 -> shares 1-3
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(smem + SL::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kMiscOff + 4);
  int* range_s = reinterpret_cast<int*>(smem + SL::kMiscOff + 8);  // first sequence, tile in it, tiles, exact, lo, total, CTAs in use
  int* rowpos = reinterpret_cast<int*>(smem + SL::kColOff);
  float* xch = reinterpret_cast<float*>(smem + SL::kXchOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(qfull, 1);
    mbar_init(qempty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], 512);  // every epilogue thread
    }
    mbar_init(drain, 1);
    for (int i = 0; i < 8; ++i) {
      mbar_init(&xfull[i], 96);
      mbar_init(&xempty[i], 32);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // this CTA's range of tiles
    const bool exact = p.B <= kMaxSeqScan;
    long long total = 0;
    if (exact) {
      for (int b = 0; b < p.B; ++b) total += (long long)p.L * p.Hkv * tiles_of(p, b, true);
    } else {
      total = (long long)p.units * tiles_of(p, 0, false);
    }
    // (a batch with fewer tiles than CTAs is spread over as many CTAs as it has tiles: no empty range lies between
    // two CTAs that share a unit)
    const long long ctas = total < (long long)gridDim.x ? total : (long long)gridDim.x;
    const bool idle = (long long)blockIdx.x >= ctas;
    const long long lo = idle ? total : total * blockIdx.x / ctas, hi = idle ? total : total * (blockIdx.x + 1) / ctas;
    int b0 = 0;
    long long r0 = lo;
    if (exact) {
      while (b0 < p.B) {
        const long long per = (long long)p.L * p.Hkv * tiles_of(p, b0, true);
        if (r0 < per) break;
        r0 -= per;
        ++b0;
      }
    } else {
      const long long per = (long long)p.L * p.Hkv * tiles_of(p, 0, false);
      b0 = (int)(lo / per);
      r0 = lo - (long long)b0 * per;
    }
    range_s[0] = b0;
    range_s[1] = (int)r0;
    range_s[2] = (int)(hi - lo);
    range_s[3] = exact ? 1 : 0;
    range_s[4] = (int)lo;     // (the host refuses shapes with 2^31 tiles or more)
    range_s[5] = (int)total;
    range_s[6] = (int)ctas;
  }
  // rows R..255 of the Q buffer are never written by TMA: keep them zero so their logits are 0. Pass 2: the operands
  // of the extra contraction step start out as zeros, the key side gets its three ones per row (128-byte rows with
  // the 128-byte swizzle: the 16-byte piece that holds columns 0-7 of row r sits at position r % 8).
  for (int x = threadIdx.x; x < (SL::kBarOff - SL::kQOff) / 16; x += kRowThreads)
    reinterpret_cast<uint4*>(q_s)[x] = make_uint4(0, 0, 0, 0);
  for (int x = threadIdx.x; x < 256; x += kRowThreads) rowpos[x] = x % p.w;
  __syncthreads();
  if (PASS == 2 && threadIdx.x < kTileKeys) {
    const int r = threadIdx.x;
    *reinterpret_cast<uint4*>(ones_s + r * 128 + (r & 7) * 16) = make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_s;
  const bool exact = range_s[3] != 0;

  auto cursor_begin = [&]() {
    TileCursor c;
    c.b = range_s[0];
    c.r = range_s[1];
    c.left = c.b < p.B ? range_s[2] : 0;
    c.done = 0;
    c.tb = c.left > 0 ? tiles_of(p, c.b, exact) : 1;
    c.per_b = p.L * p.Hkv * c.tb;
    cursor_settle(p, c, exact);
    return c;
  };

  if (warp == 0) {
    // ================================================================ TMA producer: lane 0 waits and issues the
    // copies; the whole warp walks the items with it, because in pass 2 all 32 lanes write the unit's shift rows
    const uint64_t pol_k = l2_policy_evict_first();
    const uint64_t pol_q = l2_policy_evict_last();
    int stage = 0, cur_u = -1;
    uint32_t stage_par = 0, q_par = 0;
    bool ok = true;
    for (TileCursor c = cursor_begin(); ok && c.left > 0;) {
      const Run run = cursor_run(p, c);
      cursor_advance(p, c, run, exact);
      const int u = run.u, tiles = run.tiles, key_begin = run.t0 * kTileKeys;
      if (tiles == 0) continue;
      const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
      if (u != cur_u) {  // a new run: the unit's queries (and, in pass 2, its shift rows)
        cur_u = u;
        if (lane == 0) ok = mbar_wait(qempty, q_par ^ 1, abort_flag, p.status, kSiteQEmpty);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        q_par ^= 1;
        if (PASS == 2) {
          // Row r of the shift operand: -lse_r / scale as the sum of three bf16 numbers (24 bits) in columns 0-2.
          // Multiplied by the key side's ones in the extra contraction step, the accumulator holds q.k - lse / scale
          // and the epilogue needs no per-row operand at all.
          const float inv = 1.0f / p.scale2;
          const float* src = p.lse2 + (int64_t)u * p.rs;
          for (int r = lane; r < p.n16; r += 32) {
            const float v = src[r] * inv;
            const float hi = __bfloat162float(__float2bfloat16_rn(v));
            const float mid = __bfloat162float(__float2bfloat16_rn(v - hi));
            const float low = __bfloat162float(__float2bfloat16_rn((v - hi) - mid));
            const uint32_t w0 = (__float_as_uint(hi) >> 16) | (__float_as_uint(mid) & 0xffff0000u);
            *reinterpret_cast<uint4*>(shift_s + r * 128 + (r & 7) * 16) = make_uint4(w0, __float_as_uint(low) >> 16, 0u, 0u);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();  // every lane's rows are written (and fenced) before lane 0 signals the unit ready
        }
        if (lane == 0) {
          mbar_expect_tx(qfull, (uint32_t)(p.R * 128 * kKBlocks));
          for (int kb = 0; kb < kKBlocks; ++kb)
            tma_load_5d(q_s + kb * 256 * 128, &tmap_q, qfull, kb * 64, 0, h * p.g, l, b, pol_q);
        }
      }
      if (lane == 0) {
        for (int t = 0; t < tiles; ++t) {
          ok = mbar_wait(&empty[stage], stage_par ^ 1, abort_flag, p.status, kSiteStage);
          if (!ok) break;
          mbar_expect_tx(&full[stage], (uint32_t)SL::kStageBytes);
          for (int kb = 0; kb < kKBlocks; ++kb)
            tma_load_5d(k_s + stage * SL::kStageBytes + kb * kTileKeys * 128, &tmap_k, &full[stage], kb * 64,
                        key_begin + t * kTileKeys, h, l, b, pol_k);
          if (++stage == kStages) {
            stage = 0;
            stage_par ^= 1;
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
    }
    if (!ok && lane == 0) {  // abandoned: give copies in flight time to land before the CTA's shared memory goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000ll) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      const uint32_t k_lo0 = smem_desc_lo(smem_u32(k_s)), q_lo0 = smem_desc_lo(smem_u32(q_s));
      const uint32_t ones_lo = smem_desc_lo(smem_u32(ones_s)), shift_lo = smem_desc_lo(smem_u32(shift_s));
      const uint32_t idesc2 = instr_desc_bf16(p.n16);
      int stage = 0, n_tile = 0, cur_u = -1;
      uint32_t stage_par = 0, q_par = 0;
      bool ok = true;
      for (TileCursor c = cursor_begin(); ok && c.left > 0;) {
        const Run run = cursor_run(p, c);
        cursor_advance(p, c, run, exact);
        const int u = run.u, tiles = run.tiles;
        if (tiles == 0) continue;
        if (u != cur_u) {
          if (cur_u >= 0) umma_commit(qempty);  // the queries may be replaced once the MMAs issued so far are done
          cur_u = u;
          ok = mbar_wait(qfull, q_par, abort_flag, p.status, kSiteQFull);
          if (!ok) break;
          q_par ^= 1;
        }
        for (int t = 0; t < tiles; ++t, ++n_tile) {
          const int buf = n_tile & 1;
          const uint32_t use_par = (uint32_t)(n_tile >> 1) & 1u;
          const uint32_t k_lo = k_lo0 + (uint32_t)stage * (SL::kStageBytes >> 4);
          ok = mbar_wait(&tempty[buf], use_par ^ 1, abort_flag, p.status, kSiteTEmpty) &&
               mbar_wait(&full[stage], stage_par, abort_flag, p.status, kSiteFull);
          if (!ok) break;
          tc_fence_after();
          if (PASS == 1) {  // D[row, key]: a row block of the queries is operand A, the K tile operand B
            for (int mb = 0; mb < p.mblocks; ++mb) {
              const uint32_t d_tmem = tmem_base + buf * 256 + mb * 128;
#pragma unroll
              for (int ks = 0; ks < D / 16; ++ks) {
                const int kb = ks >> 2, kk = ks & 3;
                umma_bf16(d_tmem, q_lo0 + ((kb * 256 * 128 + mb * 128 * 128 + kk * 32) >> 4),
                          k_lo + ((kb * kTileKeys * 128 + kk * 32) >> 4), kIdescRows, ks > 0 ? 1u : 0u);
              }
            }
          } else {  // D[key, row]: the K tile is operand A, all n16 query rows operand B; then the shift step
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const int kb = ks >> 2, kk = ks & 3;
              umma_bf16(tmem_base + buf * 256, k_lo + ((kb * kTileKeys * 128 + kk * 32) >> 4),
                        q_lo0 + ((kb * 256 * 128 + kk * 32) >> 4), idesc2, ks > 0 ? 1u : 0u);
            }
            umma_bf16(tmem_base + buf * 256, ones_lo, shift_lo, idesc2, 1u);
          }
          umma_commit(&empty[stage]);  // the K stage may be refilled
          umma_commit(&tfull[buf]);    // the accumulators are ready
          if (++stage == kStages) {
            stage = 0;
            stage_par ^= 1;
          }
        }
      }
      if (!ok) {  // abandoned: TMEM may only be freed once this thread's MMAs have completed
        umma_commit(drain);
        const long long t0 = clock64();
        while (!mbar_try(drain, 0) && clock64() - t0 < 20000000ll) __nanosleep(200);
      }
    }
  } else {
    // ================================================================ epilogue (warps 2-17)
    // All 16 warps work on the same tile while the MMAs of the next tile fill the other accumulator buffer;
    // warp = (TMEM lane quarter, column share); the TMEM load of a warp's next 16 columns is in flight while it works.
    const int ew = warp - 2;
    const int quarter = warp & 3;  // TMEM lanes [32 * quarter, 32 * quarter + 32)
    // pass 1: (row block mb, column share): two row blocks x 2 shares of 64 keys, or one row block x 4 shares of 32
    // pass 2: column share = a quarter of the n16 / 16 blocks of window rows (as even as possible)
    const int mb = PASS == 1 && p.mblocks == 2 ? (ew >> 2) & 1 : 0;
    const int share = PASS == 1 ? (p.mblocks == 2 ? ew >> 3 : ew >> 2) : ew >> 2;
    int blk0, nblk;  // this warp's 16-column blocks of a tile's accumulator: blk0 .. blk0 + nblk - 1
    if (PASS == 1) {
      nblk = 8 / p.cparts;
      blk0 = nblk * share;
    } else {
      const int total = p.n16 >> 4, base = total >> 2, rem = total & 3;
      nblk = base + (share < rem ? 1 : 0);
      blk0 = share * base + min(share, rem);
    }
    const uint32_t tlane = tmem_base + ((uint32_t)(quarter * 32) << 16) + (PASS == 1 ? mb * 128 : 0) + blk0 * 16;
    const uint64_t sc2 = pack2(p.scale2, p.scale2);
    int n_tile = 0;
    bool ok = true;
    // pass 1 state: running maximum and sums of the thread's window row, log2 domain; m starts below any masked
    // logit. The sum is kept on two levels (the item at hand, the run's earlier items): one accumulator over a whole
    // long sequence would lose the small terms to rounding.
    const int row = mb * 128 + quarter * 32 + lane;
    float m = 4.f * kEmptyMax, z_run = 0.f;
    uint64_t zacc[4] = {0ull, 0ull, 0ull, 0ull};  // pass 1: the item's sum, as four packed partial sums
    float* xslot = xch + quarter * 32 + lane;  // pass 2: [buffer][share - 1][128 keys]

    for (TileCursor c = cursor_begin(); ok && c.left > 0;) {
      const Run run = cursor_run(p, c);
      const int run_first = range_s[4] + c.done;  // the run's first tile in the global order
      cursor_advance(p, c, run, exact);
      const int u = run.u, tiles = run.tiles, key_begin = run.t0 * kTileKeys, n = run.n;
      float* psi = p.psi + (int64_t)u * p.n_max;
      m = 4.f * kEmptyMax;  // pass 1: every run starts its own statistics
      z_run = 0.f;
      zacc[0] = zacc[1] = zacc[2] = zacc[3] = 0ull;
      int vis = 0;  // pass 1: keys the row may see: [0, vis)
      if (PASS == 1 && row < p.R) {
        const int pos = n - p.w + row % p.w;
        if (pos >= 0) vis = p.causal ? pos + 1 : n;
      }
      for (int t = 0; t < tiles; ++t, ++n_tile) {
        const int buf = n_tile & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(&tfull[buf], (uint32_t)(n_tile >> 1) & 1u, abort_flag, p.status, kSiteTile));
        if (!ok) break;
        tc_fence_after();
        const int key0 = key_begin + t * kTileKeys;
        const uint32_t taddr = tlane + buf * 256;
        uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};  // pass 2: the key's sum over this warp's window rows
        const int key = key0 + quarter * 32 + lane;  // pass 2: the thread's key
        const bool plain = key0 + kTileKeys <= n - p.w;  // every row sees the whole tile: nothing to mask
        uint32_t ra[16], rb[16];
        auto block = [&](uint32_t (&r)[16], int j) {  // block blk0 + j of the accumulator
          if (PASS == 1) {
            const int col0 = key0 + 16 * (blk0 + j);  // first key of the block
            if (col0 + 16 > vis) {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (col0 + i >= vis) r[i] = __float_as_uint(kEmptyMax);
            }
            const float bm = block_max16(r) * p.scale2;
            if (__any_sync(0xffffffffu, bm > m)) {
              const float mn = fmaxf(m, bm);
              const float f = ex2(m - mn);
              const uint64_t f2 = pack2(f, f);
#pragma unroll
              for (int i = 0; i < 4; ++i) zacc[i] = mul2(zacc[i], f2);
              z_run *= f;
              m = mn;
            }
            const uint64_t nm2 = pack2(-m, -m);
            uint64_t x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = fma2(pack2u(r[2 * i], r[2 * i + 1]), sc2, nm2);
            zacc[0] = add2(zacc[0], exp2_sum16(x));
          } else {
            if (!plain) {  // the tiles at the window: every logit is checked against what its row may see
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const int pos = n - p.w + rowpos[16 * (blk0 + j) + i];
                const int v = pos < 0 ? 0 : (p.causal ? pos + 1 : n);
                if (key >= v) r[i] = __float_as_uint(kEmptyMax);
              }
            }
            uint64_t x[8];  // the accumulator already holds q.k - lse / scale
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = mul2(pack2u(r[2 * i], r[2 * i + 1]), sc2);
            acc[0] = add2(acc[0], exp2_sum16(x));
          }
        };
        if (plain) {  // all but the tiles at the window
          if (PASS == 1) {
            if (nblk == 4) stat_tile<4>(taddr, p.scale2, sc2, m, zacc, z_run);
            else stat_tile<2>(taddr, p.scale2, sc2, m, zacc, z_run);
          } else {
            switch (nblk) {
              case 4: psi_tile<4>(taddr, sc2, acc); break;
              case 3: psi_tile<3>(taddr, sc2, acc); break;
              case 2: psi_tile<2>(taddr, sc2, acc); break;
              case 1: psi_tile<1>(taddr, sc2, acc); break;
              default: break;
            }
          }
        } else if (nblk > 0) {
          tmem_ld16_issue(taddr, ra);
#pragma unroll 1
          for (int j = 0; j < nblk; j += 2) {
            tmem_ld_wait16(ra);
            if (j + 1 < nblk) tmem_ld16_issue(taddr + (j + 1) * 16, rb);
            block(ra, j);
            if (j + 1 < nblk) {
              tmem_ld_wait16(rb);
              if (j + 2 < nblk) tmem_ld16_issue(taddr + (j + 2) * 16, ra);
              block(rb, j + 1);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(&tempty[buf]);
        if (PASS == 1 && (t % kFoldTiles) == kFoldTiles - 1) {  // second level of the row's sum
          z_run += sum4(zacc);
          zacc[0] = zacc[1] = zacc[2] = zacc[3] = 0ull;
        }
        if (PASS == 2) {
          // the four warps that share the key add up in a fixed order: shares 1-3 hand their sums to share 0 (a
          // slot is free once share 0 has taken the tile before last)
          float total = sum4(acc);
          const uint32_t xp = (uint32_t)(n_tile >> 1) & 1u;
          if (share) {
            ok = __all_sync(0xffffffffu, mbar_wait(&xempty[buf * 4 + quarter], xp ^ 1, abort_flag, p.status, kSiteFlag));
            if (!ok) break;
            xslot[(buf * 3 + share - 1) * 128] = total;
            mbar_arrive(&xfull[buf * 4 + quarter]);
          } else {
            ok = __all_sync(0xffffffffu, mbar_wait(&xfull[buf * 4 + quarter], xp, abort_flag, p.status, kSiteFlag));
            if (!ok) break;
            total = ((total + xslot[(buf * 3 + 0) * 128]) + xslot[(buf * 3 + 1) * 128]) + xslot[(buf * 3 + 2) * 128];
            mbar_arrive(&xempty[buf * 4 + quarter]);
            if (key < p.n_max) psi[key] = key < n ? total : 0.f;
          }
        }
      }
      if (!ok) break;
      if (PASS == 1) {
        z_run += sum4(zacc);
        if (row < p.R) {
          // one pair per run: slot = this CTA's place among the CTAs that the unit's tiles are spread over (the merge
          // kernel walks the same partition). A row that saw no visible key only summed masked entries: it is
          // recorded as empty, and so is a run without keys (the uniform partition of very large batches has those).
          const long long total = range_s[5];
          const int k = (int)blockIdx.x - cta_of(total, range_s[6], (long long)run_first - run.t0);
          const bool none = tiles == 0 || m < 0.5f * kEmptyMax * p.scale2;
          if (k >= 0 && k < p.smax)
            p.part[(((int64_t)u * p.smax + k) * p.cparts + share) * p.rs + row] =
                none ? make_float2(kEmptyMax, 0.f) : make_float2(m, z_run);
          else
            set_status(p.status, MADAKV_ESHAPE);  // cannot happen: smax bounds the runs of a unit
        }
      }
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// psi of the keys no tile covers: everything from the end of the sequence's last tile
__device__ __forceinline__ void clear_tail(const RowParams& p, int u, int row) {
  const int b = u / (p.Hkv * p.L);
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const int from = (n + kTileKeys - 1) / kTileKeys * kTileKeys;
  float* psi = p.psi + (int64_t)u * p.n_max;
  for (int key = from + row; key < p.n_max; key += p.rs) psi[key] = 0.f;
}

// merge: per (unit, row) the (max, sum) pairs of all runs and column shares, in a fixed order -> log2-domain
// log-sum-exp, stored negated (pass 2 adds it inside a fused multiply-add); padding rows get a shift that turns
// every weight into 0
__global__ void score_rows_merge_kernel(RowParams p, float* nlse2, float* lse_out, int total) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= total) return;
  const int u = x / p.rs, row = x % p.rs;
  clear_tail(p, u, row);
  if (row >= p.R) {
    nlse2[x] = kEmptyMax;
    return;
  }
  const int b = u / (p.Hkv * p.L);
  // the CTAs of pass 1 that the unit's tiles were spread over: the same partition as in the kernel
  const bool exact = p.B <= kMaxSeqScan;
  long long all_tiles = 0, first = 0;  // tiles of the batch; the unit's first tile in the global order
  const int tb = tiles_of(p, b, exact);
  if (exact) {
    for (int b2 = 0; b2 < p.B; ++b2) {
      const long long per = (long long)p.L * p.Hkv * tiles_of(p, b2, true);
      if (b2 < b) first += per;
      all_tiles += per;
    }
  } else {
    all_tiles = (long long)p.units * tb;
    first = (long long)b * p.L * p.Hkv * tb;
  }
  first += (long long)(u - b * p.L * p.Hkv) * tb;
  int entries = 0;
  if (tb > 0) {
    const int ctas = (int)(all_tiles < p.grid ? all_tiles : p.grid);
    entries = p.cparts * min(p.smax, cta_of(all_tiles, ctas, first + tb - 1) - cta_of(all_tiles, ctas, first) + 1);
  }
  const float2* part = p.part + (int64_t)u * p.cparts * p.smax * p.rs + row;
  float M = kEmptyMax;
  for (int s = 0; s < entries; ++s) M = fmaxf(M, part[(int64_t)s * p.rs].x);
  float Z = 0.f;
  for (int s = 0; s < entries; ++s) {
    const float2 v = part[(int64_t)s * p.rs];
    Z += v.y * exp2f(v.x - M);  // an empty pair has sum 0
  }
  const float l2 = Z > 0.f ? M + log2f(Z) : 0.f;
  nlse2[x] = -l2;
  if (lse_out) {
    const int h = u % p.Hkv, bl = u / p.Hkv;
    const int hq = h * p.g + row / p.w, wr = row % p.w;
    lse_out[((int64_t)bl * p.Hq + hq) * p.w + wr] = Z > 0.f ? l2 * 0.6931471805599453f : -INFINITY;
  }
}

// caller-supplied natural-log sum-exps [B, L, H_q, w] -> negated log2-domain values in the (unit, row) layout of pass 2;
// a row that saw no key (-inf) and the padding rows get the shift that turns every weight into 0
__global__ void score_rows_given_lse_kernel(RowParams p, const float* lse, float* nlse2, int total) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= total) return;
  const int u = x / p.rs, row = x % p.rs;
  clear_tail(p, u, row);
  float v = kEmptyMax;
  if (row < p.R) {
    const int h = u % p.Hkv, bl = u / p.Hkv;
    const int hq = h * p.g + row / p.w, wr = row % p.w;
    const float l = lse[((int64_t)bl * p.Hq + hq) * p.w + wr];
    if (l > -INFINITY) v = -l * kLog2e;
  }
  nlse2[x] = v;
}

template <int D, int PASS>
int launch_pass(const CUtensorMap& mk, const CUtensorMap& mq, const RowParams& p, int grid, cudaStream_t st) {
  using SL = RowSmem<D, PASS>;
  if (cudaFuncSetAttribute(score_rows_kernel<D, PASS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
      cudaSuccess)
    return MADAKV_ECUDA;
  score_rows_kernel<D, PASS><<<grid, kRowThreads, SL::kAlloc, st>>>(mk, mq, p);
  return MADAKV_OK;
}

}  // namespace

// parameters shared by the two-pass and the single-pass launch; false if the shape is outside this file's range
static bool rows_setup(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                       const int32_t* seq_len, float* psi, void* ws, RowParams& p, float*& lse2, CUtensorMap& mk,
                       CUtensorMap& mq, int& grid, int& rc) {
  const int g = c.n_q_heads / c.n_kv_heads;
  const int R = g * c.window;
  rc = MADAKV_EUNSUPPORTED;
  if (c.dtype != MADAKV_BF16 || R > 256 || c.window > 256 || g > 256) return false;
  const WsLayout wl = ws_layout(c);
  p.seq_len = seq_len;
  p.psi = psi;
  p.part = reinterpret_cast<float2*>((char*)ws + wl.score_part_off);
  lse2 = reinterpret_cast<float*>((char*)ws + wl.score_lse_off);
  p.lse2 = lse2;
  p.status = reinterpret_cast<int32_t*>(ws);
  p.B = c.batch;
  p.units = c.batch * c.n_layers * c.n_kv_heads;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = g;
  p.w = c.window;
  p.R = R;
  p.n_max = c.max_seq_len;
  p.causal = c.causal;
  p.smax = wide_max_runs(c);
  p.rs = (R + 31) / 32 * 32;  // row stride of the workspace arrays
  p.mblocks = R <= 128 ? 1 : 2;
  p.cparts = R <= 128 ? 4 : 2;
  p.n16 = (R + 15) / 16 * 16;
  p.scale2 = scale_of(c) * kLog2e;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    rc = MADAKV_ECUDA;
    return false;
  }
  const long long tiles = (long long)p.units * ((c.max_seq_len + kTileKeys - 1) / kTileKeys);
  if (tiles > 0x3fffffff) return false;
  if (sms > kWideMaxGrid) sms = kWideMaxGrid;
  grid = (int)(tiles < sms ? tiles : sms);
  p.grid = grid;
  if (!make_map(&mk, k, c.head_dim, c.max_seq_len, c.n_kv_heads, c.n_layers, c.batch, sk, kTileKeys, 1) ||
      !make_map(&mq, q, c.head_dim, c.window, c.n_q_heads, c.n_layers, c.batch, sq, c.window, g))
    return false;
  return true;
}

int launch_score_rows(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                      const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st) {
  if ((c.n_q_heads / c.n_kv_heads) * c.window <= 64) return MADAKV_EUNSUPPORTED;  // the TMEM-resident kernels' range
  RowParams p;
  float* lse2;
  CUtensorMap mk, mq;
  int grid, rc;
  // the workspace layout reserves (max, sum) pairs for [units, splits, column shares, rs]
  if (!rows_setup(c, q, sq, k, sk, seq_len, psi, ws, p, lse2, mk, mq, grid, rc)) return rc;
  const int total = p.units * p.rs;
  rc = c.head_dim == 128 ? launch_pass<128, 1>(mk, mq, p, grid, st) : launch_pass<64, 1>(mk, mq, p, grid, st);
  if (rc) return rc;
  score_rows_merge_kernel<<<(total + 255) / 256, 256, 0, st>>>(p, lse2, lse, total);
  rc = c.head_dim == 128 ? launch_pass<128, 2>(mk, mq, p, grid, st) : launch_pass<64, 2>(mk, mq, p, grid, st);
  if (rc) return rc;
  return launch_status();
}

// Single-pass scoring with the rows' log-sum-exps supplied by the caller: a conversion kernel, then pass 2 alone.
// Any bf16 shape with g * w <= 256.
int launch_score_lse_rows(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                          const int32_t* seq_len, const float* lse, float* psi, void* ws, cudaStream_t st) {
  RowParams p;
  float* lse2;
  CUtensorMap mk, mq;
  int grid, rc;
  if (!rows_setup(c, q, sq, k, sk, seq_len, psi, ws, p, lse2, mk, mq, grid, rc)) return rc;
  const int total = p.units * p.rs;
  score_rows_given_lse_kernel<<<(total + 255) / 256, 256, 0, st>>>(p, lse, lse2, total);
  rc = c.head_dim == 128 ? launch_pass<128, 2>(mk, mq, p, grid, st) : launch_pass<64, 2>(mk, mq, p, grid, st);
  if (rc) return rc;
  return launch_status();
}

}  // namespace madakv
