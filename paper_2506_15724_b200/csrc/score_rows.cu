// Stage 1, tensor-core path for wide windows (Eq. 7 with the softmax of Eq. 5): bf16 inputs with 64 < g * w <= 256
// window rows per KV head (grouped-query attention with many query heads per KV head).
//
// With that many rows the work per key byte is dominated by the exponentials (g * w of them per key and pass), not
// by HBM, and a per-key owner of all rows (as in the narrow-window kernels) would need hundreds of registers. So the
// tile is turned round: the window rows sit on M (one or two blocks of 128 rows), the 128 keys of a tile on N, and a
// thread of the epilogue owns ONE window row (a TMEM lane) and sees its logits for the keys of a tile as columns.
//   pass 1  per (unit, key split): running maximum and sum of exp2 of every row over the split's keys, in-thread
//           (per 16 columns: block maximum, one rescale, 16 exponentials); one (max, sum) pair per row and split
//   merge   per (unit, row): the pairs of all splits -> the row's log-sum-exp (a separate small kernel)
//   pass 2  per (unit, key split): logits recomputed with the tile turned back (128 keys on M, the window rows on N,
//           as in the narrow-window kernels): a thread owns one key and psi(i) = sum over rows of exp2(s - lse) is an
//           in-thread sum over the columns of its TMEM lane; the rows' negated log-sum-exps come as broadcast loads
// K is streamed twice (the second time mostly from HBM): for these shapes the exponentials take longer than either
// read. The passes are separate launches, so no CTA ever waits for another CTA. Warp roles: warp 0 TMA producer,
// warp 1 MMA issuer and TMEM owner, warps 2-17 epilogue. Two warps share each (TMEM lane quarter, row block) of
// pass 1 and each (lane quarter, accumulator buffer) of pass 2 and take one half of a tile's columns each: the
// exponentials are latency-bound with two warps per scheduler, four keep the special-function unit busy. In pass 1
// the halves publish separate (max, sum) pairs; in pass 2 the upper half hands its partial psi to the lower half
// through shared memory. TMEM lane quarter = warp % 4 throughout.
// Every wait is bounded: on expiry the kernel records MADAKV_ETIMEOUT, drains and returns.
#include "tc_common.cuh"

namespace madakv {
namespace {

constexpr int kRowThreads = 576;  // 2 + 16 warps
constexpr int kSplitKeys = 2048;  // keys per work item (16 tiles)

struct RowParams {
  const int32_t* seq_len;
  float* psi;        // [units, n_max]
  float2* part;      // ws: [units, splits, 2, rs] (max, sum) of every row over each half of a split's tiles
  const float* lse2; // ws: [units, rs] NEGATED log2-domain log-sum-exp, padding rows hold kEmptyMax (pass 2)
  int32_t* status;   // ws header
  int units, L, Hq, Hkv, g, w, R, n_max, causal, splits, rs, mblocks, n16;  // n16: R rounded up to 16
  float scale2;
};

template <int D>
struct RowSmem {
  static constexpr int kStages = D == 128 ? 3 : 6;
  static constexpr int kKBlocks = D / 64;
  static constexpr int kStageBytes = kTileKeys * D * 2;
  static constexpr int kQBytes = 256 * D * 2;  // up to two blocks of 128 rows
  static constexpr int kKOff = 0;
  static constexpr int kQOff = kStages * kStageBytes;
  static constexpr int kBarOff = kQOff + kQBytes;
  // full[kStages], empty[kStages], qfull, qempty, tfull[2], tempty[2], drain, xbar[8]
  static constexpr int kNumBars = 2 * kStages + 7 + 8;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kColOff = kMiscOff + 16;            // window position (row % w) of every row [256]
  static constexpr int kXchOff = kColOff + 256 * 4;        // pass 2: partial psi of the upper column halves [2][128]
  static constexpr int kTotal = kXchOff + 2 * 128 * 4;
  static constexpr int kAlloc = kTotal + 1024;
};

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kIdescRows = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);


template <int D, int PASS>
__global__ void __launch_bounds__(kRowThreads, 1)
score_rows_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q, RowParams p) {
  using SL = RowSmem<D>;
  constexpr int kStages = SL::kStages;
  constexpr int kKBlocks = SL::kKBlocks;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* k_s = smem + SL::kKOff;
  uint8_t* q_s = smem + SL::kQOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBarOff);
  uint64_t* full = bars;               // [kStages] TMA -> MMA
  uint64_t* empty = bars + kStages;    // [kStages] MMA -> TMA
  uint64_t* qfull = empty + kStages;   // [1]       TMA -> MMA (queries of the item's unit)
  uint64_t* qempty = qfull + 1;        // [1]       MMA -> TMA
  uint64_t* tfull = qempty + 1;        // [2]       MMA -> epilogue
  uint64_t* tempty = tfull + 2;        // [2]       epilogue -> MMA
  uint64_t* drain = tempty + 2;        // [1]
  uint64_t* xbar = drain + 1;          // [8]       pass 2: upper half -> lower half of a (buffer, lane quarter) warp pair
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(smem + SL::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kMiscOff + 4);
  int* rowpos = reinterpret_cast<int*>(smem + SL::kColOff);
  float* xch = reinterpret_cast<float*>(smem + SL::kXchOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // epilogue threads in use. Pass 1: two per window row (column halves); pass 2: all 16 warps, 8 per accumulator buffer
  const int n_epi = PASS == 1 ? 256 * p.mblocks : 512;
  const int total_items = p.units * p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(qfull, 1);
    mbar_init(qempty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], PASS == 1 ? (uint32_t)n_epi : 256u);
    }
    mbar_init(drain, 1);
    for (int i = 0; i < 8; ++i) mbar_init(&xbar[i], 32);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows R..255 of the Q buffer are never written by TMA: keep them zero so their logits are 0
  for (int x = threadIdx.x; x < SL::kQBytes / 16; x += kRowThreads)
    reinterpret_cast<uint4*>(q_s)[x] = make_uint4(0, 0, 0, 0);
  for (int x = threadIdx.x; x < 256; x += kRowThreads) rowpos[x] = x % p.w;
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

  // item -> (unit, first key, number of tiles); an item beyond its sequence has no tiles
  auto item_of = [&](int item, int& u, int& key_begin, int& tiles) {
    u = item / p.splits;
    const int split = item % p.splits;
    const int b = u / (p.Hkv * p.L);
    const int n = clamped_len(p.seq_len, b, p.n_max);
    key_begin = split * kSplitKeys;
    tiles = key_begin < n ? (min(n, key_begin + kSplitKeys) - key_begin + kTileKeys - 1) / kTileKeys : 0;
  };

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      const uint64_t pol_k = l2_policy_evict_first();
      const uint64_t pol_q = l2_policy_evict_last();
      int stage = 0;
      uint32_t stage_par = 0, q_par = 0;
      bool ok = true;
      for (int it = blockIdx.x; ok && it < total_items; it += gridDim.x) {
        const int item = PASS == 1 ? it : total_items - 1 - it;  // pass 2 backwards: pass 1's last K is still in L2
        int u, key_begin, tiles;
        item_of(item, u, key_begin, tiles);
        if (tiles == 0) continue;
        const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
        ok = mbar_wait(qempty, q_par ^ 1, abort_flag, p.status, kSiteQEmpty);
        if (!ok) break;
        q_par ^= 1;
        mbar_expect_tx(qfull, (uint32_t)(p.R * 128 * kKBlocks));
        for (int kb = 0; kb < kKBlocks; ++kb)
          tma_load_5d(q_s + kb * 256 * 128, &tmap_q, qfull, kb * 64, 0, h * p.g, l, b, pol_q);
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
      if (!ok) {  // abandoned: give copies in flight time to land before the CTA's shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer: D[row, key] = Q_block . K_tile^T
    if (lane == 0) {
      const uint32_t k_lo0 = smem_desc_lo(smem_u32(k_s)), q_lo0 = smem_desc_lo(smem_u32(q_s));
      int stage = 0, n_tile = 0;
      uint32_t stage_par = 0, q_par = 0;
      bool ok = true;
      for (int it = blockIdx.x; ok && it < total_items; it += gridDim.x) {
        const int item = PASS == 1 ? it : total_items - 1 - it;  // pass 2 backwards: pass 1's last K is still in L2
        int u, key_begin, tiles;
        item_of(item, u, key_begin, tiles);
        if (tiles == 0) continue;
        ok = mbar_wait(qfull, q_par, abort_flag, p.status, kSiteQFull);
        if (!ok) break;
        q_par ^= 1;
        for (int t = 0; t < tiles; ++t, ++n_tile) {
          const int buf = n_tile & 1;
          const uint32_t use_par = (uint32_t)(n_tile >> 1) & 1u;
          ok = mbar_wait(&tempty[buf], use_par ^ 1, abort_flag, p.status, kSiteTEmpty) &&
               mbar_wait(&full[stage], stage_par, abort_flag, p.status, kSiteFull);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + (uint32_t)stage * (SL::kStageBytes >> 4);
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
          } else {  // D[key, row]: the K tile is operand A, all n16 query rows operand B
            const uint32_t d_tmem = tmem_base + buf * 256;
            const uint32_t idesc = instr_desc_bf16(p.n16);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const int kb = ks >> 2, kk = ks & 3;
              umma_bf16(d_tmem, k_lo + ((kb * kTileKeys * 128 + kk * 32) >> 4),
                        q_lo0 + ((kb * 256 * 128 + kk * 32) >> 4), idesc, ks > 0 ? 1u : 0u);
            }
          }
          umma_commit(&empty[stage]);  // the K stage may be refilled
          umma_commit(&tfull[buf]);    // the accumulators are ready
          if (++stage == kStages) {
            stage = 0;
            stage_par ^= 1;
          }
        }
        if (!ok) break;
        umma_commit(qempty);  // the queries may be replaced once this item's MMAs are done
      }
      if (!ok) {  // abandoned: TMEM may only be freed once this thread's MMAs have completed
        umma_commit(drain);
        const long long t0 = clock64();
        while (!mbar_try(drain, 0) && clock64() - t0 < 20000000ll) __nanosleep(200);
      }
    }
  } else if (PASS == 2 || (((warp - 2) >> 2) & 1) < p.mblocks) {
    // ================================================================ epilogue: a thread owns one window row (pass 1)
    // or one key of every other tile (pass 2), in both cases for one half of the tile's columns
    const int ew = warp - 2;
    const int mb = (ew >> 2) & 1;                  // row block (pass 1) or accumulator buffer (pass 2)
    const int half = ew >> 3;                      // column half
    const int quarter = warp & 3;                  // TMEM lanes [32 * quarter, 32 * quarter + 32)
    const int row = mb * 128 + quarter * 32 + lane;
    const int eidx = ew * 32 + lane;               // index among the epilogue threads in use
    const uint32_t tlane = tmem_base + ((uint32_t)(quarter * 32) << 16) + mb * 128;
    const float masked = kEmptyMax;                // raw value given to a logit the row may not see
    int n_tile = 0;
    uint32_t x_par = 0;  // pass 2: phase of the pair's exchange barrier
    bool ok = true;
    for (int it = blockIdx.x; ok && it < total_items; it += gridDim.x) {
      const int item = PASS == 1 ? it : total_items - 1 - it;
      int u, key_begin, tiles;
      item_of(item, u, key_begin, tiles);
      const int split = item % p.splits;
      const int b = u / (p.Hkv * p.L);
      const int n = clamped_len(p.seq_len, b, p.n_max);
      float* psi = p.psi + (int64_t)u * p.n_max;
      // keys the row may see: [0, vis)
      int vis = 0;
      if (row < p.R) {
        const int pos = n - p.w + row % p.w;
        if (pos >= 0) vis = p.causal ? pos + 1 : n;
      }
      if (PASS == 1) {
        float m = 4.f * kEmptyMax, z = 0.f;  // scaled (log2) domain; below any masked logit
        for (int t = 0; t < tiles; ++t, ++n_tile) {
          const int buf = n_tile & 1;
          ok = __all_sync(0xffffffffu, mbar_wait(&tfull[buf], (uint32_t)(n_tile >> 1) & 1u, abort_flag, p.status, kSiteTile));
          if (!ok) break;
          tc_fence_after();
          const int key0 = key_begin + t * kTileKeys;
          const uint32_t taddr = tlane + buf * 256;
          uint32_t ra[16], rb[16];
          auto block = [&](uint32_t (&r)[16], int c) {  // columns 16c .. 16c + 15 of the tile
            if (key0 + 16 * c + 16 > vis) {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (key0 + 16 * c + i >= vis) r[i] = __float_as_uint(masked);
            }
            float t8[8];  // maximum and sums as trees: short dependency chains (two epilogue warps per scheduler)
#pragma unroll
            for (int i = 0; i < 8; ++i) t8[i] = fmaxf(__uint_as_float(r[i]), __uint_as_float(r[i + 8]));
            const float bm = fmaxf(fmaxf(fmaxf(t8[0], t8[4]), fmaxf(t8[1], t8[5])),
                                   fmaxf(fmaxf(t8[2], t8[6]), fmaxf(t8[3], t8[7])));
            const float mn = fmaxf(m, bm * p.scale2);
            z *= ex2(m - mn);
            m = mn;
            const uint64_t nm2 = pack2(-mn, -mn), sc2 = pack2(p.scale2, p.scale2);
            uint64_t e[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float lo, hi;
              unpack2(fma2(pack2u(r[2 * i], r[2 * i + 1]), sc2, nm2), lo, hi);
              e[i] = pack2(ex2(lo), ex2(hi));
            }
            float lo, hi;
            unpack2(add2(add2(add2(e[0], e[1]), add2(e[2], e[3])), add2(add2(e[4], e[5]), add2(e[6], e[7]))), lo, hi);
            z += lo + hi;
          };
          const int c0 = 4 * half;  // this warp's 64 columns
          tmem_ld16_issue(taddr + c0 * 16, ra);
#pragma unroll 1
          for (int c = c0; c < c0 + 4; c += 2) {
            tmem_ld_wait16(ra);
            tmem_ld16_issue(taddr + (c + 1) * 16, rb);
            block(ra, c);
            tmem_ld_wait16(rb);
            if (c + 2 < c0 + 4) tmem_ld16_issue(taddr + (c + 2) * 16, ra);
            block(rb, c + 1);
          }
          tc_fence_before();
          mbar_arrive(&tempty[buf]);
        }
        if (!ok) break;
        if (row < p.R) {
          // a row that saw no visible key only summed masked entries: it is recorded as empty
          const bool none = m < 0.5f * kEmptyMax * p.scale2;
          p.part[(((int64_t)u * p.splits + split) * 2 + half) * p.rs + row] =
              none ? make_float2(kEmptyMax, 0.f) : make_float2(m, z);
        }
      } else {
        // group (warp - 2) / 4 owns accumulator buffer `group` and with it every other tile; this thread's key is
        // key0 + 32 * quarter + lane and its logits against the n16 window rows are the columns of its TMEM lane
        const int group = mb;
        const int pair = group * 4 + quarter;  // the two warps (column halves) that share a key
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + group * 256;
        const ulonglong2* ns = reinterpret_cast<const ulonglong2*>(p.lse2 + (int64_t)u * p.rs);
        const uint64_t sc2 = pack2(p.scale2, p.scale2);
        const int nblk = p.n16 >> 4, nlow = (nblk + 1) >> 1;
        const int cb = half ? nlow : 0, ce = half ? nblk : nlow;  // this warp's blocks of 16 window rows
        for (int t = 0; t < tiles; ++t, ++n_tile) {
          if ((n_tile & 1) != group) continue;
          ok = __all_sync(0xffffffffu, mbar_wait(&tfull[group], (uint32_t)(n_tile >> 1) & 1u, abort_flag, p.status, kSiteTile));
          if (!ok) break;
          tc_fence_after();
          const int key0 = key_begin + t * kTileKeys;
          const int key = key0 + quarter * 32 + lane;
          // a tile below the window's first position is seen in full by every row; otherwise every logit is checked
          const bool plain = key0 + kTileKeys <= n - p.w;
          uint64_t acc = 0ull;
          uint32_t ra[16], rb[16];
          auto block = [&](uint32_t (&r)[16], int c) {  // window rows 16c .. 16c + 15
            uint64_t sh[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const ulonglong2 v = __ldg(ns + 4 * c + j);
              sh[2 * j] = v.x;
              sh[2 * j + 1] = v.y;
            }
            if (!plain) {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const int pos = n - p.w + rowpos[16 * c + i];
                const int vis = pos < 0 ? 0 : (p.causal ? pos + 1 : n);
                if (key >= vis) r[i] = __float_as_uint(kEmptyMax);
              }
            }
            uint64_t e[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float lo, hi;
              unpack2(fma2(pack2u(r[2 * i], r[2 * i + 1]), sc2, sh[i]), lo, hi);
              e[i] = pack2(ex2(lo), ex2(hi));
            }
            acc = add2(acc, add2(add2(add2(e[0], e[1]), add2(e[2], e[3])), add2(add2(e[4], e[5]), add2(e[6], e[7]))));
          };
          if (cb < ce) tmem_ld16_issue(taddr + cb * 16, ra);
#pragma unroll 1
          for (int c = cb; c < ce; c += 2) {
            tmem_ld_wait16(ra);
            if (c + 1 < ce) tmem_ld16_issue(taddr + (c + 1) * 16, rb);
            block(ra, c);
            if (c + 1 < ce) {
              tmem_ld_wait16(rb);
              if (c + 2 < ce) tmem_ld16_issue(taddr + (c + 2) * 16, ra);
              block(rb, c + 1);
            }
          }
          float lo, hi;
          unpack2(acc, lo, hi);
          if (half) {  // hand the partial sum to the warp of the lower half
            xch[group * 128 + quarter * 32 + lane] = lo + hi;
            mbar_arrive(&xbar[pair]);
          } else {
            ok = __all_sync(0xffffffffu, mbar_wait(&xbar[pair], x_par, abort_flag, p.status, kSiteFlag));
            x_par ^= 1;
            if (!ok) break;
            const float tot = (lo + hi) + xch[group * 128 + quarter * 32 + lane];
            if (key < p.n_max) psi[key] = key < n ? tot : 0.f;
          }
          // the buffer is handed back only after the exchange: the upper half writes its next partial sum after the
          // next tile of this buffer has been computed, which needs every arrival of this one
          tc_fence_before();
          mbar_arrive(&tempty[group]);
        }
        if (!ok) break;
        // keys of the item beyond the sequence
        for (int key = key_begin + tiles * kTileKeys + eidx; key < min(key_begin + kSplitKeys, p.n_max); key += n_epi)
          psi[key] = 0.f;
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

// merge: per (unit, row) the (max, sum) pairs of all splits, in split order -> log2-domain log-sum-exp, stored
// negated (pass 2 adds it inside a fused multiply-add); padding rows get a shift that turns every weight into 0
__global__ void score_rows_merge_kernel(RowParams p, float* nlse2, float* lse_out, int total) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= total) return;
  const int u = x / p.rs, row = x % p.rs;
  if (row >= p.R) {
    nlse2[x] = kEmptyMax;
    return;
  }
  const int entries = 2 * p.splits;  // column halves of every split
  const float2* part = p.part + (int64_t)u * entries * p.rs + row;
  float M = kEmptyMax;
  for (int s = 0; s < entries; ++s) M = fmaxf(M, part[(int64_t)s * p.rs].x);
  float Z = 0.f;
  for (int s = 0; s < entries; ++s) {
    const float2 v = part[(int64_t)s * p.rs];
    Z += v.y * exp2f(v.x - M);  // an empty split has sum 0
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
  float v = kEmptyMax;
  if (row < p.R) {
    const int h = u % p.Hkv, bl = u / p.Hkv;
    const int hq = h * p.g + row / p.w, wr = row % p.w;
    const float l = lse[((int64_t)bl * p.Hq + hq) * p.w + wr];
    if (l > -INFINITY) v = -l * kLog2e;
  }
  nlse2[x] = v;
}

template <int D>
int run_rows(const CUtensorMap& mk, const CUtensorMap& mq, RowParams p, float* lse2, float* lse_out, int grid,
             cudaStream_t st) {
  using SL = RowSmem<D>;
  if (cudaFuncSetAttribute(score_rows_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
          cudaSuccess ||
      cudaFuncSetAttribute(score_rows_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
          cudaSuccess)
    return MADAKV_ECUDA;
  score_rows_kernel<D, 1><<<grid, kRowThreads, SL::kAlloc, st>>>(mk, mq, p);
  const int total = p.units * p.rs;
  score_rows_merge_kernel<<<(total + 255) / 256, 256, 0, st>>>(p, lse2, lse_out, total);
  score_rows_kernel<D, 2><<<grid, kRowThreads, SL::kAlloc, st>>>(mk, mq, p);
  return launch_status();
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
  p.units = c.batch * c.n_layers * c.n_kv_heads;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = g;
  p.w = c.window;
  p.R = R;
  p.n_max = c.max_seq_len;
  p.causal = c.causal;
  p.splits = (c.max_seq_len + kSplitKeys - 1) / kSplitKeys;
  p.rs = (R + 31) / 32 * 32;  // row stride of the workspace arrays
  p.mblocks = R <= 128 ? 1 : 2;
  p.n16 = (R + 15) / 16 * 16;
  p.scale2 = scale_of(c) * kLog2e;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    rc = MADAKV_ECUDA;
    return false;
  }
  const long long items = (long long)p.units * p.splits;
  if (items > 0x3fffffff) return false;
  grid = (int)(items < sms ? items : sms);
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
  // the workspace layout reserves (max, sum) pairs for [units, splits, 2 halves, rs]
  if (!rows_setup(c, q, sq, k, sk, seq_len, psi, ws, p, lse2, mk, mq, grid, rc)) return rc;
  return c.head_dim == 128 ? run_rows<128>(mk, mq, p, lse2, lse, grid, st) : run_rows<64>(mk, mq, p, lse2, lse, grid, st);
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
  if (c.head_dim == 128) {
    using SL = RowSmem<128>;
    if (cudaFuncSetAttribute(score_rows_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
        cudaSuccess)
      return MADAKV_ECUDA;
    score_rows_kernel<128, 2><<<grid, kRowThreads, SL::kAlloc, st>>>(mk, mq, p);
  } else {
    using SL = RowSmem<64>;
    if (cudaFuncSetAttribute(score_rows_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
        cudaSuccess)
      return MADAKV_ECUDA;
    score_rows_kernel<64, 2><<<grid, kRowThreads, SL::kAlloc, st>>>(mk, mq, p);
  }
  return launch_status();
}

}  // namespace madakv
