// Stage 1, Blackwell tensor-core path (Eq. 7 with the softmax of Eq. 5) for bf16 inputs with g * w <= 64 window rows.
//
// One persistent kernel streams every K tile exactly once from HBM and a second time from L2:
//   - the window-QK^T tile is a tcgen05.mma with the 128 keys of a tile on M, the g*w window rows on N and head_dim
//     on K; operands are staged in shared memory by TMA (128-byte swizzle), the fp32 accumulator lives in TMEM;
//   - a softmax over keys needs every row's log-sum-exp before any normalised weight can be summed over rows, so
//     the work is cut into items of 4 or 8 tiles in two phases: phase-1 items produce per-row (max, sum exp2)
//     partials, phase-2 items recompute the logits and emit psi. The item list interleaves phase 2 of chunk t with
//     phase 1 of chunk t + lag, so the second read of a K chunk comes a bounded number of chunks after the first
//     and is served by the L2 (phase-1 loads ask L2 to keep the lines, phase-2 loads to drop them);
//   - every epilogue warp publishes, per window row, the partial of its quarter of a phase-1 item and bumps that
//     row's counter of the unit; the lane whose bump completes the unit merges the row's partials (in a fixed order,
//     so the bits do not depend on who finishes) into the row's log-sum-exp and flags it. A phase-2 item waits (bounded)
//     for the flags of its unit. Every item only depends on items earlier in the global order and every CTA walks
//     its items in that order, so with all CTAs resident (grid <= SM count, one CTA per SM) the waits always end.
// Warp roles: warp 0 TMA producer; warps 1 and 10 MMA issuers that take alternate K tiles (an MMA of N <= 64 keeps
// the tensor pipe busy for ~45 cycles, about as long as one thread needs to poll the barriers of the next tile, so
// two issuers keep the pipe fed). Both issuers wait on the "landed" barrier of EVERY K tile, in load order, also of
// the tiles the other one issues, and a stage is only refilled once the tile's MMAs have completed AND the other
// issuer has reported that it saw the tile land: a barrier that is tested by parity must be taken phase by phase
// by each of its waiters, and none of them may fall two phases behind. (An issuer that only looked at its own
// tiles could test a stage's barrier one phase early when loads complete out of order, e.g. an L2 hit overtaking
// an HBM miss, and run ahead of the data; the producer then armed that barrier twice in one phase, which ended in
// a launch failure. An issuer that took every phase but did not gate the refill could fall two phases behind and
// wait for ever.) Warps 2-9 epilogue: two groups of four warps
// that take alternate work items, the four warps of a group being the four TMEM lane quarters. A thread owns one key of a tile and all window rows
// of it, so psi(i) is an in-thread sum over N. The epilogue warps never synchronise with one another: every warp
// keeps its own copy of the row shifts and visibility bounds, publishes its own (max, sum) partial per row and
// item, and counts it on the row's counter. The accumulators of a whole item stay in TMEM, so phase 1 reads them
// twice (row maximum, then one exp2 per logit) instead of rescaling a running sum; every tile's accumulator is
// handed back to the MMA warp right after its last read.
// Every wait is bounded: on expiry the kernel records MADAKV_ETIMEOUT, lets its copies drain, frees TMEM and returns.
#include "tc_common.cuh"

namespace madakv {
namespace {

constexpr int kItemCols = 256;                      // TMEM columns of one work item's accumulators
constexpr int kStagesD128 = 5;
constexpr int kThreads = 352;                        // TMA warp, MMA warp, 8 epilogue warps, second MMA warp
constexpr int kReady = 1 << 16;                     // added to a row counter when the row's log-sum-exp is published

static_assert(kTileKeys * (kItemCols / 64) == kScoreTcChunk, "the workspace is sized for the smallest work item");

struct TcParams {
  const int32_t* seq_len;
  float* psi;        // [units, n_max]
  float* lse_out;    // natural log [B,L,Hq,w] or null
  float2* part;      // ws: [units, cpu, 4 lane quarters, NPAD]
  int32_t* done;     // ws: [units, NPAD] partials published per window row; + kReady once lse2 is published
  float* lse2;       // ws: [units, NPAD] log2-domain log-sum-exp of every window row
  int32_t* status;   // ws header
  int units, L, Hq, Hkv, g, w, R, n_max, cpu, causal, lag;
  float scale2;
  long long flag_wait_cycles;  // bound of the wait for another CTA's row flags (kWaitCycles unless a test shortens it)
  int hold_flags;              // failure-path test only: the rows' log-sum-exps are computed but never flagged
};

// ------------------------------------------------------------------------------------------------ work list
struct Item {
  int phase;  // 1 or 2
  int unit, chunk;
};

// The idx-th item of CTA `cta` (grid G): first its share of the phase-1 prologue (the first `lag` chunks), then its
// super-items t = cta, cta + G, ...: phase 2 of chunk t and phase 1 of chunk t + lag (in alternating order).
__device__ __forceinline__ bool get_item(int cta, int G, int idx, int total_chunks, int lag, int cpu, Item& it) {
  const int pro = min(lag, total_chunks);
  const int my_pro = cta < pro ? (pro - cta + G - 1) / G : 0;
  int j, phase;
  if (idx < my_pro) {
    j = cta + idx * G;
    phase = 1;
  } else {
    const int k = idx - my_pro;
    // super-item slots: 2 per t while t + lag < total, then 1
    const int two = max(total_chunks - lag, 0);               // t in [0, two) have both halves
    const int my_two = cta < two ? (two - cta + G - 1) / G : 0;
    if (k < 2 * my_two) {
      // the two halves swap places in every other super-item, so that each of the two epilogue groups (which take
      // alternate items) gets phase-1 and phase-2 items in turn: a phase-1 item costs about twice a phase-2 item
      const int t = cta + (k >> 1) * G;
      if (((k & 1) != 0) != (((k >> 1) & 1) != 0)) { j = t + lag; phase = 1; } else { j = t; phase = 2; }
    } else {
      const int k2 = k - 2 * my_two;
      const int t = cta + (my_two + k2) * G;
      if (t >= total_chunks) return false;
      j = t;
      phase = 2;
    }
  }
  it.phase = phase;
  it.unit = j / cpu;
  it.chunk = j % cpu;
  return true;
}

template <int D, int NPAD>
struct SmemLayout {
  static constexpr int kStages = (D == 128 ? 1 : 2) * (NPAD == 32 ? kStagesD128 : kStagesD128 - 1);
  static constexpr int kKBlocks = D / 64;
  static constexpr int kStageBytes = kTileKeys * D * 2;
  static constexpr int kQBytes = NPAD * D * 2;
  static constexpr int kItemTiles = kItemCols / NPAD;     // tiles per work item: 8 (NPAD 32) or 4 (NPAD 64)
  static constexpr int kItemKeys = kItemTiles * kTileKeys;
  static constexpr int kItemBufs = kTmemCols / kItemCols;  // accumulator sets (one work item each) in TMEM
  static constexpr int kKOff = 0;
  static constexpr int kQOff = kStages * kStageBytes;
  static constexpr int kBarOff = kQOff + 2 * kQBytes;
  // full[kStages], seen[kStages], qfull[2], qempty[2], tfull / tempty[kItemBufs * kItemTiles], drain[2]
  static constexpr int kNumBars = 2 * kStages + 4 + 2 * kItemBufs * kItemTiles + 2;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  // misc: tmem base (4), abort flag (4), producer's stage ring (kStages <= 10 words); then per epilogue warp:
  // shift[NPAD] (negated row maxima or log-sum-exps), vis[NPAD], a padded 32 x 33 transpose tile
  static constexpr int kWarpOff = kMiscOff + 48;
  static constexpr int kWarpBytes = NPAD * 4 + NPAD * 4 + 32 * 33 * 4;
  static constexpr int kTotal = kWarpOff + 8 * kWarpBytes;
  static constexpr int kAlloc = kTotal + 1024;  // slack for the 1024-byte alignment of the operand tiles
  static_assert(kItemBufs == 2, "each epilogue group owns one accumulator set");
};

template <int D, int NPAD>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q, TcParams p) {
  using SL = SmemLayout<D, NPAD>;
  constexpr int kStages = SL::kStages;
  constexpr int kKBlocks = SL::kKBlocks;
  constexpr int kItemBufs = SL::kItemBufs;
  constexpr int kItemTiles = SL::kItemTiles;
  constexpr int kItemKeys = SL::kItemKeys;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* k_s = smem + SL::kKOff;
  uint8_t* q_s = smem + SL::kQOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBarOff);
  uint64_t* full = bars;                               // [kStages]                TMA -> MMA
  uint64_t* seen = bars + kStages;                     // [kStages]  the MMA warp that does not issue a tile -> TMA
  uint64_t* qfull = bars + 2 * kStages;                // [2]
  uint64_t* qempty = qfull + 2;                        // [2]
  uint64_t* tfull = qempty + 2;                        // [kItemBufs][kItemTiles]  MMA -> epilogue and TMA, per tile
  uint64_t* tempty = tfull + kItemBufs * kItemTiles;   // [kItemBufs][kItemTiles]  epilogue -> MMA, one per tile
  uint64_t* drain = tempty + kItemBufs * kItemTiles;   // [2] used only when the kernel gives up
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(smem + SL::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kMiscOff + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_chunks = p.units * p.cpu;

  // ---- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&seen[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&qfull[i], 1);
      mbar_init(&qempty[i], 2);  // both MMA warps commit
      mbar_init(&drain[i], 1);
    }
    for (int i = 0; i < kItemBufs * kItemTiles; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], 128);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows R..NPAD-1 of both Q buffers are never written by TMA: keep them zero so their logits are 0
  for (int x = threadIdx.x; x < 2 * SL::kQBytes / 16; x += kThreads)
    reinterpret_cast<uint4*>(q_s)[x] = make_uint4(0, 0, 0, 0);
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

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      const uint64_t pol_keep = l2_policy_evict_last(), pol_drop = l2_policy_evict_first();
      // A K stage may be refilled once the MMAs of the tile that used it last have completed. That event is the
      // tile's tfull barrier (the MMA warp commits once per tile). stage_user remembers which accumulator slot that
      // tile went to; slot_par remembers, per slot, the parity of the latest use of the slot that this thread has
      // loaded or passed (a slot of an item's unused tail is committed without a load). Waiting for that latest use
      // is unambiguous (the barrier cannot be more than one phase beyond it, because the next use needs this thread)
      // and implies the completion of every earlier use, the one that read the stage included. Short items can
      // bring a slot round again within fewer tiles than there are stages, so the parity of the stage's own tile
      // would not do.
      volatile uint32_t* stage_user = reinterpret_cast<volatile uint32_t*>(smem + SL::kMiscOff + 8);
      for (int s2 = 0; s2 < kStages; ++s2) stage_user[s2] = 0;
      uint32_t slot_par = 0;  // bit per slot (kItemBufs * kItemTiles <= 16)
      int stage = 0;
      uint32_t lap_par = 0;  // parity of the number of times the stage ring has been gone round
      int qi = 0;
      uint32_t q_par = 0;
      int active = 0;
      bool ok = true;
      Item it;
      for (int idx = 0; ok && get_item(blockIdx.x, gridDim.x, idx, total_chunks, p.lag, p.cpu, it); ++idx) {
        const int h = it.unit % p.Hkv, l = (it.unit / p.Hkv) % p.L, b = it.unit / (p.Hkv * p.L);
        const int n = clamped_len(p.seq_len, b, p.n_max);
        const int key_begin = it.chunk * kItemKeys;
        if (key_begin >= n) continue;  // nothing to load for this item
        const int ib = active % kItemBufs;
        const uint32_t use_par = (uint32_t)(active / kItemBufs) & 1u;
        ++active;
        // window queries of the unit
        ok = mbar_wait(&qempty[qi], q_par ^ 1, abort_flag, p.status, kSiteQEmpty);
        if (!ok) break;
        mbar_expect_tx(&qfull[qi], (uint32_t)(p.R * 128 * kKBlocks));
        for (int kb = 0; kb < kKBlocks; ++kb)
          tma_load_5d(q_s + qi * SL::kQBytes + kb * NPAD * 128, &tmap_q, &qfull[qi], kb * 64, 0, h * p.g, l, b,
                      pol_keep);
        qi ^= 1;
        if (qi == 0) q_par ^= 1;
        const uint64_t pol = it.phase == 1 ? pol_keep : pol_drop;
        for (int t = 0; t < kItemTiles; ++t) {
          const int key0 = key_begin + t * kTileKeys;
          const int slot = ib * kItemTiles + t;
          if (key0 >= n) {  // not loaded; the MMA warp commits its barrier all the same
            slot_par = (slot_par & ~(1u << slot)) | (use_par << slot);
            continue;
          }
          const uint32_t prev = stage_user[stage];
          if (prev & 0x200u)  // the stage's last tile: its MMAs are done, and the other MMA warp has seen it land
            ok = mbar_wait(&tfull[prev & 0xffu], (slot_par >> (prev & 0xffu)) & 1u, abort_flag, p.status, kSiteStage) &&
                 mbar_wait(&seen[stage], lap_par ^ 1u, abort_flag, p.status, kSiteStage);
          if (!ok) break;
          stage_user[stage] = (uint32_t)slot | 0x200u;
          slot_par = (slot_par & ~(1u << slot)) | (use_par << slot);
          mbar_expect_tx(&full[stage], (uint32_t)SL::kStageBytes);
          for (int kb = 0; kb < kKBlocks; ++kb)
            tma_load_5d(k_s + stage * SL::kStageBytes + kb * kTileKeys * 128, &tmap_k, &full[stage], kb * 64, key0, h,
                        l, b, pol);
          if (++stage == kStages) {
            stage = 0;
            lap_par ^= 1u;
          }
        }
      }
      if (!ok) {  // abandoned: give copies in flight time to land before the CTA's shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ================================================================ MMA issuers: the loaded K tiles of the CTA,
    // counted in load order, go to the two warps in turn
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(NPAD);
      const int me = warp == 1 ? 0 : 1;
      int turn = 0;  // parity of the running count of loaded tiles
      const uint32_t k_lo0 = smem_desc_lo(smem_u32(k_s)), q_lo0 = smem_desc_lo(smem_u32(q_s));
      int stage = 0;
      uint32_t stage_par = 0;
      int qi = 0;
      uint32_t q_par = 0;
      int active = 0;  // active items issued so far; item k uses accumulator set k % kItemBufs
      bool ok = true;
      Item it;
      for (int idx = 0; ok && get_item(blockIdx.x, gridDim.x, idx, total_chunks, p.lag, p.cpu, it); ++idx) {
        const int b = it.unit / (p.Hkv * p.L);
        const int n = clamped_len(p.seq_len, b, p.n_max);
        const int key_begin = it.chunk * kItemKeys;
        if (key_begin >= n) continue;
        const int ib = active % kItemBufs;
        const uint32_t use_par = (uint32_t)(active / kItemBufs) & 1u;
        ok = mbar_wait(&qfull[qi], q_par, abort_flag, p.status, kSiteQFull);
        if (!ok) break;
        const uint32_t q_lo = q_lo0 + (uint32_t)qi * (SL::kQBytes >> 4);
        for (int t = 0; t < kItemTiles; ++t) {
          const int key0 = key_begin + t * kTileKeys;
          if (key0 < n) {
            // the K tile must have landed (both warps take every stage barrier, phase by phase) ...
            ok = mbar_wait(&full[stage], stage_par, abort_flag, p.status, kSiteFull);
            if (!ok) break;
            if (turn == me) {
              // ... and the tile's accumulator slot must have been read for the last time
              ok = mbar_wait(&tempty[ib * kItemTiles + t], use_par ^ 1, abort_flag, p.status, kSiteTEmpty);
              if (!ok) break;
              tc_fence_after();
              const uint32_t k_lo = k_lo0 + (uint32_t)stage * (SL::kStageBytes >> 4);
              const uint32_t d_tmem = tmem_base + ib * kItemCols + t * NPAD;
#pragma unroll
              for (int ks = 0; ks < D / 16; ++ks) {
                const int kb = ks >> 2, kk = ks & 3;
                umma_bf16(d_tmem, k_lo + ((kb * kTileKeys * 128 + kk * 32) >> 4),
                          q_lo + ((kb * NPAD * 128 + kk * 32) >> 4), idesc, ks > 0 ? 1u : 0u);
              }
              // one commit per tile: the accumulator is ready for the epilogue, and the K stage may be refilled
              umma_commit(&tfull[ib * kItemTiles + t]);
            } else {
              mbar_arrive(&seen[stage]);  // this warp has taken the stage's phase; it may be refilled
            }
            turn ^= 1;
            if (++stage == kStages) {
              stage = 0;
              stage_par ^= 1;
            }
          } else if ((t & 1) == me) {
            umma_commit(&tfull[ib * kItemTiles + t]);  // every tile barrier completes once per use of the set
          }
        }
        if (!ok) break;
        umma_commit(&qempty[qi]);  // the Q buffer may be refilled once both warps' MMAs of this item are done
        qi ^= 1;
        if (qi == 0) q_par ^= 1;
        ++active;
      }
      if (!ok) {
        // abandoned: TMEM may only be freed once this thread's MMAs have completed
        umma_commit(&drain[me]);
        const long long t0 = clock64();
        while (!mbar_try(&drain[me], 0) && clock64() - t0 < 20000000ll) __nanosleep(200);
      }
    }
  } else {
    // ================================================================ epilogue: two groups of four warps; group e
    // takes the active items of its parity, warp = TMEM lane quarter. A thread owns one key of each tile. The warps
    // run independently of one another.
    constexpr int kBlocks = NPAD / 16;              // 16-row blocks per tile
    const int grp = (warp - 2) >> 2;              // 0 or 1
    const int quarter = warp & 3;                 // TMEM lanes [32 * quarter, 32 * quarter + 32)
    const int et = (quarter << 5) | lane;         // key index inside the tile
    uint8_t* wbase = smem + SL::kWarpOff + (warp - 2) * SL::kWarpBytes;
    float* shift_s = reinterpret_cast<float*>(wbase);
    int* vis_s = reinterpret_cast<int*>(wbase + NPAD * 4);
    float* tr = reinterpret_cast<float*>(wbase + NPAD * 8);
    const uint64_t* shift2 = reinterpret_cast<const uint64_t*>(shift_s);
    const uint64_t scale2x = pack2(p.scale2, p.scale2);
    int active = 0;
    bool ok = true;
    Item it;
    for (int idx = 0; ok && get_item(blockIdx.x, gridDim.x, idx, total_chunks, p.lag, p.cpu, it); ++idx) {
      const int h = it.unit % p.Hkv, bl = it.unit / p.Hkv, b = bl / p.L;
      const int n = clamped_len(p.seq_len, b, p.n_max);
      const int key_begin = it.chunk * kItemKeys;
      float* psi = p.psi + (int64_t)it.unit * p.n_max;
      if (key_begin >= n) {
        if (it.phase == 2 && grp == 0)  // beyond the sequence: psi = 0
          for (int t = 0; t < kItemTiles; ++t) {
            const int key = key_begin + t * kTileKeys + et;
            if (key < p.n_max) psi[key] = 0.f;
          }
        continue;
      }
      const int k_item = active++;
      if ((k_item & 1) != grp) continue;
      const int ib = k_item % kItemBufs;
      const uint32_t use_par = (uint32_t)(k_item / kItemBufs) & 1u;
      const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + ib * kItemCols;
      uint64_t* tf = &tfull[ib * kItemTiles];
      uint64_t* te = &tempty[ib * kItemTiles];
      const int nt = min(kItemTiles, (n - key_begin + kTileKeys - 1) / kTileKeys);
      const int n_chunks_active = (n + kItemKeys - 1) / kItemKeys;
      // keys below this bound are seen by every window row
      const int all_bound = (n >= p.w) ? (p.causal ? n - p.w + 1 : n) : 0;
      auto wait_tile = [&](int t) -> bool {
        const bool w_ok = __all_sync(0xffffffffu, mbar_wait(&tf[t], use_par, abort_flag, p.status, kSiteTile));
        tc_fence_after();
        return w_ok;
      };
      auto release_tile = [&](int t) {  // this thread has read tile t's accumulator for the last time
        tc_fence_before();
        mbar_arrive(&te[t]);
      };

      __syncwarp();  // the warp's readers of shift_s / vis_s of the previous item are done
#pragma unroll
      for (int cb = 0; cb < NPAD; cb += 32) {
        const int row = cb + lane;
        // per-row visibility bound (exclusive key index) of this unit
        int vis = 0;
        if (row < p.R) {
          const int pos = n - p.w + row % p.w;
          if (pos >= 0) vis = p.causal ? pos + 1 : n;
        }
        vis_s[row] = vis;
        if (it.phase == 2) {
          // wait until the row's log-sum-exp is published (all phase-1 items of the unit are done)
          const int32_t* flag = p.done + (int64_t)it.unit * NPAD + row;
          const long long t0 = clock64();
          int spins = 0;
          while (true) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
            if (v >= kReady) break;
            if (*abort_flag) break;
            __nanosleep(64);
            if ((++spins & 255) == 0 && clock64() - t0 > p.flag_wait_cycles) {
              give_up(abort_flag, p.status, kSiteFlag);
              break;
            }
          }
          // negated for the exponent's fused multiply-add; padding rows get a huge shift (they add exp2(-huge) = 0)
          shift_s[row] = row < p.R ? -__ldcg(p.lse2 + (int64_t)it.unit * NPAD + row) : kEmptyMax;
        }
      }
      __syncwarp();
      ok = __all_sync(0xffffffffu, !*abort_flag);
      if (!ok) break;

      // An item is read tile by tile in blocks of 16 window rows (16 TMEM columns); the load of the next block is in
      // flight while the current one is processed. `body(j, r, t)` gets block j of tile t; `before_tile(t)` runs
      // before the first load of tile t.
      auto sweep = [&](auto before_tile, auto body) -> bool {
        uint32_t ra[16], rb[16];
        if (!before_tile(0)) return false;
        tmem_ld16_issue(tbase, ra);
        for (int t = 0; t < nt; ++t) {
#pragma unroll
          for (int j = 0; j < kBlocks; j += 2) {
            tmem_ld_wait16(ra);
            tmem_ld16_issue(tbase + t * NPAD + (j + 1) * 16, rb);
            body(std::integral_constant<int, 0>(), j, ra, t);
            tmem_ld_wait16(rb);
            if (j + 2 < kBlocks) {
              tmem_ld16_issue(tbase + t * NPAD + (j + 2) * 16, ra);
            } else if (t + 1 < nt) {
              if (!before_tile(t + 1)) return false;
              tmem_ld16_issue(tbase + (t + 1) * NPAD, ra);
            }
            body(std::integral_constant<int, 1>(), j + 1, rb, t);
          }
        }
        return true;
      };

      if (it.phase == 1) {
        // pass A: maximum of the raw logits per window row over this lane's keys
        float st_m[NPAD];
#pragma unroll
        for (int c = 0; c < NPAD; ++c) st_m[c] = kEmptyMax;
        ok = sweep([&](int t) { return wait_tile(t); },
                   [&](auto, int j, uint32_t (&r)[16], int t) {
                     const int key0 = key_begin + t * kTileKeys;
                     if (key0 + kTileKeys > all_bound) mask_block16(r, key0 + et, vis_s + j * 16);
#pragma unroll
                     for (int c = 0; c < 16; ++c) st_m[j * 16 + c] = fmaxf(st_m[j * 16 + c], __uint_as_float(r[c]));
                   });
        if (!ok) break;
        // pass B: sum of exp2 against the warp's maximum (second read of the accumulators, still in TMEM). The
        // (negated, scaled) maxima are uniform over the warp: they go to the warp's shift_s and are read back as
        // packed pairs, which keeps 32 registers free
        uint64_t z2[NPAD / 2];
#pragma unroll
        for (int c = 0; c < NPAD; ++c) {
          const float wm = warp_max(st_m[c]);
          if (lane == (c & 31)) shift_s[c] = -(wm * p.scale2);
        }
#pragma unroll
        for (int i = 0; i < NPAD / 2; ++i) z2[i] = 0ull;
        __syncwarp();
        sweep([&](int) { return true; },
              [&](auto, int j, uint32_t (&r)[16], int t) {
                const int key0 = key_begin + t * kTileKeys;
                if (j == kBlocks - 1) release_tile(t);  // all loads of the tile have completed
                if (key0 + kTileKeys > all_bound) mask_block16(r, key0 + et, vis_s + j * 16);
                exp_accumulate16(r, scale2x, shift2 + j * 8, z2 + j * 8);
              });
        for (int t = nt; t < kItemTiles; ++t) release_tile(t);  // unused slots: keep the barrier phases in step
        // Sum over the 32 lanes of the warp through a padded shared-memory transpose (fixed order): lane j ends up
        // with the sum of row cb + j, publishes the warp's partial of that row, counts it, and if that completes
        // the unit merges all partials of the row into its log-sum-exp.
#pragma unroll
        for (int cb = 0; cb < NPAD; cb += 32) {
          const int row = cb + lane;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float lo, hi;
            unpack2(z2[cb / 2 + c], lo, hi);
            tr[(2 * c) * 33 + lane] = lo;
            tr[(2 * c + 1) * 33 + lane] = hi;
          }
          __syncwarp();
          float zsum = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) zsum += tr[lane * 33 + i];
          float m2 = -shift_s[row];
          // a row of which the whole warp saw no visible key summed exp2(0) for its masked entries: it is empty
          if (m2 < 0.5f * kEmptyMax * p.scale2) {
            m2 = kEmptyMax;
            zsum = 0.f;
          }
          __syncwarp();
          float2* part = p.part + (int64_t)it.unit * p.cpu * (4 * NPAD) + row;
          __stcg(part + (int64_t)(it.chunk * 4 + quarter) * NPAD, make_float2(m2, zsum));
          int32_t* cnt = p.done + (int64_t)it.unit * NPAD + row;
          int old;
          asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(cnt) : "memory");
          if (old == 4 * n_chunks_active - 1) {
            float M = kEmptyMax, Z = 0.f;
            for (int e0 = 0; e0 < 4 * n_chunks_active; e0 += 8) {  // 4 * n_chunks_active is a multiple of 4
              float2 v[8];
#pragma unroll
              for (int j = 0; j < 8; ++j)
                v[j] = e0 + j < 4 * n_chunks_active ? __ldcg(part + (int64_t)(e0 + j) * NPAD)
                                                    : make_float2(kEmptyMax, 0.f);
#pragma unroll
              for (int j = 0; j < 8; ++j) merge_stats(M, Z, v[j].x, v[j].y);
            }
            const float lse2 = (Z > 0.f) ? M + log2f(Z) : 0.f;
            __stcg(p.lse2 + (int64_t)it.unit * NPAD + row, lse2);
            if (p.lse_out && row < p.R) {
              const int hq = h * p.g + row / p.w, wr = row % p.w;
              p.lse_out[((int64_t)bl * p.Hq + hq) * p.w + wr] = (Z > 0.f) ? lse2 * 0.6931471805599453f : -INFINITY;
            }
            if (!p.hold_flags)
              asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(cnt), "r"(kReady) : "memory");
          }
        }
      } else {
        uint64_t acc = 0ull;
        ok = sweep([&](int t) { return wait_tile(t); },
                   [&](auto, int j, uint32_t (&r)[16], int t) {
                     const int key = key_begin + t * kTileKeys + et;
                     if (j == kBlocks - 1) release_tile(t);  // all loads of the tile have completed
                     if (key - et + kTileKeys > all_bound) mask_block16(r, key, vis_s + j * 16);
                     acc = exp_sum16(r, scale2x, shift2 + j * 8, j == 0 ? 0ull : acc);
                     if (j == kBlocks - 1) {
                       float lo, hi;
                       unpack2(acc, lo, hi);
                       if (key < p.n_max) psi[key] = (key < n) ? lo + hi : 0.f;
                     }
                   });
        if (!ok) break;
        for (int t = nt; t < kItemTiles; ++t) {  // tiles beyond the sequence
          const int key = key_begin + t * kTileKeys + et;
          if (key < p.n_max) psi[key] = 0.f;
          release_tile(t);
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

// ------------------------------------------------------------------------------------------------ host side
template <int D, int NPAD>
int run_tc(const CUtensorMap& mk, const CUtensorMap& mq, const TcParams& p, int grid, cudaStream_t st) {
  using SL = SmemLayout<D, NPAD>;
  if (cudaFuncSetAttribute(score_tc_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kAlloc) !=
      cudaSuccess)
    return MADAKV_ECUDA;
  score_tc_kernel<D, NPAD><<<grid, kThreads, SL::kAlloc, st>>>(mk, mq, p);
  return launch_status();
}

}  // namespace

// A tensor-core path can run at all: a compute-capability-10 device, the tensor-map encoder of the driver, and no
// request for the generic path (MADAKV_SCORE_PATH=generic, tests).
bool tc_device_ok() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10)
    return false;
  const char* force = getenv("MADAKV_SCORE_PATH");
  if (force && force[0] == 'g') return false;
  return encode_fn() != nullptr;
}

bool score_tc_supported(const madakv_config& c, madakv_strides sq, madakv_strides sk) {
  const int g = c.n_q_heads / c.n_kv_heads;
  if (c.dtype != MADAKV_BF16 || g * c.window > 64 || c.window > 256 || g > 256) return false;
  (void)sq;
  (void)sk;
  return tc_device_ok();
}

int launch_score_tc(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                    const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st) {
  const WsLayout wl = ws_layout(c);
  const int g = c.n_q_heads / c.n_kv_heads;
  TcParams p;
  p.seq_len = seq_len;
  p.psi = psi;
  p.lse_out = lse;
  p.part = reinterpret_cast<float2*>((char*)ws + wl.score_part_off);
  p.done = reinterpret_cast<int32_t*>((char*)ws + wl.score_done_off);
  p.lse2 = reinterpret_cast<float*>((char*)ws + wl.score_lse_off);
  p.status = reinterpret_cast<int32_t*>(ws);
  p.units = c.batch * c.n_layers * c.n_kv_heads;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = g;
  p.w = c.window;
  p.R = g * c.window;
  p.n_max = c.max_seq_len;
  const int item_keys = kTileKeys * (kItemCols / (p.R <= 32 ? 32 : 64));
  p.cpu = (c.max_seq_len + item_keys - 1) / item_keys;
  p.causal = c.causal;
  p.scale2 = scale_of(c) * kLog2e;
  const int npad = p.R <= 32 ? 32 : 64;

  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MADAKV_ECUDA;
  const long long total = (long long)p.units * p.cpu;
  if (total > 0x3fffffff) return MADAKV_EUNSUPPORTED;
  const int grid = (int)(total < sms ? total : sms);
  // Phase 1 leads phase 2 by two work items per CTA: the K chunks in between (2 * grid items of 256 KB) stay within
  // the L2. A longer lead only spills the L2, and leads beyond two items per CTA are not used at all: in a run of
  // the whole pass with a lead of three and more items per CTA (and MMA warps that did not yet take every stage
  // barrier in order) the device reported a launch failure. The lead must cover a whole unit (all its phase-1 items come before its first phase-2 item);
  // sequences too long for that take the generic path. MADAKV_SCORE_LAG (tests) can shorten the lead.
  int lag = 2 * grid;
  if (const char* e = getenv("MADAKV_SCORE_LAG")) {
    const int v = atoi(e);
    if (v >= 1 && v < lag) lag = v;
  }
  if (lag < p.cpu) lag = p.cpu;
  if (lag > 2 * grid) return MADAKV_EUNSUPPORTED;
  p.lag = lag;
  // Failure-path test (no GPU fault involved): MADAKV_TEST_HOLD_FLAGS=1 withholds the row flags, so every phase-2 item
  // runs into its bounded wait, and MADAKV_TEST_WAIT_CYCLES shortens that wait from ~2 s to the given number of clock
  // cycles (at least 100 000). The kernel then records MADAKV_ETIMEOUT, drains and returns by itself.
  p.flag_wait_cycles = kWaitCycles;
  p.hold_flags = 0;
  if (const char* e = getenv("MADAKV_TEST_WAIT_CYCLES")) {
    const long long v = atoll(e);
    if (v >= 100000 && v < kWaitCycles) p.flag_wait_cycles = v;
  }
  if (const char* e = getenv("MADAKV_TEST_HOLD_FLAGS")) p.hold_flags = atoi(e) == 1;

  CUtensorMap mk, mq;
  if (!make_map(&mk, k, c.head_dim, c.max_seq_len, c.n_kv_heads, c.n_layers, c.batch, sk, kTileKeys, 1) ||
      !make_map(&mq, q, c.head_dim, c.window, c.n_q_heads, c.n_layers, c.batch, sq, c.window, g))
    return MADAKV_EUNSUPPORTED;
  if (cudaMemsetAsync(p.done, 0, (size_t)p.units * npad * sizeof(int32_t), st) != cudaSuccess) return MADAKV_ECUDA;
  if (c.head_dim == 128) return npad == 32 ? run_tc<128, 32>(mk, mq, p, grid, st) : run_tc<128, 64>(mk, mq, p, grid, st);
  return npad == 32 ? run_tc<64, 32>(mk, mq, p, grid, st) : run_tc<64, 64>(mk, mq, p, grid, st);
}

}  // namespace madakv
