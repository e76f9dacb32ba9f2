// Stage 1, TMEM-resident tensor-core path (Eq. 7 with the softmax of Eq. 5) for bf16 inputs with g * w <= 64 window
// rows and sequences short enough that all logits of one unit fit the tensor memory of a thread-block cluster.
//
// A softmax over keys needs every window row's log-sum-exp over ALL keys before any normalised weight can be summed
// over rows. Here the logits are not recomputed for that second step: a cluster of C CTAs (C SMs) takes one unit
// (sequence, layer, KV head) at a time, CTA r computes the window-QK^T tiles of its share of the keys with tcgen05.mma
// (128 keys of a tile on M, the g*w window rows on N, head_dim on K; operands by TMA, 128-byte swizzle) and KEEPS all
// its fp32 accumulators in TMEM (512 columns = 16 tiles of 32 rows or 8 tiles of 64 rows). The epilogue warps read
// them from TMEM as they arrive for the rows' (max, sum of exp2) statistics (one sweep against a per-lane reference
// logit for up to 32 rows, with an exact fallback; a maximum sweep and a sum sweep for 64), and once more when the (max, sum) pairs of all warps of the
// cluster have been exchanged through distributed shared memory and merged into the rows' log-sum-exps, for the
// weights exp2(s - lse) whose sum over rows is psi. So K is read from HBM exactly once and each tile takes one MMA pass.
//
// Warp roles per CTA: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-9 epilogue (two groups of four
// warps = the four TMEM lane quarters; group e takes the CTA's tiles of parity e; a thread owns one key of a tile and
// all window rows of it). The TMEM slots form a ring over the CTA's tiles of consecutive units and a tile's slot is
// handed back to the MMA warp after its last read: when a unit leaves slots free, the MMAs of the next unit run ahead
// into them during this unit's exchange and last sweep, and the TMA ring runs ahead with them.
// Synchronisation between CTAs exists only inside a cluster (whose CTAs are co-scheduled by the hardware): every lane
// of every epilogue warp sends its rows' pairs into each peer's shared memory with asynchronous stores that count
// their bytes on that peer's mbarrier.
// Every wait is bounded: on expiry the CTA records MADAKV_ETIMEOUT, drains and leaves through the final cluster barrier.
#include "tc_common.cuh"

namespace madakv {
namespace {

constexpr int kClThreads = 320;  // TMA warp, MMA warp, 8 epilogue warps
constexpr int kMaxCluster = 8;
enum { kSiteStats = 9 };

struct ClParams {
  const int32_t* seq_len;
  float* psi;       // [units, n_max]
  float* lse_out;   // natural log [B,L,Hq,w] or null
  int32_t* status;  // ws header
  int units, L, Hq, Hkv, g, w, R, n_max, causal, C;
  int per_max;  // most tiles a CTA gets of one unit (at most the number of TMEM slots)
  float scale2;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t num_clusters_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
  return r;
}
// shared::cluster address of `saddr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// Asynchronous store of a pair into a CTA of the cluster that, on landing, counts its 8 bytes on an mbarrier of that
// CTA: the receiver's wait on the barrier's transaction count orders the data, so the sender needs neither a fence
// nor an arrival of its own and goes straight on to its own wait.
__device__ __forceinline__ void st_async_f2(uint32_t raddr, float a, float b, uint32_t rbar) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(raddr),
               "f"(a), "f"(b), "r"(rbar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int D, int NPAD>
struct ClSmem {
  static constexpr int kStages = NPAD == 32 ? (D == 128 ? 5 : 10) : (D == 128 ? 3 : 6);  // 160 KB or 96 KB of K in flight
  static constexpr int kKBlocks = D / 64;
  static constexpr int kStageBytes = kTileKeys * D * 2;
  static constexpr int kQBytes = NPAD * D * 2;
  static constexpr int kSlots = kTmemCols / NPAD;  // accumulator tiles a CTA can hold: 16 or 8
  static constexpr int kKOff = 0;
  static constexpr int kQOff = kStages * kStageBytes;
  static constexpr int kBarOff = kQOff + 2 * kQBytes;
  // full[kStages], qfull[2], qempty[2], tfull[kSlots], tempty[kSlots], stats[2], drain[1]
  static constexpr int kNumBars = kStages + 4 + 2 * kSlots + 3;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  // misc: tmem base (4), abort flag (4), producer's stage ring (kStages <= 10 words)
  static constexpr int kWarpOff = kMiscOff + 48;
  // per epilogue warp: shift[NPAD], vis[NPAD]
  static constexpr int kWarpBytes = NPAD * 4 + NPAD * 4;
  static constexpr int kStatsOff = kWarpOff + 8 * kWarpBytes;
  // exchanged (max, sum) pairs: [2 unit parities][C CTAs][8 warps][NPAD rows]
  static constexpr int stats_bytes(int C) { return 2 * C * 8 * NPAD * 8; }
  static constexpr int alloc_bytes(int C) { return kStatsOff + stats_bytes(C) + 1024; }
};

template <int D, int NPAD>
__global__ void __launch_bounds__(kClThreads, 1)
score_cluster_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q, ClParams p) {
  using SL = ClSmem<D, NPAD>;
  constexpr int kStages = SL::kStages;
  constexpr int kKBlocks = SL::kKBlocks;
  constexpr int kSlots = SL::kSlots;
  constexpr int kBlocks = NPAD / 16;  // 16-row blocks per tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* k_s = smem + SL::kKOff;
  uint8_t* q_s = smem + SL::kQOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kBarOff);
  uint64_t* full = bars;                  // [kStages]  TMA -> MMA
  uint64_t* qfull = bars + kStages;       // [2]
  uint64_t* qempty = qfull + 2;           // [2]
  uint64_t* tfull = qempty + 2;           // [kSlots]   MMA -> epilogue and TMA
  uint64_t* tempty = tfull + kSlots;      // [kSlots]   epilogue -> MMA (128 arrivals: the four warps of the tile's group)
  uint64_t* stats_bar = tempty + kSlots;  // [2]        bytes sent by all epilogue lanes of the cluster -> this CTA's epilogue warps
  uint64_t* drain = stats_bar + 2;        // [1]        used only when the kernel gives up
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(smem + SL::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::kMiscOff + 4);
  float2* stats = reinterpret_cast<float2*>(smem + SL::kStatsOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = p.C;
  const int rank = (int)cluster_ctarank();
  const int cluster = (int)cluster_id_x(), n_clusters = (int)num_clusters_x();

  // ---- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&qfull[i], 1);
      mbar_init(&qempty[i], 1);
      mbar_init(&stats_bar[i], 1);  // one local arrival that announces the bytes of a unit's exchange
    }
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], 128);
    }
    mbar_init(&drain[0], 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows R..NPAD-1 of both Q buffers are never written by TMA: keep them zero so their logits are 0
  for (int x = threadIdx.x; x < 2 * SL::kQBytes / 16; x += kClThreads)
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
  cluster_sync_all();  // the peers' barriers are initialised before anyone arrives on them
  const uint32_t tmem_base = *tmem_base_s;

  // the tiles of unit u that belong to this CTA: [tile0, tile0 + my_tiles) of the unit's ceil(n / 128) tiles
  auto my_share = [&](int n, int& tile0, int& my_tiles) {
    const int tiles = (n + kTileKeys - 1) / kTileKeys;
    const int per = (tiles + C - 1) / C;
    tile0 = rank * per;
    my_tiles = max(0, min(per, tiles - tile0));
  };
  // TMEM slots are a ring over the CTA's tiles of consecutive units: every role keeps the same running position
  // (`ring`: slot of the current unit's first tile) and advances it by the unit's tile count.
  auto slot_at = [&](int ring, int jj) { return (ring + jj) & (kSlots - 1); };
  static_assert((kSlots & (kSlots - 1)) == 0, "slot ring uses a power-of-two mask");

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();  // K is read once
      const uint64_t pol_q = l2_policy_evict_last();
      // A K stage may be refilled once the MMAs of the tile that used it last have completed: that is the tile's
      // tfull barrier. stage_user remembers the slot, slot_par the parity of the slot's latest use by this thread
      // (a slot comes round every kSlots tiles, a stage every kStages < kSlots tiles, so the latest use of the slot
      // is the use that read the stage).
      volatile uint32_t* stage_user = reinterpret_cast<volatile uint32_t*>(smem + SL::kMiscOff + 8);
      for (int s2 = 0; s2 < kStages; ++s2) stage_user[s2] = 0;
      uint32_t slot_par = 0, slot_used = 0;
      int stage = 0, qi = 0, ring = 0;
      uint32_t q_par = 0;
      bool ok = true;
      for (int u = cluster; ok && u < p.units; u += n_clusters) {
        const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
        const int n = clamped_len(p.seq_len, b, p.n_max);
        int tile0, my_tiles;
        my_share(n, tile0, my_tiles);
        if (my_tiles == 0) continue;
        const int sb = ring;
        ring = slot_at(ring, my_tiles);
        ok = mbar_wait(&qempty[qi], q_par ^ 1, abort_flag, p.status, kSiteQEmpty);
        if (!ok) break;
        mbar_expect_tx(&qfull[qi], (uint32_t)(p.R * 128 * kKBlocks));
        for (int kb = 0; kb < kKBlocks; ++kb)
          tma_load_5d(q_s + qi * SL::kQBytes + kb * NPAD * 128, &tmap_q, &qfull[qi], kb * 64, 0, h * p.g, l, b, pol_q);
        qi ^= 1;
        if (qi == 0) q_par ^= 1;
        for (int jj = 0; jj < my_tiles; ++jj) {
          const int j = slot_at(sb, jj);
          const uint32_t prev = stage_user[stage];
          if (prev & 0x200u)
            ok = mbar_wait(&tfull[prev & 0xffu], (slot_par >> (prev & 0xffu)) & 1u, abort_flag, p.status, kSiteStage);
          if (!ok) break;
          // parity of this use of slot j: uses of a slot alternate 0, 1, 0, ...
          if (slot_used & (1u << j)) slot_par ^= 1u << j;
          slot_used |= 1u << j;
          stage_user[stage] = (uint32_t)j | 0x200u;
          mbar_expect_tx(&full[stage], (uint32_t)SL::kStageBytes);
          for (int kb = 0; kb < kKBlocks; ++kb)
            tma_load_5d(k_s + stage * SL::kStageBytes + kb * kTileKeys * 128, &tmap_k, &full[stage], kb * 64,
                        (tile0 + jj) * kTileKeys, h, l, b, pol);
          if (++stage == kStages) stage = 0;
        }
      }
      if (!ok) {  // abandoned: give copies in flight time to land before the CTA's shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(NPAD);
      const uint32_t k_lo0 = smem_desc_lo(smem_u32(k_s)), q_lo0 = smem_desc_lo(smem_u32(q_s));
      uint32_t slot_par = 0, slot_used = 0;  // parity of the current use of every slot
      int stage = 0, qi = 0, ring = 0;
      uint32_t stage_par = 0, q_par = 0;
      bool ok = true;
      for (int u = cluster; ok && u < p.units; u += n_clusters) {
        const int b = u / (p.Hkv * p.L);
        const int n = clamped_len(p.seq_len, b, p.n_max);
        int tile0, my_tiles;
        my_share(n, tile0, my_tiles);
        if (my_tiles == 0) continue;
        const int sb = ring;
        ring = slot_at(ring, my_tiles);
        ok = mbar_wait(&qfull[qi], q_par, abort_flag, p.status, kSiteQFull);
        if (!ok) break;
        const uint32_t q_lo = q_lo0 + (uint32_t)qi * (SL::kQBytes >> 4);
        for (int jj = 0; jj < my_tiles; ++jj) {
          const int j = slot_at(sb, jj);
          if (slot_used & (1u << j)) slot_par ^= 1u << j;
          slot_used |= 1u << j;
          const uint32_t use_par = (slot_par >> j) & 1u;
          // the slot's previous accumulator must have been read for the last time, and the K tile must have landed
          ok = mbar_wait(&tempty[j], use_par ^ 1, abort_flag, p.status, kSiteTEmpty) &&
               mbar_wait(&full[stage], stage_par, abort_flag, p.status, kSiteFull);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + (uint32_t)stage * (SL::kStageBytes >> 4);
          const uint32_t d_tmem = tmem_base + j * NPAD;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const int kb = ks >> 2, kk = ks & 3;
            umma_bf16(d_tmem, k_lo + ((kb * kTileKeys * 128 + kk * 32) >> 4), q_lo + ((kb * NPAD * 128 + kk * 32) >> 4),
                      idesc, ks > 0 ? 1u : 0u);
          }
          umma_commit(&tfull[j]);  // the accumulator is ready for the epilogue, and the K stage may be refilled
          if (++stage == kStages) {
            stage = 0;
            stage_par ^= 1;
          }
        }
        if (!ok) break;
        umma_commit(&qempty[qi]);  // the Q buffer may be refilled once this unit's MMAs are done
        qi ^= 1;
        if (qi == 0) q_par ^= 1;
      }
      if (!ok) {
        // abandoned: TMEM may only be freed once this thread's MMAs have completed
        umma_commit(&drain[0]);
        const long long t0 = clock64();
        while (!mbar_try(&drain[0], 0) && clock64() - t0 < 20000000ll) __nanosleep(200);
      }
    }
  } else {
    // ================================================================ epilogue
    const int ew = warp - 2;                 // 0..7
    const int grp = ew >> 2;                 // takes the CTA's tiles of this parity
    const int quarter = warp & 3;            // TMEM lanes [32 * quarter, 32 * quarter + 32)
    const int et = (quarter << 5) | lane;    // key index inside the tile
    uint8_t* wbase = smem + SL::kWarpOff + ew * SL::kWarpBytes;
    float* shift_s = reinterpret_cast<float*>(wbase);
    int* vis_s = reinterpret_cast<int*>(wbase + NPAD * 4);
    const uint64_t* shift2 = reinterpret_cast<const uint64_t*>(shift_s);
    const uint64_t scale2x = pack2(p.scale2, p.scale2);
    const uint32_t tlane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    uint32_t slot_par = 0, slot_used = 0;  // parity of the current use of every slot
    uint32_t unit_par = 0;                 // parity of the units this cluster has taken
    int ring = 0;
    // what depends on the sequence only is kept from unit to unit (the units of a sequence follow one another)
    int b = -1, b_end = 0, n = 0, tile0 = 0, my_tiles = 0, all_bound = 0, tiles_end = 0;
    bool ok = true;
    for (int u = cluster; ok && u < p.units; u += n_clusters, unit_par ^= 1) {
      if (u >= b_end) {
        b = u / (p.Hkv * p.L);
        b_end = (b + 1) * p.Hkv * p.L;
        n = clamped_len(p.seq_len, b, p.n_max);
        my_share(n, tile0, my_tiles);
        all_bound = (n >= p.w) ? (p.causal ? n - p.w + 1 : n) : 0;  // keys below are seen by every row
        tiles_end = ((n + kTileKeys - 1) / kTileKeys) * kTileKeys;
        __syncwarp();  // the warp's readers of vis_s for the previous sequence are done
#pragma unroll
        for (int cb = 0; cb < NPAD; cb += 32) {
          const int row = cb + lane;
          int vis = 0;  // per-row visibility bound (exclusive key index)
          if (row < p.R) {
            const int pos = n - p.w + row % p.w;
            if (pos >= 0) vis = p.causal ? pos + 1 : n;
          }
          vis_s[row] = vis;
        }
        __syncwarp();
      }
      float* psi = p.psi + (int64_t)u * p.n_max;
      const int cnt = my_tiles > grp ? (my_tiles - grp + 1) / 2 : 0;  // this group's tiles: grp, grp + 2, ...
      const int sb = ring;
      ring = slot_at(ring, my_tiles);
      if (rank == 0) {  // positions beyond the unit's last tile
        for (int key = tiles_end + ew * 32 + lane; key < p.n_max; key += 256) psi[key] = 0.f;
      }
      {  // parity of this use of the unit's slots (either group's: a slot serves tiles of both groups as the ring
         // moves on): the slots [sb, sb + my_tiles) of the ring as a bit mask
        const uint32_t run = my_tiles >= 32 ? 0xffffffffu : (1u << my_tiles) - 1u;
        const uint32_t all = kSlots >= 32 ? 0xffffffffu : (1u << kSlots) - 1u;
        const uint32_t used_now = ((run << sb) | (run >> ((kSlots - sb) & 31))) & all;
        slot_par ^= used_now & slot_used;
        slot_used |= used_now;
      }
      auto wait_tile = [&](int i) -> bool {
        const int j = slot_at(sb, grp + 2 * i);
        const bool w_ok =
            __all_sync(0xffffffffu, mbar_wait(&tfull[j], (slot_par >> j) & 1u, abort_flag, p.status, kSiteTile));
        tc_fence_after();
        return w_ok;
      };
      auto release_tile = [&](int i) {
        tc_fence_before();
        mbar_arrive(&tempty[slot_at(sb, grp + 2 * i)]);
      };
      // The group's tiles are read in blocks of 16 window rows (16 TMEM columns); the load of the next block is in
      // flight while the current one is processed. `body(j, r, i)` gets block j of the group's i-th tile.
      auto sweep = [&](auto before_tile, auto body) -> bool {
        if (cnt == 0) return true;
        uint32_t ra[16], rb[16];
        if (!before_tile(0)) return false;
        tmem_ld16_issue(tlane + slot_at(sb, grp) * NPAD, ra);
        for (int i = 0; i < cnt; ++i) {
          const uint32_t taddr = tlane + slot_at(sb, grp + 2 * i) * NPAD;
#pragma unroll
          for (int j = 0; j < kBlocks; j += 2) {
            tmem_ld_wait16(ra);
            tmem_ld16_issue(taddr + (j + 1) * 16, rb);
            body(j, ra, i);
            tmem_ld_wait16(rb);
            if (j + 2 < kBlocks) {
              tmem_ld16_issue(taddr + (j + 2) * 16, ra);
            } else if (i + 1 < cnt) {
              if (!before_tile(i + 1)) return false;
              tmem_ld16_issue(tlane + slot_at(sb, grp + 2 * i + 2) * NPAD, ra);
            }
            body(j + 1, rb, i);
          }
        }
        return true;
      };

      uint64_t z2[NPAD / 2];
      // Exact statistics in two sweeps: the warp's maximum per row, then the sum of exp2 against it. The (negated,
      // scaled) maxima are uniform over the warp: they go to the warp's shift_s and are read back as packed pairs.
      auto exact_stats = [&]() -> bool {
        float st_m[NPAD];
#pragma unroll
        for (int c = 0; c < NPAD; ++c) st_m[c] = kEmptyMax;
        const bool s_ok = sweep([&](int i) { return wait_tile(i); },
                                [&](int j, uint32_t (&r)[16], int i) {
                                  const int key0 = (tile0 + grp + 2 * i) * kTileKeys;
                                  if (key0 + kTileKeys > all_bound) mask_block16(r, key0 + et, vis_s + j * 16);
#pragma unroll
                                  for (int c = 0; c < 16; ++c)
                                    st_m[j * 16 + c] = fmaxf(st_m[j * 16 + c], __uint_as_float(r[c]));
                                });
        if (!s_ok) return false;
        __syncwarp();
#pragma unroll
        for (int c = 0; c < NPAD; ++c) {
          const float wm = warp_max(st_m[c]);
          if (lane == (c & 31)) shift_s[c] = -(wm * p.scale2);
        }
#pragma unroll
        for (int i = 0; i < NPAD / 2; ++i) z2[i] = 0ull;
        __syncwarp();
        sweep([&](int) { return true; },
              [&](int j, uint32_t (&r)[16], int i) {
                const int key0 = (tile0 + grp + 2 * i) * kTileKeys;
                if (key0 + kTileKeys > all_bound) mask_block16(r, key0 + et, vis_s + j * 16);
                exp_accumulate16(r, scale2x, shift2 + j * 8, z2 + j * 8);
              });
        return true;
      };
      if constexpr (NPAD == 32) {
        // One sweep as the tiles arrive: every lane takes, per window row, its logit of the group's first tile as the
        // reference and sums exp2(s - reference) over its keys (the reference's own term is 1). No maximum is needed
        // as long as no later logit lies ~100 binades above the reference; if a sum leaves that range (or a
        // reference was a masked logit), the warp redoes the unit's statistics exactly. Afterwards the lanes'
        // references are replaced by the warp's maximum of them.
        uint64_t negm2[NPAD / 2];
#pragma unroll
        for (int i = 0; i < NPAD / 2; ++i) {
          negm2[i] = pack2(-4.f * kEmptyMax, -4.f * kEmptyMax);  // no tile: reference below any masked logit
          z2[i] = 0ull;
        }
        ok = sweep([&](int i) { return wait_tile(i); },
                   [&](int j, uint32_t (&r)[16], int i) {
                     const int key0 = (tile0 + grp + 2 * i) * kTileKeys;
                     if (key0 + kTileKeys > all_bound) mask_block16(r, key0 + et, vis_s + j * 16);
                     if (i == 0) {
#pragma unroll
                       for (int c = 0; c < 8; ++c)
                         negm2[j * 8 + c] = pack2(-(__uint_as_float(r[2 * c]) * p.scale2),
                                                  -(__uint_as_float(r[2 * c + 1]) * p.scale2));
                     }
                     exp_accumulate16(r, scale2x, negm2 + j * 8, z2 + j * 8);
                   });
        if (!ok) break;
        float st_m[NPAD], st_z[NPAD];
        bool bad = false;
#pragma unroll
        for (int i = 0; i < NPAD / 2; ++i) {
          float a, b2;
          unpack2(negm2[i], a, b2);
          st_m[2 * i] = -a;
          st_m[2 * i + 1] = -b2;
          unpack2(z2[i], st_z[2 * i], st_z[2 * i + 1]);
          bad = bad || !(st_z[2 * i] < 1.0e30f) || !(st_z[2 * i + 1] < 1.0e30f);  // also catches inf and NaN
        }
        if (__any_sync(0xffffffffu, bad)) {
          ok = exact_stats();
          if (!ok) break;
        } else {
          __syncwarp();
#pragma unroll
          for (int c = 0; c < NPAD; ++c) {
            const float wm = warp_max(st_m[c]);
            st_z[c] *= ex2(st_m[c] - wm);
            if (lane == (c & 31)) shift_s[c] = -wm;
          }
#pragma unroll
          for (int i = 0; i < NPAD / 2; ++i) z2[i] = pack2(st_z[2 * i], st_z[2 * i + 1]);
          __syncwarp();
        }
      } else {
        ok = exact_stats();
        if (!ok) break;
      }
      // Sum over the 32 lanes by a transposing shuffle reduction (fixed order): lane j ends up with the sum of
      // row cb + j. It then stores the warp's (max, sum) of that row into every CTA of the cluster and arrives on
      // that CTA's barrier.
      float2* my_stats = stats + ((size_t)(unit_par * C + rank) * 8 + ew) * NPAD;
      float2 mine[NPAD / 32];
#pragma unroll
      for (int cb = 0; cb < NPAD; cb += 32) {
        float zv[32];
#pragma unroll
        for (int c = 0; c < 16; ++c) unpack2(z2[cb / 2 + c], zv[2 * c], zv[2 * c + 1]);
        float zsum = warp_rowsum32(zv);
        float m2 = -shift_s[cb + lane];
        // a row of which the whole warp saw no visible key summed exp2(0) for its masked entries: it is empty
        if (cnt == 0 || m2 < 0.5f * kEmptyMax * p.scale2) {
          m2 = kEmptyMax;
          zsum = 0.f;
        }
        mine[cb / 32] = make_float2(m2, zsum);
      }
      // this CTA's barrier of the unit expects one pair per epilogue lane, window-row block and CTA of the cluster
      if (ew == 0 && lane == 0) mbar_expect_tx(&stats_bar[unit_par], (uint32_t)(C * 8 * NPAD * sizeof(float2)));
      for (int peer = 0; peer < C; ++peer) {
        const uint32_t rbar = map_to_rank(smem_u32(&stats_bar[unit_par]), (uint32_t)peer);
#pragma unroll
        for (int cb = 0; cb < NPAD; cb += 32)
          st_async_f2(map_to_rank(smem_u32(my_stats + cb + lane), (uint32_t)peer), mine[cb / 32].x, mine[cb / 32].y,
                      rbar);
      }
      // wait for the pairs of every warp of the cluster (bounded)
      {
        // the barrier completes once per two units: its phase parity for this unit is the parity of (units taken / 2)
        const uint32_t par = (uint32_t)(((u - cluster) / n_clusters) >> 1) & 1u;
        bool got = mbar_try_cluster(&stats_bar[unit_par], par);
        if (!got) {
          const long long t0 = clock64();
          int spins = 0;
          while (!(got = mbar_try_cluster(&stats_bar[unit_par], par))) {
            if ((++spins & 63) == 0) {
              if (*abort_flag) break;
              if (clock64() - t0 > kWaitCycles) {
                give_up(abort_flag, p.status, kSiteStats);
                break;
              }
            }
          }
        }
        ok = __all_sync(0xffffffffu, got);
        if (!ok) break;
      }
      // every lane merges the pairs of its rows in a fixed order (CTA rank, then warp) into the row's log-sum-exp
#pragma unroll
      for (int cb = 0; cb < NPAD; cb += 32) {
        const int row = cb + lane;
        // maximum first, then the sums rescaled to it, eight independent terms at a time (fixed order)
        const float2* src = stats + (size_t)unit_par * C * 8 * NPAD + row;
        float M = kEmptyMax, Z = 0.f;
        for (int e0 = 0; e0 < C * 8; e0 += 8) {
#pragma unroll
          for (int j = 0; j < 8; ++j) M = fmaxf(M, src[(size_t)(e0 + j) * NPAD].x);
        }
        for (int e0 = 0; e0 < C * 8; e0 += 8) {
          float t[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float2 v = src[(size_t)(e0 + j) * NPAD];
            t[j] = v.y * ex2(v.x - M);  // an empty entry has sum 0
          }
          Z += ((t[0] + t[1]) + (t[2] + t[3])) + ((t[4] + t[5]) + (t[6] + t[7]));
        }
        const float lse2 = (Z > 0.f) ? M + log2f(Z) : 0.f;
        // negated for the exponent's fused multiply-add; padding rows get a huge shift (they add exp2(-huge) = 0)
        shift_s[row] = row < p.R ? -lse2 : kEmptyMax;
        if (p.lse_out && rank == 0 && ew == 0 && row < p.R) {
          const int h = u % p.Hkv, bl = u / p.Hkv;
          const int hq = h * p.g + row / p.w, wr = row % p.w;
          p.lse_out[((int64_t)bl * p.Hq + hq) * p.w + wr] = (Z > 0.f) ? lse2 * 0.6931471805599453f : -INFINITY;
        }
      }
      __syncwarp();
      // sweep 3: psi(i) = sum over window rows of exp2(s - lse); the slot goes back to the MMA warp
      uint64_t acc = 0ull;
      sweep([&](int) { return true; },
            [&](int j, uint32_t (&r)[16], int i) {
              const int key = (tile0 + grp + 2 * i) * kTileKeys + et;
              if (j == kBlocks - 1) release_tile(i);  // all loads of the tile have completed
              if (key - et + kTileKeys > all_bound) mask_block16(r, key, vis_s + j * 16);
              acc = exp_sum16(r, scale2x, shift2 + j * 8, j == 0 ? 0ull : acc);
              if (j == kBlocks - 1) {
                float lo, hi;
                unpack2(acc, lo, hi);
                if (key < p.n_max) psi[key] = (key < n) ? lo + hi : 0.f;
              }
            });
    }
  }

  // ---- teardown: no CTA of the cluster may leave while a peer can still write into its shared memory
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

template <int D, int NPAD>
int run_cluster(const CUtensorMap& mk, const CUtensorMap& mq, const ClParams& p, int sms, cudaStream_t st) {
  using SL = ClSmem<D, NPAD>;
  const int smem = SL::alloc_bytes(p.C);
  auto kern = score_cluster_kernel<D, NPAD>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      (p.C > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
    cudaGetLastError();
    return MADAKV_EUNSUPPORTED;
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // as many clusters as the device can hold at once (one CTA per SM), at most one per unit
  cfg.gridDim = dim3((unsigned)(sms / p.C * p.C));
  int max_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg) != cudaSuccess || max_clusters < 1) {
    cudaGetLastError();
    return MADAKV_EUNSUPPORTED;
  }
  const int clusters = min(min(max_clusters, sms / p.C), p.units);
  if (getenv("MADAKV_DEBUG"))
    fprintf(stderr, "madakv: score cluster kernel: cluster size %d, %d of at most %d clusters, %d B shared memory\n", p.C,
            clusters, max_clusters, smem);
  cfg.gridDim = dim3((unsigned)(clusters * p.C));
  if (cudaLaunchKernelEx(&cfg, kern, mk, mq, p) != cudaSuccess) {
    cudaGetLastError();
    return MADAKV_ECUDA;
  }
  return launch_status();
}

}  // namespace

// The cluster size for a shape, or 0 if the logits of the longest sequence do not fit the TMEM of kMaxCluster CTAs.
// Any size from 1 to 8 works (a unit's tiles are dealt out in equal shares, the last ranks get the remainder). The
// default is the smallest size whose per-CTA share fits; MADAKV_CLUSTER_SIZE forces another size that fits.
static int cluster_size_for(const madakv_config& c, int* per_max) {
  const int R = (c.n_q_heads / c.n_kv_heads) * c.window;
  const int npad = R <= 32 ? 32 : 64;
  const int slots = kTmemCols / npad;
  const int tiles = (c.max_seq_len + kTileKeys - 1) / kTileKeys;
  if (const char* e = getenv("MADAKV_CLUSTER_SIZE")) {
    const int C = atoi(e);
    if (C >= 1 && C <= kMaxCluster && (tiles + C - 1) / C <= slots) {
      *per_max = (tiles + C - 1) / C;
      return C;
    }
  }
  for (int C = 1; C <= kMaxCluster; ++C) {
    const int per = (tiles + C - 1) / C;
    if (per <= slots) {
      *per_max = per;
      return C;
    }
  }
  return 0;
}

int launch_score_cluster(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                         const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st) {
  const int g = c.n_q_heads / c.n_kv_heads;
  if (c.dtype != MADAKV_BF16 || g * c.window > 64) return MADAKV_EUNSUPPORTED;
  int per_max = 0;
  const int C = cluster_size_for(c, &per_max);
  if (C == 0) return MADAKV_EUNSUPPORTED;
  if (const char* e = getenv("MADAKV_SCORE_PATH"))
    if (e[0] == 't') return MADAKV_EUNSUPPORTED;  // tests: force the two-phase kernel
  ClParams p;
  p.seq_len = seq_len;
  p.psi = psi;
  p.lse_out = lse;
  p.status = reinterpret_cast<int32_t*>(ws);
  p.units = c.batch * c.n_layers * c.n_kv_heads;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = g;
  p.w = c.window;
  p.R = g * c.window;
  p.n_max = c.max_seq_len;
  p.causal = c.causal;
  p.C = C;
  p.per_max = per_max;
  p.scale2 = scale_of(c) * kLog2e;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MADAKV_ECUDA;
  CUtensorMap mk, mq;
  if (!make_map(&mk, k, c.head_dim, c.max_seq_len, c.n_kv_heads, c.n_layers, c.batch, sk, kTileKeys, 1) ||
      !make_map(&mq, q, c.head_dim, c.window, c.n_q_heads, c.n_layers, c.batch, sq, c.window, g))
    return MADAKV_EUNSUPPORTED;
  const int npad = p.R <= 32 ? 32 : 64;
  if (c.head_dim == 128)
    return npad == 32 ? run_cluster<128, 32>(mk, mq, p, sms, st) : run_cluster<128, 64>(mk, mq, p, sms, st);
  return npad == 32 ? run_cluster<64, 32>(mk, mq, p, sms, st) : run_cluster<64, 64>(mk, mq, p, sms, st);
}

}  // namespace madakv
