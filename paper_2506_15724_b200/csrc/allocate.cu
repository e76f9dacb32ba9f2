// Stages 2-3: modality masses and preference (Eq. 6, Eq. 8), sparsity counts (Eq. 9), layer compensation
// (Eq. 10-11) and the integer per-head, per-modality budgets.
//
// All sums of psi are exact: psi is mapped to 2^-32 fixed point (psi_fix) and added as 64-bit integers, so the
// results do not depend on the order of summation or on the launch shape. Eq. 9 is a "top-p" count: a three- or four-pass
// radix descent over the order-preserving bit pattern of psi with per-bucket (count, mass) histograms in shared
// memory finds the bucket in which the descending prefix mass reaches theta * W_m; ties inside the final bucket
// share one value, so the remaining count is a division. The keys of a unit sit in registers between passes. The layer recurrence is a scalar fp64 scan per sequence
// with explicitly rounded operations (no FMA contraction), so it is reproducible bit for bit.
#include "common.cuh"

namespace madakv {
namespace {

typedef unsigned long long u64;
constexpr int NT = 512;
constexpr int KPT = 16;            // keys a thread holds in registers per round
constexpr int ROUND = NT * KPT;    // keys a block takes per round
constexpr unsigned int kFull = 0xffffffffu;

struct AllocParams {
  const float* psi;
  const uint8_t* mask;
  const int32_t* seq_len;
  const int32_t* budget;
  double* mass;
  double* pref;
  int32_t* demand;
  double* phi;
  int32_t* budgets;
  int L, Hkv, n_max, mpa, hcc_mode, keep_window, window;
  u64 theta_fix;  // floor(theta * 2^32)
};

// Shared histograms of one radix pass: per (modality, digit) a count and an exact 64-bit mass kept as two 32-bit
// words (32-bit shared atomics are native; the carry of the low word is detected from the value the atomic returns).
// A digit has DIG bits. Sequences of more than one round are re-read from L2 in every pass, and with 10-bit digits the
// 30 bits in which importance values differ at most take three passes instead of four (long: allocation 0.26 -> 0.20
// ms); a sequence that sits in registers gains nothing from that and pays for the larger histograms (llava 0.067 ->
// 0.073 ms), so configs whose sequences fit one round keep 8-bit digits.
// Bucket b sits at word b + b / kPerLane: the bucket walk has lane j read buckets kPerLane * j + i, which in a dense
// array would be a many-way bank conflict on every load; with the skew the 32 lanes of a load hit 32 different banks.
template <int DIG>
struct Hist {
  static constexpr int kBuckets = 1 << DIG;        // per modality
  static constexpr int kPerLane = kBuckets / 32;   // buckets a lane of the walking warp owns
  static constexpr int kWords = 2 * kBuckets + 2 * 32;
  unsigned int cnt[kWords], mlo[kWords], mhi[kWords];
  __device__ __forceinline__ static int slot(int bucket) { return bucket + bucket / kPerLane; }
};
#define hist_slot(b) (Hist<DIG>::slot(b))
template <int DIG>
__device__ __forceinline__ void hist_add(Hist<DIG>& h, int bucket, u64 m) {
  const int s = hist_slot(bucket);
  atomicAdd(&h.cnt[s], 1u);
  const unsigned int add = (unsigned int)m;
  const unsigned int old = atomicAdd(&h.mlo[s], add);
  const unsigned int hi = (unsigned int)(m >> 32) + ((unsigned int)(old + add) < old ? 1u : 0u);
  if (hi) atomicAdd(&h.mhi[s], hi);  // rare: importance values are mostly below 1, carries are few
}
template <int DIG>
__device__ __forceinline__ u64 hist_mass(const Hist<DIG>& h, int bucket) {
  const int s = hist_slot(bucket);
  return ((u64)h.mhi[s] << 32) | h.mlo[s];
}

// One warp walks the buckets of modality m in ascending digit order (digits are taken from kmax - key, so this is
// descending importance): the first bucket at which the running mass `above + mass[dig]` reaches need_c is the one
// the threshold falls into (the last bucket if none does). Lane j owns buckets kPerLane * j ..; a warp prefix scan of
// the lanes' totals tells which lane holds that bucket, and that lane alone walks its buckets. Returns the bucket,
// and updates above / above_c to the mass / count strictly before it (identical in every lane).
template <int DIG>
__device__ __forceinline__ int descend(const Hist<DIG>& h, int m, u64 need_c, u64& above, unsigned int& above_c,
                                       unsigned int& cnt_at) {
  constexpr int kBuckets = Hist<DIG>::kBuckets, kPerLane = Hist<DIG>::kPerLane;
  const int lane = threadIdx.x & 31;
  const int first = m * kBuckets + lane * kPerLane;
  u64 lm = 0;
  unsigned int lc = 0;
#pragma unroll 8
  for (int i = 0; i < kPerLane; ++i) {
    lm += hist_mass(h, first + i);
    lc += h.cnt[hist_slot(first + i)];
  }
  u64 sm = lm;
  unsigned int sc = lc;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const u64 tm = __shfl_up_sync(kFull, sm, off);
    const unsigned int tc = __shfl_up_sync(kFull, sc, off);
    if (lane >= off) {
      sm += tm;
      sc += tc;
    }
  }
  // the lane whose buckets take the running mass to the threshold (lane 31 if none does)
  u64 a = above + (sm - lm);
  unsigned int ac = above_c + (sc - lc), c_at = 0;
  const unsigned int hit = __ballot_sync(kFull, a + lm >= need_c || lane == 31);
  const int win = __ffs(hit) - 1;
  int found = kPerLane - 1;
  if (lane == win) {
    for (int i = 0; i < kPerLane; ++i) {
      const u64 mi = hist_mass(h, first + i);
      const unsigned int ci = h.cnt[hist_slot(first + i)];
      if (a + mi >= need_c || i == kPerLane - 1) {
        found = i;
        c_at = ci;
        break;
      }
      a += mi;
      ac += ci;
    }
  }
  above = __shfl_sync(kFull, a, win);
  above_c = __shfl_sync(kFull, ac, win);
  cnt_at = __shfl_sync(kFull, c_at, win);
  return win * kPerLane + __shfl_sync(kFull, found, win);
}

// One block per unit. A thread keeps KPT keys in registers (loaded once when the sequence fits one round, else
// re-read from L2 every pass), so a pass costs no dependent global loads.
//
// The radix digits are not taken from the key itself but from t = kmax - key, starting at the highest bit in which
// the unit's keys differ (kmax, kmin: largest and smallest key of the unit). Importance values share their sign and
// most exponent bits, so digits of the raw key would put nearly all keys into a handful of buckets and serialise
// the shared atomics; the digits of t spread them over the whole histogram. Ascending t is descending importance.
template <int DIG>
__global__ void __launch_bounds__(NT, 2) alloc_unit_kernel(AllocParams p) {
  constexpr int kDigitBits = DIG, kBuckets = Hist<DIG>::kBuckets, kPerLane = Hist<DIG>::kPerLane;
  constexpr int kHistWords = Hist<DIG>::kWords;
  __shared__ Hist<DIG> hist;
  __shared__ uint32_t s_prefix[2];
  __shared__ int s_done[2];
  __shared__ u64 s_W[2];
  __shared__ uint32_t s_red[2][NT / 32];

  const int u = blockIdx.x;
  const int b = u / (p.Hkv * p.L);
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const float* psi = p.psi + (int64_t)u * p.n_max;
  const uint8_t* mask = p.mask + (int64_t)b * p.n_max;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rounds = (n + ROUND - 1) / ROUND;

  uint32_t key[KPT];
  uint32_t flags = 0;  // bit j: key j exists; bit 16 + j: key j is a visual token
  // a thread takes KPT consecutive keys of a round (which keys a thread holds does not matter: all sums are exact);
  // a full, aligned stretch comes in four 16-byte loads of scores and one of mask bytes
  const bool vec = (p.n_max & 3) == 0 && (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
  auto load_round = [&](int r) {
    flags = 0;
    const int i0 = r * ROUND + (int)threadIdx.x * KPT;
    if (vec && i0 + KPT <= n) {
#pragma unroll
      for (int j = 0; j < KPT; j += 4) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(psi + i0 + j));
        key[j] = psi_key(v.x);
        key[j + 1] = psi_key(v.y);
        key[j + 2] = psi_key(v.z);
        key[j + 3] = psi_key(v.w);
      }
      const uint4 mv = __ldg(reinterpret_cast<const uint4*>(mask + i0));
      flags = 0xffffu | ((nonzero_bytes(mv.x) | (nonzero_bytes(mv.y) << 4) | (nonzero_bytes(mv.z) << 8) |
                          (nonzero_bytes(mv.w) << 12)) << 16);
    } else {
#pragma unroll
      for (int j = 0; j < KPT; ++j) {
        const int i = i0 + j;
        key[j] = 0;
        if (i < n) {
          key[j] = psi_key(__ldg(psi + i));
          flags |= (1u << j) | (__ldg(mask + i) ? (0x10000u << j) : 0u);
        }
      }
    }
  };

  // range of the unit's keys
  uint32_t kmax = 0, kmin = 0xffffffffu;
  for (int r = 0; r < rounds; ++r) {
    load_round(r);
#pragma unroll
    for (int j = 0; j < KPT; ++j)
      if ((flags >> j) & 1u) {
        kmax = max(kmax, key[j]);
        kmin = min(kmin, key[j]);
      }
  }
  kmax = __reduce_max_sync(kFull, kmax);
  kmin = __reduce_min_sync(kFull, kmin);
  if (lane == 0) {
    s_red[0][warp] = kmax;
    s_red[1][warp] = kmin;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NT / 32; ++i) {
    kmax = max(kmax, s_red[0][i]);
    kmin = min(kmin, s_red[1][i]);
  }
  if (kmin > kmax) kmin = kmax;  // no keys at all
  // significant bits of t = kmax - key; at least one pass always runs (it also yields the masses of Eq. 6)
  const int top = max(32 - __clz(kmax - kmin), 1);
  if (rounds == 1) {
#pragma unroll
    for (int j = 0; j < KPT; ++j) key[j] = (flags >> j) & 1u ? kmax - key[j] : 0xffffffffu;  // (see the passes)
  }

  // state of the descent, kept by warp m (all lanes alike) for modality m
  u64 need_c = 0, above = 0;
  unsigned int above_c = 0;

  // Eq. 9: radix descent, both modalities at once. The first pass sees every key, so its histogram also yields the
  // modality masses W_v, W_t of Eq. 6. `rem` counts the bits of t not yet resolved.
  for (int rem = top, pass = 0; rem > 0; ++pass) {
    const int bits = min(rem, kDigitBits), shift = rem - bits;
    const uint32_t dmask = (1u << bits) - 1u;
    for (int x = threadIdx.x; x < kHistWords; x += NT) {
      hist.cnt[x] = 0;
      hist.mlo[x] = 0;
      hist.mhi[x] = 0;
    }
    __syncthreads();
    const uint32_t pre0 = pass ? s_prefix[0] : 0u, pre1 = pass ? s_prefix[1] : 0u;
    const bool act0 = pass == 0 || !s_done[0], act1 = pass == 0 || !s_done[1];
    if (act0 || act1) {
      for (int r = 0; r < rounds; ++r) {
        if (rounds > 1) {
          load_round(r);
#pragma unroll
          for (int j = 0; j < KPT; ++j) key[j] = (flags >> j) & 1u ? kmax - key[j] : 0xffffffffu;
        }
        // One comparison per key: t of an existing key is below 2^top <= 2^31, a slot without a key holds all ones,
        // and a modality that is done gets a prefix no shifted t can equal (rem >= 1).
        const uint32_t want0 = act0 ? pre0 : 0xffffffffu, want1 = act1 ? pre1 : 0xffffffffu;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
          const bool vis = (flags >> (16 + j)) & 1u;
          if ((key[j] >> rem) == (vis ? want0 : want1))
            hist_add(hist, (vis ? 0 : kBuckets) + (int)((key[j] >> shift) & dmask), psi_fix(kmax - key[j]));
        }
      }
    }
    __syncthreads();
    if (warp < 2) {
      const int m = warp;
      if (pass == 0) {
        u64 wsum = 0;
#pragma unroll 8
        for (int j = 0; j < kPerLane; ++j) wsum += hist_mass(hist, m * kBuckets + lane * kPerLane + j);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) wsum += __shfl_xor_sync(kFull, wsum, off);
        const u64 W = wsum;
        // need = theta_fix * W (96 bits); the prefix test  prefix * 2^32 >= need  is  prefix >= ceil(need / 2^32)
        const u64 hi = __umul64hi(p.theta_fix, W), lo = p.theta_fix * W;
        need_c = (hi << 32) + (lo >> 32) + ((lo & 0xffffffffull) ? 1ull : 0ull);
        if (lane == 0) {
          s_prefix[m] = 0;
          s_done[m] = (need_c == 0);
          s_W[m] = W;
          p.mass[(int64_t)u * 2 + m] = __ull2double_rn(W) / 4294967296.0;
          if (need_c == 0) p.demand[(int64_t)u * 2 + m] = 0;
        }
      }
      __syncwarp();
      if (need_c != 0) {
        unsigned int c_at = 0;
        const int dig = min(descend(hist, m, need_c, above, above_c, c_at), (int)dmask);
        if (lane == 0) {
          const uint32_t prefix = (s_prefix[m] << bits) | (uint32_t)dig;
          s_prefix[m] = prefix;
          if (shift == 0) {
            // t is resolved: every key in the final bucket has the value kmax - prefix; take as few of them as
            // reach the threshold
            const u64 each = psi_fix(kmax - prefix);
            unsigned int take = c_at;
            if (each > 0) {
              const u64 t = (need_c - above + each - 1) / each;
              if (t < (u64)take) take = (unsigned int)t;
            }
            p.demand[(int64_t)u * 2 + m] = (int32_t)(above_c + take);
          }
        }
      }
    }
    __syncthreads();
    if (pass == 0 && threadIdx.x == 0) {
      const u64 W0 = s_W[0], W1 = s_W[1], tot = W0 + W1;
      p.pref[(int64_t)u * 2 + 0] = tot ? __ddiv_rn(__ull2double_rn(W0), __ull2double_rn(tot)) : 0.0;
      p.pref[(int64_t)u * 2 + 1] = tot ? __ddiv_rn(__ull2double_rn(W1), __ull2double_rn(tot)) : 0.0;
    }
    rem = shift;
  }
}

// Visual tokens among the first n of a sequence, counted by the whole block into *s_nv (which the caller has zeroed
// behind a barrier); the caller synchronises before reading it.
__device__ __forceinline__ void count_visual(const uint8_t* mask, int n, int* s_nv) {
  int c = 0;
  if ((reinterpret_cast<uintptr_t>(mask) & 15) == 0) {  // 16 tokens per load
    const int n16 = n >> 4;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask) + i);
      const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int k = 0; k < 4; ++k)  // a byte counts if it is not zero
        c += __popc(((w4[k] | (w4[k] >> 1) | (w4[k] >> 2) | (w4[k] >> 3) | (w4[k] >> 4) | (w4[k] >> 5) | (w4[k] >> 6) |
                      (w4[k] >> 7)) & 0x01010101u));
    }
    for (int i = (n16 << 4) + threadIdx.x; i < n; i += blockDim.x) c += mask[i] ? 1 : 0;
  } else {
    for (int i = threadIdx.x; i < n; i += blockDim.x) c += mask[i] ? 1 : 0;
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(s_nv, c);
}
// Eq. 10's sum over the heads of one layer (both modalities), by one warp; every lane returns it.
__device__ __forceinline__ long long layer_demand(const int32_t* demand_layer, int Hkv) {
  long long dem = 0;
  for (int x = threadIdx.x & 31; x < 2 * Hkv; x += 32) dem += (long long)demand_layer[x];
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) dem += __shfl_xor_sync(0xffffffffu, dem, off);
  return dem;
}
// The layer's integer budget Phi^l from phi^l, and phi^{l+1} (Eq. 10-11); l counts from 1, the update exists for l < L.
__device__ __forceinline__ double rounded_budget(double ph, double lo, double hi) {
  return fmin(fmax(floor(__dadd_rn(ph, 0.5)), lo), hi);
}
__device__ __forceinline__ double next_phi(double ph, long long dem, int Hkv, int L, int l, int hcc_mode, double lo,
                                           double hi) {
  const double K = __dsub_rn((double)dem, __dmul_rn((double)Hkv, ph));  // Eq. 10
  double next = ph;
  if (hcc_mode == MADAKV_HCC_PAPER || hcc_mode == MADAKV_HCC_DEMAND)
    next = __dsub_rn(ph, __ddiv_rn(K, (double)((long long)Hkv * (L - l))));  // Eq. 11, per-head units
  else if (hcc_mode == MADAKV_HCC_LITERAL)
    next = __dsub_rn(ph, __ddiv_rn(K, (double)(L - l)));  // Eq. 11 as printed
  return fmin(fmax(next, lo), hi);
}
// Eq. 8 integerised for one head: the visual share rounded half up, the rest to text, surplus of a modality with too
// few tokens passed to the other. With `keep_demand` (mode DEMAND, every layer but the last) the head keeps what
// Eq. 9 asked for instead. lo_v, lo_t: the proxy tokens of each modality when they are retained unconditionally
// (cfg->keep_window), else 0: budgets are floored at them, the head's total at their sum.
__device__ __forceinline__ void split_budget(const AllocParams& p, int64_t u, double Phi, int n, int n_v, int n_t,
                                             int lo_v, int lo_t, bool keep_demand) {
  if (keep_demand) {
    const int dv = p.demand[u * 2], dt = p.demand[u * 2 + 1];
    p.budgets[u * 2] = p.mpa ? max(dv, lo_v) : 0;
    p.budgets[u * 2 + 1] = p.mpa ? max(dt, lo_t) : min(max(dv + dt, lo_v + lo_t), n);
    return;
  }
  const int P = max((int)Phi, lo_v + lo_t);
  int bv, bt;
  if (p.mpa) {
    bv = (int)floor(__dadd_rn(__dmul_rn(p.pref[u * 2], Phi), 0.5));  // Eq. 8, rounded half up
    bv = min(max(bv, lo_v), P - lo_t);
    bt = P - bv;
    if (bv > n_v) { bt += bv - n_v; bv = n_v; }
    if (bt > n_t) { bv = min(n_v, bv + (bt - n_t)); bt = n_t; }
  } else {
    bv = 0;
    bt = min(P, n);
  }
  p.budgets[u * 2] = bv;
  p.budgets[u * 2 + 1] = bt;
}

// One block per sequence: Eq. 10-11 as a scalar scan over layers, then Eq. 8 integerised for every (layer, head).
__global__ void alloc_seq_kernel(AllocParams p) {
  extern __shared__ double s_Phi[];  // [L] rounded budgets, then [L] demand sums (as long long)
  long long* s_dem = reinterpret_cast<long long*>(s_Phi + p.L);
  __shared__ int s_nv, s_wv;
  const int b = blockIdx.x;
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const int wlen = p.keep_window ? min(p.window, n) : 0;  // proxy tokens retained unconditionally
  if (threadIdx.x == 0) s_nv = s_wv = 0;
  __syncthreads();
  count_visual(p.mask + (int64_t)b * p.n_max, n, &s_nv);
  if (wlen > 0) count_visual(p.mask + (int64_t)b * p.n_max + (n - wlen), wlen, &s_wv);
  // Eq. 10's sum over heads, one warp per layer (integers: any order gives the same sum)
  for (int l = threadIdx.x >> 5; l < p.L; l += blockDim.x >> 5) {
    const long long dem = layer_demand(p.demand + ((int64_t)b * p.L + l) * p.Hkv * 2, p.Hkv);
    if ((threadIdx.x & 31) == 0) s_dem[l] = dem;
  }
  __syncthreads();
  const int n_v = s_nv, n_t = n - n_v;
  const int lo_v = p.mpa ? s_wv : 0, lo_t = wlen - lo_v;
  if (threadIdx.x == 0) {
    const double lo = n >= 1 ? 1.0 : 0.0, hi = (double)n;
    double ph = (double)p.budget[b];
    for (int l = 1; l <= p.L; ++l) {
      p.phi[(int64_t)b * p.L + (l - 1)] = ph;
      s_Phi[l - 1] = rounded_budget(ph, lo, hi);
      if (l < p.L) ph = next_phi(ph, s_dem[l - 1], p.Hkv, p.L, l, p.hcc_mode, lo, hi);
    }
  }
  __syncthreads();
  for (int x = threadIdx.x; x < p.L * p.Hkv; x += blockDim.x)
    split_budget(p, (int64_t)b * p.L * p.Hkv + x, s_Phi[x / p.Hkv], n, n_v, n_t, lo_v, lo_t,
                 p.hcc_mode == MADAKV_HCC_DEMAND && x / p.Hkv + 1 < p.L);
}

// One block per sequence, one layer of a layer-by-layer pass: the same arithmetic as one trip of the scan above. The
// per-layer arrays (pref, demand, budgets) hold this layer only; phi [B, depth] is the state carried between calls.
__global__ void alloc_layer_kernel(AllocParams p, int depth, int layer) {
  __shared__ int s_nv, s_wv;
  __shared__ double s_Phi;
  __shared__ long long s_dem;
  const int b = blockIdx.x;
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const int wlen = p.keep_window ? min(p.window, n) : 0;
  if (threadIdx.x == 0) s_nv = s_wv = 0;
  __syncthreads();
  count_visual(p.mask + (int64_t)b * p.n_max, n, &s_nv);
  if (wlen > 0) count_visual(p.mask + (int64_t)b * p.n_max + (n - wlen), wlen, &s_wv);
  if (threadIdx.x < 32) {
    const long long dem = layer_demand(p.demand + (int64_t)b * p.Hkv * 2, p.Hkv);
    if (threadIdx.x == 0) s_dem = dem;
  }
  __syncthreads();
  const int n_v = s_nv, n_t = n - n_v;
  const int lo_v = p.mpa ? s_wv : 0, lo_t = wlen - lo_v;
  if (threadIdx.x == 0) {
    const double lo = n >= 1 ? 1.0 : 0.0, hi = (double)n;
    const int l = layer + 1;  // the paper counts layers from 1
    double ph;
    if (layer == 0) {
      ph = (double)p.budget[b];
      p.phi[(int64_t)b * depth] = ph;
    } else {
      ph = p.phi[(int64_t)b * depth + layer];
    }
    s_Phi = rounded_budget(ph, lo, hi);
    if (l < depth) p.phi[(int64_t)b * depth + l] = next_phi(ph, s_dem, p.Hkv, depth, l, p.hcc_mode, lo, hi);
  }
  __syncthreads();
  for (int x = threadIdx.x; x < p.Hkv; x += blockDim.x)
    split_budget(p, (int64_t)b * p.Hkv + x, s_Phi, n, n_v, n_t, lo_v, lo_t,
                 p.hcc_mode == MADAKV_HCC_DEMAND && layer + 1 < depth);
}

// 8-bit digits while every sequence fits one round of the kernel, 10-bit digits beyond
void launch_alloc_unit(const madakv_config& c, const AllocParams& p, int units, cudaStream_t st) {
  if (c.max_seq_len <= ROUND) alloc_unit_kernel<8><<<units, NT, 0, st>>>(p);
  else alloc_unit_kernel<10><<<units, NT, 0, st>>>(p);
}

}  // namespace

int launch_allocate(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                    const int32_t* budget, double* mass, double* pref, int32_t* demand, double* phi, int32_t* budgets,
                    void* ws, cudaStream_t st) {
  (void)ws;
  AllocParams p;
  p.psi = psi;
  p.mask = mask;
  p.seq_len = seq_len;
  p.budget = budget;
  p.mass = mass;
  p.pref = pref;
  p.demand = demand;
  p.phi = phi;
  p.budgets = budgets;
  p.L = c.n_layers;
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.mpa = c.mpa;
  p.hcc_mode = c.hcc_mode;
  p.keep_window = c.keep_window;
  p.window = c.window;
  p.theta_fix = (u64)((double)c.theta * 4294967296.0);
  const int units = c.batch * c.n_layers * c.n_kv_heads;
  launch_alloc_unit(c, p, units, st);
  alloc_seq_kernel<<<c.batch, 1024, c.n_layers * (sizeof(double) + sizeof(long long)), st>>>(p);
  return launch_status();
}

int launch_allocate_layer(const madakv_config& c, int layer, const float* psi, const uint8_t* mask,
                          const int32_t* seq_len, const int32_t* budget, double* mass, double* pref, int32_t* demand,
                          double* phi, int32_t* budgets, void* ws, cudaStream_t st) {
  (void)ws;
  AllocParams p;
  p.psi = psi;
  p.mask = mask;
  p.seq_len = seq_len;
  p.budget = budget;
  p.mass = mass;
  p.pref = pref;
  p.demand = demand;
  p.phi = phi;
  p.budgets = budgets;
  p.L = 1;  // the per-layer arrays hold one layer
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.mpa = c.mpa;
  p.hcc_mode = c.hcc_mode;
  p.keep_window = c.keep_window;
  p.window = c.window;
  p.theta_fix = (u64)((double)c.theta * 4294967296.0);
  if (psi) launch_alloc_unit(c, p, c.batch * c.n_kv_heads, st);  // else: done by launch_demand_layer
  alloc_layer_kernel<<<c.batch, 1024, 0, st>>>(p, c.n_layers, layer);
  return launch_status();
}

int launch_demand_layer(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                        double* mass, double* pref, int32_t* demand, void* ws, cudaStream_t st) {
  (void)ws;
  AllocParams p;
  p.psi = psi;
  p.mask = mask;
  p.seq_len = seq_len;
  p.budget = nullptr;
  p.mass = mass;
  p.pref = pref;
  p.demand = demand;
  p.phi = nullptr;
  p.budgets = nullptr;
  p.L = 1;  // the per-layer arrays hold one layer
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.mpa = c.mpa;
  p.hcc_mode = c.hcc_mode;
  p.keep_window = c.keep_window;
  p.window = c.window;
  p.theta_fix = (u64)((double)c.theta * 4294967296.0);
  launch_alloc_unit(c, p, c.batch * c.n_kv_heads, st);
  return launch_status();
}

}  // namespace madakv
