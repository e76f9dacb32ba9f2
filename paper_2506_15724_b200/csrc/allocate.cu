// Stages 2-3: modality masses and preference (Eq. 6, Eq. 8), sparsity counts (Eq. 9), layer compensation
// (Eq. 10-11) and the integer per-head, per-modality budgets.
//
// All sums of psi are exact: psi is mapped to 2^-32 fixed point (psi_fix) and added as 64-bit integers, so the
// results do not depend on the order of summation or on the launch shape. Eq. 9 is a "top-p" count: a 4-pass
// radix descent over the order-preserving bit pattern of psi with per-bucket (count, mass) histograms in shared
// memory finds the bucket in which the descending prefix mass reaches theta * W_m; ties inside the final bucket
// share one value, so the remaining count is a division. The layer recurrence is a scalar fp64 scan per sequence
// with explicitly rounded operations (no FMA contraction), so it is reproducible bit for bit.
#include "common.cuh"

namespace madakv {
namespace {

typedef unsigned long long u64;
typedef unsigned __int128 u128;
constexpr int NT = 512;

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
  int L, Hkv, n_max, mpa, hcc_mode;
  u64 theta_fix;  // floor(theta * 2^32)
};

__device__ __forceinline__ u64 block_sum_u64(u64 v, u64* scratch /*[NT/32]*/) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  u64 t = 0;
  for (int i = 0; i < NT / 32; ++i) t += scratch[i];
  return t;
}

__global__ void __launch_bounds__(NT) alloc_unit_kernel(AllocParams p) {
  __shared__ unsigned int cnt[2][256];
  __shared__ u64 msum[2][256];
  __shared__ u64 scratch[NT / 32];
  __shared__ uint32_t s_prefix[2];
  __shared__ u64 s_above_mass[2];
  __shared__ unsigned int s_above_cnt[2];
  __shared__ int s_done[2];

  const int u = blockIdx.x;
  const int b = u / (p.Hkv * p.L);
  const int n = min(p.seq_len[b], p.n_max);
  const float* psi = p.psi + (int64_t)u * p.n_max;
  const uint8_t* mask = p.mask + (int64_t)b * p.n_max;

  // Eq. 6: W_v, W_t
  u64 wv = 0, wt = 0;
  for (int i = threadIdx.x; i < n; i += NT) {
    const u64 f = psi_fix(psi_key(psi[i]));
    if (mask[i]) wv += f; else wt += f;
  }
  const u64 W[2] = {block_sum_u64(wv, scratch), block_sum_u64(wt, scratch)};
  const u128 need[2] = {(u128)p.theta_fix * W[0], (u128)p.theta_fix * W[1]};

  if (threadIdx.x < 2) {
    s_prefix[threadIdx.x] = 0;
    s_above_mass[threadIdx.x] = 0;
    s_above_cnt[threadIdx.x] = 0;
    s_done[threadIdx.x] = (need[threadIdx.x] == 0);
  }
  if (threadIdx.x == 0) {
    const u64 tot = W[0] + W[1];
    p.mass[(int64_t)u * 2 + 0] = __ull2double_rn(W[0]) / 4294967296.0;
    p.mass[(int64_t)u * 2 + 1] = __ull2double_rn(W[1]) / 4294967296.0;
    p.pref[(int64_t)u * 2 + 0] = tot ? __ddiv_rn(__ull2double_rn(W[0]), __ull2double_rn(tot)) : 0.0;
    p.pref[(int64_t)u * 2 + 1] = tot ? __ddiv_rn(__ull2double_rn(W[1]), __ull2double_rn(tot)) : 0.0;
  }
  __syncthreads();

  // Eq. 9: radix descent, both modalities at once
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int x = threadIdx.x; x < 512; x += NT) {
      (&cnt[0][0])[x] = 0;
      (&msum[0][0])[x] = 0;
    }
    __syncthreads();
    const uint32_t pre0 = s_prefix[0], pre1 = s_prefix[1];
    const bool act0 = !s_done[0], act1 = !s_done[1];
    for (int i = threadIdx.x; i < n; i += NT) {
      const uint32_t key = psi_key(psi[i]);
      const int m = mask[i] ? 0 : 1;
      if ((m == 0 ? act0 : act1) && (key & himask) == (m == 0 ? pre0 : pre1)) {
        const int dig = (key >> shift) & 255;
        atomicAdd(&cnt[m][dig], 1u);
        atomicAdd(&msum[m][dig], psi_fix(key));
      }
    }
    __syncthreads();
    if (threadIdx.x < 2 && !s_done[threadIdx.x]) {
      const int m = threadIdx.x;
      u64 above = s_above_mass[m];
      unsigned int above_c = s_above_cnt[m];
      int dig = 255;
      for (; dig > 0; --dig) {
        if (((u128)(above + msum[m][dig]) << 32) >= need[m]) break;
        above += msum[m][dig];
        above_c += cnt[m][dig];
      }
      s_above_mass[m] = above;
      s_above_cnt[m] = above_c;
      s_prefix[m] |= (uint32_t)dig << shift;
      if (pass == 3) {
        // every key in the final bucket has the same value: take as few of them as reach the threshold
        const u64 each = psi_fix(s_prefix[m]);
        unsigned int take = cnt[m][dig];
        if (each > 0) {
          const u128 rest = need[m] - ((u128)above << 32);
          const u128 per = (u128)each << 32;
          const u128 t = (rest + per - 1) / per;
          if (t < (u128)take) take = (unsigned int)t;
        }
        p.demand[(int64_t)u * 2 + m] = (int32_t)(above_c + take);
      }
    }
    __syncthreads();
  }
  if (threadIdx.x < 2 && need[threadIdx.x] == 0) p.demand[(int64_t)u * 2 + threadIdx.x] = 0;
}

// One block per sequence: Eq. 10-11 as a scalar scan over layers, then Eq. 8 integerised for every (layer, head).
__global__ void alloc_seq_kernel(AllocParams p) {
  extern __shared__ double s_Phi[];  // [L]
  __shared__ int s_nv;
  const int b = blockIdx.x;
  const int n = min(p.seq_len[b], p.n_max);
  if (threadIdx.x == 0) s_nv = 0;
  __syncthreads();
  int c = 0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) c += p.mask[(int64_t)b * p.n_max + i] ? 1 : 0;
  atomicAdd(&s_nv, c);
  __syncthreads();
  const int n_v = s_nv, n_t = n - n_v;
  if (threadIdx.x == 0) {
    const double lo = n >= 1 ? 1.0 : 0.0, hi = (double)n;
    double ph = (double)p.budget[b];
    for (int l = 1; l <= p.L; ++l) {
      p.phi[(int64_t)b * p.L + (l - 1)] = ph;
      s_Phi[l - 1] = fmin(fmax(floor(__dadd_rn(ph, 0.5)), lo), hi);
      if (l < p.L) {
        long long dem = 0;
        for (int h = 0; h < p.Hkv; ++h) {
          const int64_t u = ((int64_t)b * p.L + (l - 1)) * p.Hkv + h;
          dem += (long long)p.demand[u * 2] + p.demand[u * 2 + 1];
        }
        const double K = __dsub_rn((double)dem, __dmul_rn((double)p.Hkv, ph));  // Eq. 10
        double next = ph;
        if (p.hcc_mode == MADAKV_HCC_PAPER)
          next = __dsub_rn(ph, __ddiv_rn(K, (double)((long long)p.Hkv * (p.L - l))));  // Eq. 11, per-head units
        else if (p.hcc_mode == MADAKV_HCC_LITERAL)
          next = __dsub_rn(ph, __ddiv_rn(K, (double)(p.L - l)));  // Eq. 11 as printed
        ph = fmin(fmax(next, lo), hi);
      }
    }
  }
  __syncthreads();
  for (int x = threadIdx.x; x < p.L * p.Hkv; x += blockDim.x) {
    const int l = x / p.Hkv;
    const int64_t u = (int64_t)b * p.L * p.Hkv + x;
    const double Phi = s_Phi[l];
    const int P = (int)Phi;
    int bv, bt;
    if (p.mpa) {
      bv = (int)floor(__dadd_rn(__dmul_rn(p.pref[u * 2], Phi), 0.5));  // Eq. 8, rounded half up
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
  p.theta_fix = (u64)((double)c.theta * 4294967296.0);
  const int units = c.batch * c.n_layers * c.n_kv_heads;
  alloc_unit_kernel<<<units, NT, 0, st>>>(p);
  alloc_seq_kernel<<<c.batch, 256, c.n_layers * sizeof(double), st>>>(p);
  return launch_status();
}

}  // namespace madakv
