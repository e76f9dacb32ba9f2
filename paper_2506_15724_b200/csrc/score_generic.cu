// Stage 1, generic path (Eq. 7 with the softmax of Eq. 5): fp32 FMA arithmetic for any dtype, window and group
// size. It is the only path for fp32 inputs (TF32 tensor cores would not keep fp32 logits) and the fallback for
// shapes the tensor-core path does not take.
//
// Three kernels, all deterministic (fixed reduction order, no floating-point atomics):
//   stats   per (unit, chunk of kScoreChunk keys): running (max, sum exp2) of every window row over the chunk
//   reduce  per (unit, row): combine the chunk partials into the row's log2-domain log-sum-exp
//   psi     per (unit, 64-key tile): recompute the logits, psi(i) = sum_rows exp2(s2 - lse2_row)
// Logits are kept in the log2 domain: s2 = (q . k) * scale * log2(e).
#include "common.cuh"

namespace madakv {
namespace {

constexpr int KT = 64;        // keys per shared-memory tile
constexpr int RT = 32;        // window rows per shared-memory tile
constexpr int NT = 128;       // threads: 16 key lanes x 8 row groups; a thread owns keys kl+16j and rows 4rg+i
constexpr float kLog2e = 1.4426950408889634f;

struct ScoreParams {
  const void* q;
  const void* k;
  madakv_strides sq, sk;
  const int32_t* seq_len;
  float* lse_out;   // natural log, [B,L,Hq,w] or null
  float* psi;       // [units, n_max]
  float* lse2;      // ws: [units, R]
  float2* part;     // ws: [units, chunks, R]
  int L, Hq, Hkv, g, w, R, n_max, chunks, causal;
  float scale2;     // scale * log2(e)
};

template <typename T, int D>
__device__ __forceinline__ void load_k_tile(float* ks, const T* kbase, int64_t tok_stride, int key0, int n) {
  constexpr int LD = D + 4;
  for (int x = threadIdx.x; x < KT * (D / 4); x += NT) {
    const int kk = x / (D / 4), c4 = x % (D / 4);
    const int key = key0 + kk;
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (key < n) {
      const T* src = kbase + (int64_t)key * tok_stride + c4 * 4;
      if constexpr (sizeof(T) == 4) {
        val = *reinterpret_cast<const float4*>(src);
      } else {
        const uint2 raw = *reinterpret_cast<const uint2*>(src);
        val = make_float4(bf16_lo(raw.x), bf16_hi(raw.x), bf16_lo(raw.y), bf16_hi(raw.y));
      }
    }
    *reinterpret_cast<float4*>(ks + kk * LD + c4 * 4) = val;
  }
}

// Rows r0..r0+RT-1 of the unit's window-query matrix (row index = head_in_group * w + window_row).
template <typename T, int D>
__device__ __forceinline__ void load_q_tile(float* qs, const ScoreParams& p, int b, int l, int h, int r0) {
  constexpr int LD = D + 4;
  const T* q = reinterpret_cast<const T*>(p.q);
  for (int x = threadIdx.x; x < RT * (D / 4); x += NT) {
    const int rr = x / (D / 4), c4 = x % (D / 4);
    const int row = r0 + rr;
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row < p.R) {
      const int hq = h * p.g + row / p.w, wr = row % p.w;
      const T* src = q + b * p.sq.batch + l * p.sq.layer + hq * p.sq.head + wr * p.sq.token + c4 * 4;
      if constexpr (sizeof(T) == 4) {
        val = *reinterpret_cast<const float4*>(src);
      } else {
        const uint2 raw = *reinterpret_cast<const uint2*>(src);
        val = make_float4(bf16_lo(raw.x), bf16_hi(raw.x), bf16_lo(raw.y), bf16_hi(raw.y));
      }
    }
    *reinterpret_cast<float4*>(qs + rr * LD + c4 * 4) = val;
  }
}

// acc[j][i] = sum_c ks[key kl+16j][c] * qs[row 4rg+i][c]
template <int D>
__device__ __forceinline__ void tile_dots(const float* ks, const float* qs, int kl, int rg, float acc[4][4]) {
  constexpr int LD = D + 4;
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
#pragma unroll 4
  for (int c = 0; c < D; c += 4) {
    float4 kv[4], qv[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) kv[j] = *reinterpret_cast<const float4*>(ks + (kl + 16 * j) * LD + c);
#pragma unroll
    for (int i = 0; i < 4; ++i) qv[i] = *reinterpret_cast<const float4*>(qs + (rg * 4 + i) * LD + c);
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[j][i] = fmaf(kv[j].x, qv[i].x, acc[j][i]);
        acc[j][i] = fmaf(kv[j].y, qv[i].y, acc[j][i]);
        acc[j][i] = fmaf(kv[j].z, qv[i].z, acc[j][i]);
        acc[j][i] = fmaf(kv[j].w, qv[i].w, acc[j][i]);
      }
  }
}

// Last key a window row may see (exclusive bound), or 0 if the row does not exist.
__device__ __forceinline__ int row_visible(const ScoreParams& p, int row, int n) {
  if (row >= p.R) return 0;
  const int pos = n - p.w + row % p.w;
  if (pos < 0) return 0;
  return p.causal ? pos + 1 : n;
}

template <typename T, int D>
__global__ void __launch_bounds__(NT) score_stats_kernel(ScoreParams p) {
  extern __shared__ __align__(16) float smem[];
  float* ks = smem;
  float* qs = smem + KT * (D + 4);
  const int u = blockIdx.y, chunk = blockIdx.x;
  const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const int kl = threadIdx.x % 16, rg = threadIdx.x / 16;
  const int key_begin = chunk * kScoreChunk, key_end = min(n, key_begin + kScoreChunk);
  const T* kbase = reinterpret_cast<const T*>(p.k) + b * p.sk.batch + l * p.sk.layer + h * p.sk.head;
  float2* part = p.part + ((int64_t)u * p.chunks + chunk) * p.R;

  for (int r0 = 0; r0 < p.R; r0 += RT) {
    __syncthreads();
    load_q_tile<T, D>(qs, p, b, l, h, r0);
    float m[4], z[4];
    int vis[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      m[i] = -INFINITY;
      z[i] = 0.f;
      vis[i] = row_visible(p, r0 + rg * 4 + i, n);
    }
    for (int key0 = key_begin; key0 < key_end; key0 += KT) {
      __syncthreads();
      load_k_tile<T, D>(ks, kbase, p.sk.token, key0, n);
      __syncthreads();
      float acc[4][4];
      tile_dots<D>(ks, qs, kl, rg, acc);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int key = key0 + kl + 16 * j;
          if (key < vis[i]) {
            const float s2 = acc[j][i] * p.scale2;
            if (s2 > m[i]) {
              z[i] *= exp2f(m[i] - s2);  // exp2f(-inf) = 0 on the first key
              m[i] = s2;
            }
            z[i] += exp2f(s2 - m[i]);
          }
        }
    }
    // combine the 16 key lanes of each row (lanes of one row group sit in one half warp)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) {
        const float mo = __shfl_xor_sync(0xffffffffu, m[i], off);
        const float zo = __shfl_xor_sync(0xffffffffu, z[i], off);
        const float mn = fmaxf(m[i], mo);
        const float za = (m[i] == -INFINITY) ? 0.f : z[i] * exp2f(m[i] - mn);
        const float zb = (mo == -INFINITY) ? 0.f : zo * exp2f(mo - mn);
        m[i] = mn;
        z[i] = za + zb;
      }
      const int row = r0 + rg * 4 + i;
      if (kl == 0 && row < p.R) part[row] = make_float2(m[i], z[i]);
    }
  }
}

__global__ void score_reduce_kernel(ScoreParams p, int total_rows) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;  // (unit, row)
  if (x >= total_rows) return;
  const int u = x / p.R, row = x % p.R;
  const float2* part = p.part + (int64_t)u * p.chunks * p.R + row;
  float m = -INFINITY;
  for (int c = 0; c < p.chunks; ++c) m = fmaxf(m, part[(int64_t)c * p.R].x);
  float z = 0.f;
  for (int c = 0; c < p.chunks; ++c) {
    const float2 pz = part[(int64_t)c * p.R];
    if (pz.x != -INFINITY) z += pz.y * exp2f(pz.x - m);
  }
  const float lse2 = (m == -INFINITY) ? -INFINITY : m + log2f(z);
  p.lse2[x] = lse2;
  if (p.lse_out) {
    const int h = u % p.Hkv, bl = u / p.Hkv;
    const int hq = h * p.g + row / p.w, wr = row % p.w;
    p.lse_out[((int64_t)bl * p.Hq + hq) * p.w + wr] = lse2 * 0.6931471805599453f;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(NT) score_psi_kernel(ScoreParams p) {
  extern __shared__ __align__(16) float smem[];
  float* ks = smem;
  float* qs = smem + KT * (D + 4);
  __shared__ float red[8][KT];
  __shared__ float lse_s[RT];
  const int u = blockIdx.y, key0 = blockIdx.x * KT;
  const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
  const int n = clamped_len(p.seq_len, b, p.n_max);
  float* psi = p.psi + (int64_t)u * p.n_max;
  if (key0 >= n) {  // beyond the sequence: psi = 0
    for (int x = threadIdx.x; x < KT; x += NT)
      if (key0 + x < p.n_max) psi[key0 + x] = 0.f;
    return;
  }
  const int kl = threadIdx.x % 16, rg = threadIdx.x / 16;
  const T* kbase = reinterpret_cast<const T*>(p.k) + b * p.sk.batch + l * p.sk.layer + h * p.sk.head;
  load_k_tile<T, D>(ks, kbase, p.sk.token, key0, n);
  float sum[4] = {0.f, 0.f, 0.f, 0.f};
  for (int r0 = 0; r0 < p.R; r0 += RT) {
    __syncthreads();
    load_q_tile<T, D>(qs, p, b, l, h, r0);
    if (threadIdx.x < RT) lse_s[threadIdx.x] = (r0 + threadIdx.x < p.R) ? p.lse2[(int64_t)u * p.R + r0 + threadIdx.x] : 0.f;
    __syncthreads();
    float acc[4][4];
    tile_dots<D>(ks, qs, kl, rg, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int vis = row_visible(p, r0 + rg * 4 + i, n);
      const float lse2 = lse_s[rg * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (key0 + kl + 16 * j < vis) sum[j] += exp2f(acc[j][i] * p.scale2 - lse2);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) red[rg][kl + 16 * j] = sum[j];
  __syncthreads();
  if (threadIdx.x < KT) {
    float t = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) t += red[r][threadIdx.x];
    if (key0 + threadIdx.x < p.n_max) psi[key0 + threadIdx.x] = (key0 + threadIdx.x < n) ? t : 0.f;
  }
}

// caller-supplied natural-log sum-exps [B, L, H_q, w] -> log2-domain values in the (unit, row) order of the psi kernel
__global__ void score_given_lse_kernel(ScoreParams p, const float* lse, int total_rows) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= total_rows) return;
  const int u = x / p.R, row = x % p.R;
  const int h = u % p.Hkv, bl = u / p.Hkv;
  const int hq = h * p.g + row / p.w, wr = row % p.w;
  p.lse2[x] = lse[((int64_t)bl * p.Hq + hq) * p.w + wr] * 1.4426950408889634f;
}

template <typename T, int D>
int run_given_lse(const ScoreParams& p, const float* lse, int units, cudaStream_t st) {
  const size_t smem = (size_t)(KT + RT) * (D + 4) * sizeof(float);
  if (cudaFuncSetAttribute(score_psi_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return MADAKV_ECUDA;
  const int total_rows = units * p.R;
  score_given_lse_kernel<<<(total_rows + 255) / 256, 256, 0, st>>>(p, lse, total_rows);
  score_psi_kernel<T, D><<<dim3((p.n_max + KT - 1) / KT, units), NT, smem, st>>>(p);
  return launch_status();
}

template <typename T, int D>
int run(const ScoreParams& p, int units, cudaStream_t st) {
  const size_t smem = (size_t)(KT + RT) * (D + 4) * sizeof(float);
  if (cudaFuncSetAttribute(score_stats_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
          cudaSuccess ||
      cudaFuncSetAttribute(score_psi_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
          cudaSuccess)
    return MADAKV_ECUDA;
  score_stats_kernel<T, D><<<dim3(p.chunks, units), NT, smem, st>>>(p);
  const int total_rows = units * p.R;
  score_reduce_kernel<<<(total_rows + 255) / 256, 256, 0, st>>>(p, total_rows);
  score_psi_kernel<T, D><<<dim3((p.n_max + KT - 1) / KT, units), NT, smem, st>>>(p);
  return launch_status();
}

}  // namespace

static ScoreParams generic_params(const madakv_config& c, const void* q, madakv_strides sq, const void* k,
                                  madakv_strides sk, const int32_t* seq_len, float* lse, float* psi, void* ws) {
  const WsLayout wl = ws_layout(c);
  ScoreParams p;
  p.q = q;
  p.k = k;
  p.sq = sq;
  p.sk = sk;
  p.seq_len = seq_len;
  p.lse_out = lse;
  p.psi = psi;
  p.lse2 = reinterpret_cast<float*>((char*)ws + wl.score_lse_off);
  p.part = reinterpret_cast<float2*>((char*)ws + wl.score_part_off);
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = c.n_q_heads / c.n_kv_heads;
  p.w = c.window;
  p.R = p.g * p.w;
  p.n_max = c.max_seq_len;
  p.chunks = wl.score_chunks;
  p.causal = c.causal;
  p.scale2 = scale_of(c) * kLog2e;
  return p;
}

int launch_score_generic(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                         const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st) {
  const ScoreParams p = generic_params(c, q, sq, k, sk, seq_len, lse, psi, ws);
  const int units = c.batch * c.n_layers * c.n_kv_heads;
  if (units > 65535) return MADAKV_EUNSUPPORTED;
  if (c.dtype == MADAKV_F32) return c.head_dim == 64 ? run<float, 64>(p, units, st) : run<float, 128>(p, units, st);
  return c.head_dim == 64 ? run<__nv_bfloat16, 64>(p, units, st) : run<__nv_bfloat16, 128>(p, units, st);
}

// Single-pass scoring (Eq. 7) with the softmax normalisers supplied: tensor-core kernel for bf16 with g * w <= 256,
// the fp32 psi kernel otherwise.
int launch_score_lse(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                     const int32_t* seq_len, const float* lse, float* psi, void* ws, cudaStream_t st) {
  if (tc_device_ok()) {  // false also when MADAKV_SCORE_PATH asks for the fp32 kernels
    const int rc = launch_score_lse_rows(c, q, sq, k, sk, seq_len, lse, psi, ws, st);
    if (rc != MADAKV_EUNSUPPORTED) return rc;
  }
  const ScoreParams p = generic_params(c, q, sq, k, sk, seq_len, nullptr, psi, ws);
  const int units = c.batch * c.n_layers * c.n_kv_heads;
  if (units > 65535) return MADAKV_EUNSUPPORTED;
  if (c.dtype == MADAKV_F32)
    return c.head_dim == 64 ? run_given_lse<float, 64>(p, lse, units, st) : run_given_lse<float, 128>(p, lse, units, st);
  return c.head_dim == 64 ? run_given_lse<__nv_bfloat16, 64>(p, lse, units, st)
                          : run_given_lse<__nv_bfloat16, 128>(p, lse, units, st);
}

int launch_score(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                 const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st) {
  if (score_tc_supported(c, sq, sk)) {
    // tensor-core paths: logits resident in a cluster's TMEM when a unit fits, else the two-phase kernel; shapes
    // they decline go the generic way
    int rc = launch_score_cluster(c, q, sq, k, sk, seq_len, lse, psi, ws, st);
    if (rc != MADAKV_EUNSUPPORTED) return rc;
    rc = launch_score_tc(c, q, sq, k, sk, seq_len, lse, psi, ws, st);
    if (rc != MADAKV_EUNSUPPORTED) return rc;
  }
  if (tc_device_ok()) {
    // wide windows (64 < g * w <= 256): window rows on M, one row per epilogue thread
    const int rc = launch_score_rows(c, q, sq, k, sk, seq_len, lse, psi, ws, st);
    if (rc != MADAKV_EUNSUPPORTED) return rc;
  }
  return launch_score_generic(c, q, sq, k, sk, seq_len, lse, psi, ws, st);
}

}  // namespace madakv
