// Stage 5: cache append (Eq. 4) and decode attention over the ragged per-head cache (Eq. 5).
//
//   append   copies k_new / v_new behind every segment of the layer(s) and bumps kept_len
//   partial  one block per (segment, split of kDecodeChunk rows): a group of LPR lanes owns a cache row (16 bytes
//            per lane), the g query heads of the KV group share every K/V row read; online softmax in the log2
//            domain, fp32 accumulation; the block's row groups are merged in shared memory
//   merge    one block per query head: fixed-order combination of the split partials, rounding to dtype once
#include <mutex>

#include "common.cuh"

namespace madakv {
namespace {

constexpr int NT = 128;
constexpr int kDecodeGridX = 32;  // blocks per segment at most
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeParams {
  const void* q;
  const void* k_new;
  const void* v_new;
  void* k_c;
  void* v_c;
  const int64_t* seg_off;
  int32_t* kept_len;
  int64_t capacity;
  void* out;
  float* lse_out;
  float* part;  // ws: [B*L*Hq, splits, D + 2]
  void* ws;
  int L, Hq, Hkv, g, layer, splits;
  float scale2;
};

__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ int unit_of(const DecodeParams& p, int y) {
  // y enumerates the (sequence, KV head) pairs of the selected layer, or all units when layer < 0
  if (p.layer < 0) return y;
  const int b = y / p.Hkv, h = y % p.Hkv;
  return (b * p.L + p.layer) * p.Hkv + h;
}

template <int ROW_BYTES>
__global__ void append_kernel(DecodeParams p, int n_sel) {
  constexpr int LPR = ROW_BYTES / 16;
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  const int y = x / LPR, lane = x % LPR;
  if (y >= n_sel) return;
  const int u = unit_of(p, y);
  const int len = p.kept_len[u];
  const int64_t row = p.seg_off[u] + len;
  if (row + 1 > p.seg_off[u + 1] || row + 1 > p.capacity) {
    if (lane == 0) set_status(p.ws, MADAKV_ECAPACITY);
    return;
  }
  const uint4 kv = *reinterpret_cast<const uint4*>((const char*)p.k_new + (int64_t)u * ROW_BYTES + lane * 16);
  const uint4 vv = *reinterpret_cast<const uint4*>((const char*)p.v_new + (int64_t)u * ROW_BYTES + lane * 16);
  *reinterpret_cast<uint4*>((char*)p.k_c + row * ROW_BYTES + lane * 16) = kv;
  *reinterpret_cast<uint4*>((char*)p.v_c + row * ROW_BYTES + lane * 16) = vv;
  __syncwarp(__activemask());
  if (lane == 0) p.kept_len[u] = len + 1;
}

template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const void* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static void cvt(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const void* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
  }
  __device__ static void cvt(const uint4& v, float* f) {
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
  }
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(NT) decode_partial_kernel(DecodeParams p) {
  constexpr int EPL = Vec16<T>::N;          // elements per lane
  constexpr int LPR = D / EPL;              // lanes per row
  constexpr int GROUPS = NT / LPR;          // rows in flight per block
  constexpr int ROW_BYTES = D * (int)sizeof(T);
  __shared__ float s_o[GROUPS][G][D];
  __shared__ float s_m[GROUPS][G], s_l[GROUPS][G];

  const int u = unit_of(p, blockIdx.y);
  const int len = p.kept_len[u];
  // split 0 always reports, so an empty segment is well defined; a block beyond the segment has nothing to do
  if (blockIdx.x != 0 && (int)blockIdx.x * kDecodeChunk >= len) return;
  const int64_t off = p.seg_off[u];
  const int h = u % p.Hkv, bl = u / p.Hkv;
  const int lane = threadIdx.x % LPR, grp = threadIdx.x / LPR;

  float qr[G][EPL];
#pragma unroll
  for (int i = 0; i < G; ++i) {
    if (i < p.g) {
      const T* qp = reinterpret_cast<const T*>(p.q) + ((int64_t)bl * p.Hq + h * p.g + i) * D + lane * EPL;
      Vec16<T>::load(qp, qr[i]);
    } else {
#pragma unroll
      for (int c = 0; c < EPL; ++c) qr[i][c] = 0.f;
    }
  }
  // the grid has at most kDecodeGridX blocks per segment: a block takes splits blockIdx.x, blockIdx.x + gridDim.x, ...
  // (segments of an evicted cache are a few splits long, those of a full cache hundreds)
  for (int split = blockIdx.x; split == 0 || split * kDecodeChunk < len; split += gridDim.x) {
  const int row_begin = split * kDecodeChunk;
  const int row_end = min(len, row_begin + kDecodeChunk);
  float m[G], l[G], o[G][EPL];
#pragma unroll
  for (int i = 0; i < G; ++i) {
    m[i] = -INFINITY;
    l[i] = 0.f;
#pragma unroll
    for (int c = 0; c < EPL; ++c) o[i][c] = 0.f;
  }
  const char* kc = (const char*)p.k_c + off * ROW_BYTES + lane * 16;
  const char* vc = (const char*)p.v_c + off * ROW_BYTES + lane * 16;
  // U rows per thread are in flight at a time: all their 16-byte K and V loads are issued before the first use, so a
  // block keeps GROUPS * U * 2 * ROW_BYTES bytes on the wire (the online-softmax chain below is short next to the
  // memory latency). Uniform trip count: the shuffles need full warps.
  constexpr int U = G <= 2 ? 4 : 2;
  for (int r0 = row_begin; r0 < row_end; r0 += GROUPS * U) {
    uint4 kraw[U], vraw[U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int r = r0 + grp + GROUPS * j;
      kraw[j] = vraw[j] = make_uint4(0u, 0u, 0u, 0u);
      if (r < row_end) {
        kraw[j] = __ldcs(reinterpret_cast<const uint4*>(kc + (int64_t)r * ROW_BYTES));
        vraw[j] = __ldcs(reinterpret_cast<const uint4*>(vc + (int64_t)r * ROW_BYTES));
      }
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const bool valid = r0 + grp + GROUPS * j < row_end;
      float kf[EPL], vf[EPL];
      Vec16<T>::cvt(kraw[j], kf);
      Vec16<T>::cvt(vraw[j], vf);
      // all heads of the group at once (heads beyond g have zero queries): the dot products, then the lane
      // reductions of all heads interleaved, then the softmax updates, so that independent chains overlap
      float sc[G];
#pragma unroll
      for (int i = 0; i < G; ++i) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < EPL; ++c) s = fmaf(qr[i][c], kf[c], s);
        sc[i] = s;
      }
#pragma unroll
      for (int sh = LPR / 2; sh >= 1; sh >>= 1) {
#pragma unroll
        for (int i = 0; i < G; ++i) sc[i] += __shfl_xor_sync(0xffffffffu, sc[i], sh);
      }
      if (valid) {
#pragma unroll
        for (int i = 0; i < G; ++i) {
          const float s = sc[i] * p.scale2;
          if (s > m[i]) {
            const float f = fast_ex2(m[i] - s);  // exp2(-inf) = 0 on the first row
            l[i] *= f;
#pragma unroll
            for (int c = 0; c < EPL; ++c) o[i][c] *= f;
            m[i] = s;
          }
          const float pw = fast_ex2(s - m[i]);
          l[i] += pw;
#pragma unroll
          for (int c = 0; c < EPL; ++c) o[i][c] = fmaf(pw, vf[c], o[i][c]);
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < G; ++i) {
    if (lane == 0) {
      s_m[grp][i] = m[i];
      s_l[grp][i] = l[i];
    }
#pragma unroll
    for (int c = 0; c < EPL; ++c) s_o[grp][i][lane * EPL + c] = o[i][c];
  }
  __syncthreads();
  for (int x = threadIdx.x; x < p.g * D; x += NT) {
    const int i = x / D, c = x % D;
    float M = -INFINITY;
#pragma unroll
    for (int gq = 0; gq < GROUPS; ++gq) M = fmaxf(M, s_m[gq][i]);
    float Lsum = 0.f, O = 0.f;
#pragma unroll
    for (int gq = 0; gq < GROUPS; ++gq) {
      const float f = (s_m[gq][i] == -INFINITY) ? 0.f : exp2f(s_m[gq][i] - M);
      Lsum += s_l[gq][i] * f;
      O += s_o[gq][i][c] * f;
    }
    float* dst = p.part + (((int64_t)bl * p.Hq + h * p.g + i) * p.splits + split) * (D + 2);
    dst[c] = O;
    if (c == 0) {
      dst[D] = M;
      dst[D + 1] = Lsum;
    }
  }
  __syncthreads();  // the shared arrays are reused by the next split
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(D) decode_merge_kernel(DecodeParams p) {
  // blockIdx.x enumerates the query heads of the selected layer(s)
  int row;
  if (p.layer < 0) {
    row = blockIdx.x;
  } else {
    const int b = blockIdx.x / p.Hq, hq = blockIdx.x % p.Hq;
    row = (b * p.L + p.layer) * p.Hq + hq;
  }
  const int bl = row / p.Hq, hq = row % p.Hq;
  const int u = bl * p.Hkv + hq / p.g;
  const int len = p.kept_len[u];
  const int used = max(1, (len + kDecodeChunk - 1) / kDecodeChunk);
  const float* part = p.part + (int64_t)row * p.splits * (D + 2);
  const int c = threadIdx.x;
  float M = -INFINITY;
  for (int s = 0; s < used; ++s) M = fmaxf(M, part[s * (D + 2) + D]);
  float Lsum = 0.f, O = 0.f;
  for (int s = 0; s < used; ++s) {
    const float ms = part[s * (D + 2) + D];
    const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
    Lsum += part[s * (D + 2) + D + 1] * f;
    O += part[s * (D + 2) + c] * f;
  }
  const float res = Lsum > 0.f ? O / Lsum : 0.f;
  if constexpr (sizeof(T) == 4)
    reinterpret_cast<float*>(p.out)[(int64_t)row * D + c] = res;
  else
    reinterpret_cast<__nv_bfloat16*>(p.out)[(int64_t)row * D + c] = __float2bfloat16_rn(res);
  if (p.lse_out && c == 0) p.lse_out[row] = Lsum > 0.f ? (M + log2f(Lsum)) * kLn2 : -INFINITY;
}

template <typename T, int D>
int run(const DecodeParams& p, const madakv_config& c, cudaStream_t st) {
  const int n_sel = (p.layer < 0 ? c.batch * c.n_layers : c.batch) * c.n_kv_heads;
  if (p.k_new) {
    constexpr int LPR = D * (int)sizeof(T) / 16;
    append_kernel<D * (int)sizeof(T)><<<(n_sel * LPR + 127) / 128, 128, 0, st>>>(p, n_sel);
  }
  if (n_sel > 65535) return MADAKV_EUNSUPPORTED;
  const dim3 grid(p.splits < kDecodeGridX ? p.splits : kDecodeGridX, n_sel);
  if (p.g == 1) decode_partial_kernel<T, D, 1><<<grid, NT, 0, st>>>(p);
  else if (p.g == 2) decode_partial_kernel<T, D, 2><<<grid, NT, 0, st>>>(p);
  else if (p.g <= 4) decode_partial_kernel<T, D, 4><<<grid, NT, 0, st>>>(p);
  else if (p.g <= 8) decode_partial_kernel<T, D, 8><<<grid, NT, 0, st>>>(p);
  else return MADAKV_EUNSUPPORTED;
  decode_merge_kernel<T, D><<<n_sel * p.g, D, 0, st>>>(p);
  return launch_status();
}

}  // namespace

int launch_decode(const madakv_config& c, int layer, const void* q, const void* k_new, const void* v_new, void* k_c,
                  void* v_c, const int64_t* seg_off, int32_t* kept_len, int64_t capacity, void* out, float* lse_out,
                  void* ws, cudaStream_t st) {
  const WsLayout wl = ws_layout(c);
  DecodeParams p;
  p.q = q;
  p.k_new = k_new;
  p.v_new = v_new;
  p.k_c = k_c;
  p.v_c = v_c;
  p.seg_off = seg_off;
  p.kept_len = kept_len;
  p.capacity = capacity;
  p.out = out;
  p.lse_out = lse_out;
  p.part = reinterpret_cast<float*>((char*)ws + wl.decode_off);
  p.ws = ws;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = c.n_q_heads / c.n_kv_heads;
  p.layer = layer;
  p.splits = wl.decode_splits;
  p.scale2 = scale_of(c) * kLog2e;
  if (c.dtype == MADAKV_F32) return c.head_dim == 64 ? run<float, 64>(p, c, st) : run<float, 128>(p, c, st);
  return c.head_dim == 64 ? run<__nv_bfloat16, 64>(p, c, st) : run<__nv_bfloat16, 128>(p, c, st);
}

}  // namespace madakv

// ---------------------------------------------------------------------------------------------------------------
// madakv_decode_attn_static: the same attention kernels with their split partials in a fixed array of the library
// image, for callers that have no way to provide (or allocate) a workspace.
// ---------------------------------------------------------------------------------------------------------------

// Split partials of the no-allocation entry point. One copy per GPU that loads the library, shared by all calls.
static __device__ __align__(256) unsigned char g_static_scratch[MADAKV_STATIC_SCRATCH_BYTES];

namespace madakv {
namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};  // device address of g_static_scratch on each device, once looked up

// In host code the name g_static_scratch is only a handle; the address kernels can use comes from the runtime,
// per device, with that device current.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MADAKV_ECUDA;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return MADAKV_ECUDA;
    }
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return MADAKV_OK;
}

}  // namespace
}  // namespace madakv

extern "C" int madakv_decode_attn_static(const madakv_config* cfg, int32_t layer, const void* q, const void* k_c,
                                         const void* v_c, const int64_t* seg_off, const int32_t* kept_len,
                                         int64_t capacity, void* out, float* lse_out, void* stream) {
  using namespace madakv;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!q || !k_c || !v_c || !seg_off || !kept_len || !out) return MADAKV_EINVAL;
  if (layer < -1 || layer >= cfg->n_layers) return MADAKV_ESHAPE;
  if (capacity <= 0) return MADAKV_ECAPACITY;
  if (!aligned16(q) || !aligned16(k_c) || !aligned16(v_c) || !aligned16(out) || ((uintptr_t)seg_off & 7) ||
      ((uintptr_t)kept_len & 3) || ((uintptr_t)lse_out & 3))
    return MADAKV_EALIGN;
  const madakv_config& c = *cfg;
  const int splits = ws_layout(c).decode_splits;
  const size_t need = (size_t)c.batch * c.n_layers * c.n_q_heads * (size_t)splits * (c.head_dim + 2) * sizeof(float);
  if (need > (size_t)MADAKV_STATIC_SCRATCH_BYTES) return MADAKV_ESTATIC;
  void* scratch = nullptr;
  if ((rc = static_scratch(&scratch))) return rc;

  DecodeParams p;
  p.q = q;
  p.k_new = nullptr;  // no append: the caches and kept_len are only read
  p.v_new = nullptr;
  p.k_c = const_cast<void*>(k_c);
  p.v_c = const_cast<void*>(v_c);
  p.seg_off = seg_off;
  p.kept_len = const_cast<int32_t*>(kept_len);
  p.capacity = capacity;
  p.out = out;
  p.lse_out = lse_out;
  p.part = reinterpret_cast<float*>(scratch);
  p.ws = nullptr;  // only the append kernel reports through the workspace
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = c.n_q_heads / c.n_kv_heads;
  p.layer = layer;
  p.splits = splits;
  p.scale2 = scale_of(c) * kLog2e;
  cudaStream_t st = (cudaStream_t)stream;
  if (c.dtype == MADAKV_F32) return c.head_dim == 64 ? run<float, 64>(p, c, st) : run<float, 128>(p, c, st);
  return c.head_dim == 64 ? run<__nv_bfloat16, 64>(p, c, st) : run<__nv_bfloat16, 128>(p, c, st);
}
