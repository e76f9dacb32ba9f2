// Shared declarations of the MadaKV CUDA library (host-side validation helpers, workspace layout, small device helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "madakv.h"

namespace madakv {

// ---------------------------------------------------------------------------------------------------------------
// Workspace layout (device memory owned by the caller)
//   [0, 256)                 header: int32 status, then counters used by persistent kernels
//   [256, ..)                stage 4 scratch: visual-token count per sequence [B] int32, visual tokens among the
//                            proxy tokens per sequence [B] int32
//   [.., .. + score)         stage 1 scratch: finished-item counters [units * rows] int32, log2-domain row
//                            log-sum-exp [units * rows] fp32 (rows = g * w padded to a multiple of 32), per-chunk
//                            partial (max, sum) pairs (see ws_layout)
//   [.., .. + decode)        stage 5 scratch: split partials [B * L * H_q * splits * (d + 2)] fp32
// Stages 2-3 keep their scratch in shared memory.
// ---------------------------------------------------------------------------------------------------------------
constexpr size_t kHeaderBytes = 256;
constexpr int kScoreChunk = 1024;   // keys per (max, sum) partial of the generic scoring path
constexpr int kScoreTcChunk = 512;  // keys per work item (and per partial) of the tensor-core scoring path
constexpr int kDecodeChunk = 256;   // cache rows per split of decode attention

struct WsHeader {
  int32_t status;        // madakv_status set by device code
  int32_t wait_site;     // diagnostic: which bounded wait gave up (site | block << 8), written with MADAKV_ETIMEOUT
  int32_t reserved[62];
};
static_assert(sizeof(WsHeader) == kHeaderBytes, "header size");

struct WsLayout {
  size_t seq_nv_off, score_done_off, score_lse_off, score_part_off, decode_off, decode_len_off, total;
  int score_chunks, score_tc_chunks, decode_splits;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Wide-window scoring: its two passes run on at most kWideMaxGrid CTAs, each taking a contiguous, equally long range
// of the 128-key tiles of all units; pass 1 leaves one partial per (unit, CTA that holds tiles of it). A unit of t
// tiles meets at most ceil(t / floor(T / G)) + 1 of the G ranges (T tiles in all), and T >= L * Hkv * t, which
// gives the bound below whatever the lengths in the batch are.
constexpr int kWideMaxGrid = 160;
inline int wide_max_runs(const madakv_config& c) {
  const long long lh = (long long)c.n_layers * c.n_kv_heads;
  long long runs = (2ll * kWideMaxGrid + lh - 1) / lh + 1;
  const long long tiles = (c.max_seq_len + 127) / 128;
  if (runs > kWideMaxGrid) runs = kWideMaxGrid;
  if (runs > tiles) runs = tiles;
  return (int)(runs < 1 ? 1 : runs);
}

inline WsLayout ws_layout(const madakv_config& c) {
  WsLayout w;
  const size_t units = (size_t)c.batch * c.n_layers * c.n_kv_heads;
  const size_t rows = (size_t)(c.n_q_heads / c.n_kv_heads) * c.window;
  w.score_chunks = (c.max_seq_len + kScoreChunk - 1) / kScoreChunk;
  w.decode_splits = (c.max_seq_len + c.max_new_tokens + kDecodeChunk - 1) / kDecodeChunk;
  size_t off = kHeaderBytes;
  w.seq_nv_off = off;
  off = align_up(off + 2 * (size_t)c.batch * sizeof(int32_t), 256);  // per sequence: visual tokens, visual proxy tokens
  const size_t rows_pad = (rows + 31) / 32 * 32;  // the tensor-core path pads the row count
  w.score_done_off = off;
  off = align_up(off + units * rows_pad * sizeof(int32_t), 256);
  w.score_lse_off = off;
  off = align_up(off + units * rows_pad * sizeof(float), 256);
  w.score_part_off = off;
  w.score_tc_chunks = (c.max_seq_len + kScoreTcChunk - 1) / kScoreTcChunk;
  // partials: the generic path keeps one (max, sum) per (chunk, row); the tensor-core path (rows <= 64 only) one
  // per (work item, TMEM lane quarter, padded row)
  size_t part = units * (size_t)w.score_chunks * rows * sizeof(float2);
  if (rows <= 64) {
    const size_t tc = units * rows_pad * (size_t)w.score_tc_chunks * 4 * sizeof(float2);
    part = tc > part ? tc : part;
  } else if (rows <= 256) {  // wide-window path: per run of a unit and padded row one pair for each column share
    const size_t wide = units * (size_t)wide_max_runs(c) * (rows <= 128 ? 4 : 2) * rows_pad * sizeof(float2);
    part = wide > part ? wide : part;
  }
  off = align_up(off + part, 256);
  w.decode_off = off;
  off = align_up(off + (size_t)c.batch * c.n_layers * c.n_q_heads * (size_t)w.decode_splits * (c.head_dim + 2) *
                           sizeof(float), 256);
  w.decode_len_off = off;  // rows each segment's attention covered in an appending decode call
  off = align_up(off + units * sizeof(int32_t), 256);
  w.total = off;
  return w;
}

// Host-side checks shared by all entry points. Returns MADAKV_OK or the first violated rule.
inline int check_config(const madakv_config* c) {
  if (!c) return MADAKV_EINVAL;
  if (c->struct_size != sizeof(madakv_config)) return MADAKV_EINVAL;
  if (c->dtype != MADAKV_F32 && c->dtype != MADAKV_BF16) return MADAKV_EUNSUPPORTED;
  if (c->batch <= 0 || c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->max_seq_len <= 0 ||
      c->window <= 0)
    return MADAKV_ESHAPE;
  if (c->n_q_heads % c->n_kv_heads) return MADAKV_ESHAPE;
  if (c->head_dim != 64 && c->head_dim != 128) return MADAKV_EUNSUPPORTED;
  if (c->window > 1024 || (int64_t)(c->n_q_heads / c->n_kv_heads) * c->window > 4096) return MADAKV_EUNSUPPORTED;
  if (c->max_seq_len > (1 << 20)) return MADAKV_EUNSUPPORTED;
  if (c->causal != 0 && c->causal != 1) return MADAKV_EINVAL;
  if (c->mpa != 0 && c->mpa != 1) return MADAKV_EINVAL;
  if (c->hcc_mode < MADAKV_HCC_OFF || c->hcc_mode > MADAKV_HCC_DEMAND) return MADAKV_EINVAL;
  if (c->max_new_tokens < 0) return MADAKV_ESHAPE;
  if (!(c->theta >= 0.0f && c->theta <= 1.0f)) return MADAKV_EINVAL;
  if (!(c->softmax_scale >= 0.0f)) return MADAKV_EINVAL;
  if (c->keep_window != 0 && c->keep_window != 1) return MADAKV_EINVAL;
  if (c->pool_kernel < 1 || c->pool_kernel % 2 == 0) return MADAKV_EINVAL;
  if (c->pool_kernel > 15) return MADAKV_EUNSUPPORTED;
  return MADAKV_OK;
}

inline int elem_bytes(const madakv_config& c) { return c.dtype == MADAKV_F32 ? 4 : 2; }
inline bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }
inline bool strides_ok(const madakv_config& c, const madakv_strides& s) {
  const int64_t e = elem_bytes(c);
  return s.token >= c.head_dim && (s.batch * e) % 16 == 0 && (s.layer * e) % 16 == 0 && (s.head * e) % 16 == 0 &&
         (s.token * e) % 16 == 0 && s.batch >= 0 && s.layer >= 0 && s.head >= 0;
}
inline int check_ws(const madakv_config& c, const void* ws, size_t ws_bytes) {
  if (!ws) return MADAKV_EINVAL;
  if ((uintptr_t)ws & 255) return MADAKV_EALIGN;
  if (ws_bytes < ws_layout(c).total) return MADAKV_EWORKSPACE;
  return MADAKV_OK;
}
inline float scale_of(const madakv_config& c) {
  return c.softmax_scale > 0.0f ? c.softmax_scale : 1.0f / sqrtf((float)c.head_dim);
}
inline int launch_status() {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return MADAKV_OK;
  if (getenv("MADAKV_DEBUG")) fprintf(stderr, "madakv: CUDA error %d (%s)\n", (int)e, cudaGetErrorString(e));
  return MADAKV_ECUDA;
}

// Launch with programmatic stream serialisation: the grid may be scheduled while the kernel before it in the stream is
// still running, which hides its launch latency. A kernel launched this way calls pdl_wait() before it touches global
// memory (the call returns once the kernels before it have completed and their writes are visible; it is a no-op in a
// kernel launched the ordinary way) and pdl_go() to let the kernel after it be scheduled.
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  // a stream that is being captured gets the ordinary launch (full serialisation: the waits in the kernels are no-ops)
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) cap = cudaStreamCaptureStatusActive;
  if (cap == cudaStreamCaptureStatusNone) {
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---------------------------------------------------------------------------------------------------------------
// Device helpers
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_go() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
// ---------------------------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float ld_f32(const float* p) { return *p; }
__device__ __forceinline__ float ld_f32(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// Order-preserving integer image of a non-negative importance value; anything not > 0 (incl. NaN) maps to 0.
// Length of sequence b as the kernels use it: the caller's seq_len[b] brought into [0, n_max] (the header asks for
// that range; a value outside it must not turn into an index outside the arrays).
__device__ __forceinline__ int clamped_len(const int32_t* seq_len, int b, int n_max) {
  return max(0, min(seq_len[b], n_max));
}
__device__ __forceinline__ uint32_t psi_key(float x) { return x > 0.0f ? __float_as_uint(x) : 0u; }
// Bit i of the result: byte i of the word is not zero (four mask bytes at a time).
__device__ __forceinline__ uint32_t nonzero_bytes(uint32_t w) {
  const uint32_t x = ((((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) & 0x80808080u) >> 7;  // bits 0, 8, 16, 24
  return (x & 1u) | ((x >> 7) & 2u) | ((x >> 14) & 4u) | ((x >> 21) & 8u);
}
// floor(x * 2^32) of a key produced by psi_key.
__device__ __forceinline__ unsigned long long psi_fix(uint32_t key) {
  return key ? __float2ull_rz(__uint_as_float(key) * 4294967296.0f) : 0ull;
}

__device__ __forceinline__ void set_status(void* ws, int code) { atomicCAS((int*)ws, 0, code); }
#endif

// Stage launchers implemented in the .cu files (all return a madakv_status).
int launch_score(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                 const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st);
int launch_score_lse(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                     const int32_t* seq_len, const float* lse, float* psi, void* ws, cudaStream_t st);
int launch_score_lse_rows(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                          const int32_t* seq_len, const float* lse, float* psi, void* ws, cudaStream_t st);
bool tc_device_ok();
bool score_tc_supported(const madakv_config& c, madakv_strides sq, madakv_strides sk);
int launch_score_tc(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                    const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st);
int launch_score_cluster(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                         const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st);
int launch_score_rows(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                      const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st);
int launch_score_generic(const madakv_config& c, const void* q, madakv_strides sq, const void* k, madakv_strides sk,
                         const int32_t* seq_len, float* lse, float* psi, void* ws, cudaStream_t st);
int launch_allocate(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                    const int32_t* budget, double* mass, double* pref, int32_t* demand, double* phi, int32_t* budgets,
                    void* ws, cudaStream_t st);
int launch_allocate_layer(const madakv_config& c, int layer, const float* psi, const uint8_t* mask,
                          const int32_t* seq_len, const int32_t* budget, double* mass, double* pref, int32_t* demand,
                          double* phi, int32_t* budgets, void* ws, cudaStream_t st);
int launch_demand_layer(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                        double* mass, double* pref, int32_t* demand, void* ws, cudaStream_t st);
int launch_select(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                  const int32_t* budgets, int32_t* kept_len, int64_t* seg_off, int32_t* kept_idx, int64_t capacity,
                  void* ws, cudaStream_t st);
int launch_compact(const madakv_config& c, const void* k, const void* v, madakv_strides s, const int32_t* kept_idx,
                   const int64_t* seg_off, const int32_t* kept_len, void* k_c, void* v_c, int64_t capacity, void* ws,
                   cudaStream_t st);
int launch_decode(const madakv_config& c, int layer, const void* q, const void* k_new, const void* v_new, void* k_c,
                  void* v_c, const int64_t* seg_off, int32_t* kept_len, int64_t capacity, void* out, float* lse_out,
                  void* ws, cudaStream_t st);

}  // namespace madakv
