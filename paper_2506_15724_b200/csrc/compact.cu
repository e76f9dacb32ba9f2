// Stage 4b: gather the kept K/V rows of every unit into the ragged per-head cache (bit copies).
//
// A row is d * elem_bytes = 128..512 bytes = LPR lanes of 16 bytes; a warp moves 32 / LPR rows of K and of V per
// instruction. Reads are whole 128-byte lines at random rows, writes are contiguous.
#include "common.cuh"

namespace madakv {
namespace {

constexpr int NT = 256;
constexpr int ROWS_PER_BLOCK = 128;
constexpr int kMaxBlocksX = 64;  // blocks per unit at most

struct CompactParams {
  const char* k;
  const char* v;
  char* k_c;
  char* v_c;
  const int32_t* kept_idx;
  const int64_t* seg_off;
  const int32_t* kept_len;
  const int32_t* seq_len;  // unused (bounds come from n_max); kept for symmetry
  int64_t capacity;
  int64_t stride_b, stride_l, stride_h, stride_t;  // bytes
  int L, Hkv, n_max, row_bytes, headroom;
};

template <int LPR>  // 16-byte lanes per row
__global__ void __launch_bounds__(NT) compact_kernel(CompactParams p) {
  const int u = blockIdx.y;
  const int len = p.kept_len[u];
  if ((int)blockIdx.x * ROWS_PER_BLOCK >= len) return;
  const int64_t off = p.seg_off[u];
  // a segment that selection refused (MADAKV_ECAPACITY: it would end beyond the cache) has no index list: skip it
  if (off + len + p.headroom > p.capacity) return;
  const int h = u % p.Hkv, l = (u / p.Hkv) % p.L, b = u / (p.Hkv * p.L);
  const int64_t src_base = b * p.stride_b + l * p.stride_l + h * p.stride_h;
  const int lane = threadIdx.x % LPR, sub = threadIdx.x / LPR;
  constexpr int RPI = NT / LPR;  // rows per block iteration
  // a block takes every gridDim.x-th stretch of ROWS_PER_BLOCK rows (the grid has at most kMaxBlocksX blocks per
  // unit: with one block per stretch of the longest possible segment nearly all blocks of a long-context call were
  // launched only to return)
  for (int row0 = blockIdx.x * ROWS_PER_BLOCK; row0 < len; row0 += gridDim.x * ROWS_PER_BLOCK) {
  const int row_end = min(len, row0 + ROWS_PER_BLOCK);
#pragma unroll 2
  for (int r = row0 + sub; r < row_end; r += RPI) {
    const int idx = p.kept_idx[off + r];
    if (idx < 0 || idx >= p.n_max) continue;
    const int64_t src = src_base + (int64_t)idx * p.stride_t + lane * 16;
    const int64_t dst = (off + r) * (int64_t)p.row_bytes + lane * 16;
    const uint4 kv = __ldg(reinterpret_cast<const uint4*>(p.k + src));
    const uint4 vv = __ldg(reinterpret_cast<const uint4*>(p.v + src));
    *reinterpret_cast<uint4*>(p.k_c + dst) = kv;
    *reinterpret_cast<uint4*>(p.v_c + dst) = vv;
  }
  }
}

}  // namespace

int launch_compact(const madakv_config& c, const void* k, const void* v, madakv_strides s, const int32_t* kept_idx,
                   const int64_t* seg_off, const int32_t* kept_len, void* k_c, void* v_c, int64_t capacity, void* ws,
                   cudaStream_t st) {
  (void)ws;
  const int e = elem_bytes(c);
  CompactParams p;
  p.k = (const char*)k;
  p.v = (const char*)v;
  p.k_c = (char*)k_c;
  p.v_c = (char*)v_c;
  p.kept_idx = kept_idx;
  p.seg_off = seg_off;
  p.kept_len = kept_len;
  p.seq_len = nullptr;
  p.capacity = capacity;
  p.stride_b = s.batch * e;
  p.stride_l = s.layer * e;
  p.stride_h = s.head * e;
  p.stride_t = s.token * e;
  p.L = c.n_layers;
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.row_bytes = c.head_dim * e;
  p.headroom = c.max_new_tokens;
  const int units = c.batch * c.n_layers * c.n_kv_heads;
  if (units > 65535) return MADAKV_EUNSUPPORTED;
  const int stretches = (c.max_seq_len + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK;
  const dim3 grid(stretches < kMaxBlocksX ? stretches : kMaxBlocksX, units);
  switch (p.row_bytes / 16) {
    case 8: compact_kernel<8><<<grid, NT, 0, st>>>(p); break;
    case 16: compact_kernel<16><<<grid, NT, 0, st>>>(p); break;
    case 32: compact_kernel<32><<<grid, NT, 0, st>>>(p); break;
    default: return MADAKV_EUNSUPPORTED;
  }
  return launch_status();
}

}  // namespace madakv
