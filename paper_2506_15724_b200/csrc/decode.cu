// Stage 5: cache append (Eq. 4) and decode attention over the ragged per-head cache (Eq. 5).
//
//   append   (Eq. 4) has no kernel of its own: the partial block whose share holds the new row copies it from
//            k_new / v_new behind the segment and attends over it; the merge kernel bumps kept_len
//   partial  up to 8, 16 or 32 blocks per segment (blocks_per_segment), each taking an equal share of the segment's rows (the share is a
//            function of the segment's length alone: short segments use fewer blocks, never fewer than kDecodeMinRows
//            rows each): a group of LPR lanes owns a cache row (16 bytes per lane), the g query heads of the KV group
//            share every K/V row read; online softmax in the log2 domain, fp32 accumulation; the block's row groups
//            are merged in shared memory. For bf16 caches with 3 <= g <= 16 the same share is computed by
//            decode_partial_mma_kernel on the tensor cores instead.
//   merge    one block per query head: fixed-order combination of the blocks' partials, rounding to dtype once
#include <mutex>

#include "common.cuh"

namespace madakv {
namespace {

constexpr int NT = 128;
constexpr int kDecodeSlots = 32;    // blocks (and partials) per segment at most
constexpr int kDecodeMinRows = 512; // a block's share of a segment is at least this many rows: shorter shares leave
                                    // the block's load pipeline no time to fill (measured: 256 rows cost 5-8 %)
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
  float* part;  // ws: [B*L*Hq, slots, D + 2]
  int32_t* eff_len;  // ws: [units] rows each segment's attention covered (appending calls; else null)
  void* ws;
  int L, Hq, Hkv, g, layer, slots, n_sel, min_rows, slot_fast;
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

// Rows of unit u's segment that attention may read. A segment that selection refused (it, with its headroom, ends
// beyond the cache: MADAKV_ECAPACITY was reported and neither indices nor rows were written) counts as empty, and so
// does one whose length does not fit its own slot: nothing beyond `capacity` rows is ever touched.
__device__ __forceinline__ bool segment_refused(const DecodeParams& p, int u) {
  const int64_t off = p.seg_off[u], end = p.seg_off[u + 1];
  return off < 0 || end < off || end > p.capacity;
}
__device__ __forceinline__ int segment_rows(const DecodeParams& p, int u) {
  const int len = p.kept_len[u];
  if (segment_refused(p, u) || len < 0 || p.seg_off[u] + (int64_t)len > p.seg_off[u + 1]) return 0;
  return len;
}
// The blocks of a segment of `len` rows: how many take part, and the rows of block x (a multiple of 16 each, so
// that the 16-row chunks of the warps never straddle two blocks). Block 0 always takes part: an empty segment still
// gets a well-defined partial.
__device__ __forceinline__ int segment_blocks(const DecodeParams& p, int len) {
  return max(1, min(p.slots, (len + p.min_rows - 1) / p.min_rows));
}
__device__ __forceinline__ void block_rows(const DecodeParams& p, int len, int x, int& row_begin, int& row_end) {
  const int nb = segment_blocks(p, len);
  const int share = ((len + nb - 1) / nb + 15) / 16 * 16;
  row_begin = min(len, x * share);
  row_end = min(len, row_begin + share);
}

// What a block of unit u works on. When the call appends (Eq. 4), the new row is part of the attention: the one block
// whose share holds it copies it from k_new / v_new into the cache and reads it from there, all others see the old
// rows only. kept_len itself is bumped by the merge kernel, after every block of both kernels has read the old value
// (merge blocks read the length the partial kernel recorded in the workspace instead). A segment without room for the
// row (or one that selection refused) is left as it is and MADAKV_ECAPACITY is recorded.
struct SegView {
  int len;      // rows attention covers, the appended one included
  int new_row;  // its index in the segment, or -1
};
__device__ __forceinline__ SegView segment_view(const DecodeParams& p, int u, bool reporter) {
  SegView v;
  v.len = segment_rows(p, u);
  v.new_row = -1;
  if (p.k_new) {
    const int len = p.kept_len[u];
    if (segment_refused(p, u) || len < 0 || p.seg_off[u] + (int64_t)len + 1 > p.seg_off[u + 1]) {
      if (reporter) set_status(p.ws, MADAKV_ECAPACITY);
    } else {
      v.new_row = len;
      v.len = len + 1;
    }
  }
  return v;
}
// The owner of the appended row (the block whose rows include it) stores it into the cache.
template <int ROW_BYTES>
__device__ __forceinline__ void store_new_row(const DecodeParams& p, int u, int64_t off, const SegView& v, int row_begin,
                                              int row_end) {
  constexpr int LPR = ROW_BYTES / 16;
  if (v.new_row < row_begin || v.new_row >= row_end || (int)threadIdx.x >= LPR) return;
  const int64_t row = off + v.new_row;
  const uint4 kv = *reinterpret_cast<const uint4*>((const char*)p.k_new + (int64_t)u * ROW_BYTES + threadIdx.x * 16);
  const uint4 vv = *reinterpret_cast<const uint4*>((const char*)p.v_new + (int64_t)u * ROW_BYTES + threadIdx.x * 16);
  *reinterpret_cast<uint4*>((char*)p.k_c + row * ROW_BYTES + threadIdx.x * 16) = kv;
  *reinterpret_cast<uint4*>((char*)p.v_c + row * ROW_BYTES + threadIdx.x * 16) = vv;
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

  pdl_wait();
  pdl_go();
  const int y = p.slot_fast ? blockIdx.x / p.slots : blockIdx.x % p.n_sel;
  const int u = unit_of(p, y);
  const int slot = p.slot_fast ? blockIdx.x % p.slots : blockIdx.x / p.n_sel;
  const SegView view = segment_view(p, u, slot == 0 && threadIdx.x == 0);
  const int len = view.len;
  if (slot == 0 && threadIdx.x == 0 && p.eff_len) p.eff_len[u] = len;
  if (slot >= segment_blocks(p, len)) return;
  int row_begin, row_end;
  block_rows(p, len, slot, row_begin, row_end);
  const int64_t off = p.seg_off[u];
  store_new_row<ROW_BYTES>(p, u, off, view, row_begin, row_end);
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
  // the appended row is read from where it comes from, not from the cache row this block is writing
  const char* kn = view.new_row >= 0 ? (const char*)p.k_new + (int64_t)u * ROW_BYTES + lane * 16 : nullptr;
  const char* vn = view.new_row >= 0 ? (const char*)p.v_new + (int64_t)u * ROW_BYTES + lane * 16 : nullptr;
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
        const bool fresh = r == view.new_row;
        kraw[j] = __ldcs(reinterpret_cast<const uint4*>(fresh ? kn : kc + (int64_t)r * ROW_BYTES));
        vraw[j] = __ldcs(reinterpret_cast<const uint4*>(fresh ? vn : vc + (int64_t)r * ROW_BYTES));
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
    float* dst = p.part + (((int64_t)bl * p.Hq + h * p.g + i) * p.slots + slot) * (D + 2);
    dst[c] = O;
    if (c == 0) {
      dst[D] = M;
      dst[D + 1] = Lsum;
    }
  }
}

// ---- grouped-query partial on the warp-level tensor-core path (bf16, 3 <= g <= 16) ----------------------------------
// One K/V row serves g query heads: in scalar code that is 2 * g * D fused multiply-adds per 2 * D * 2 bytes read and
// the kernel is bound by the FMA pipe from g = 4 on. Here the g heads sit on the 16 rows of an m16n8k16 tile (rows
// beyond g carry zero queries): a warp takes 16 cache rows at a time, S = Q K^T as 2 key blocks x D/16 MMAs, the
// online softmax on the accumulator fragments, P rounded to bf16 and reused in place as the A operand of O += P V
// (D/8 MMAs). K and V rows go global -> shared with 16-byte asynchronous copies, double-buffered per warp, rows padded
// by 16 bytes so that the 8x8 matrix loads are free of bank conflicts. Warps work independently on interleaved
// 16-row chunks of the split and are merged in shared memory at its end.
constexpr int kMmaWarps = 4;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // zero bytes read: the 16 destination bytes are filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <int D>
struct MmaTile {
  static constexpr int PITCH = D * 2 + 16;            // bytes from one staged row to the next
  static constexpr int TILE = 16 * PITCH;             // 16 rows of K or of V
  static constexpr int WARP = 4 * TILE;               // two buffers of (K, V)
  static constexpr int OPITCH = D + 8;                // floats from one head's merged row to the next
  static constexpr int BYTES = kMmaWarps * WARP;
  static_assert(16 * OPITCH * 4 + 2 * 16 * 4 <= WARP, "the merge staging reuses a warp's K/V buffers");
};

template <int D>
__global__ void __launch_bounds__(kMmaWarps * 32, 3) decode_partial_mma_kernel(DecodeParams p) {
  using MT = MmaTile<D>;
  constexpr int ROW_BYTES = D * 2;
  constexpr int LPR = ROW_BYTES / 16;  // 16-byte pieces per row
  constexpr int KC = D / 16;           // contraction chunks of Q K^T
  constexpr int NB = D / 8;            // 8-column blocks of the output
  extern __shared__ __align__(16) unsigned char dsmem[];

  pdl_wait();
  pdl_go();
  const int u = unit_of(p, p.slot_fast ? blockIdx.x / p.slots : blockIdx.x % p.n_sel);
  const int slot = p.slot_fast ? blockIdx.x % p.slots : blockIdx.x / p.n_sel;
  const SegView view = segment_view(p, u, slot == 0 && threadIdx.x == 0);
  const int len = view.len;
  if (slot == 0 && threadIdx.x == 0 && p.eff_len) p.eff_len[u] = len;
  if (slot >= segment_blocks(p, len)) return;
  int row_begin, row_end;
  block_rows(p, len, slot, row_begin, row_end);
  const int64_t off = p.seg_off[u];
  store_new_row<D * 2>(p, u, off, view, row_begin, row_end);
  const int h = u % p.Hkv, bl = u / p.Hkv;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int hr = lane / 4, t = lane % 4;  // fragment coordinates: row (head) hr and hr + 8, column pair t
  unsigned char* wsm = dsmem + warp * MT::WARP;
  const uint32_t wsm_a = smem_addr(wsm);

  // Q as A fragments, one per contraction chunk: (head hr, d 2t..2t+1), (head hr+8, same), (head hr, d 2t+8..), ...
  uint32_t qa[KC][4];
  {
    const __nv_bfloat16* q0 = reinterpret_cast<const __nv_bfloat16*>(p.q) + ((int64_t)bl * p.Hq + h * p.g) * D;
#pragma unroll
    for (int c = 0; c < KC; ++c) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int head = hr + 8 * (j & 1), dcol = c * 16 + 2 * t + 8 * (j >> 1);
        qa[c][j] = head < p.g ? *reinterpret_cast<const uint32_t*>(q0 + (int64_t)head * D + dcol) : 0u;
      }
    }
  }
  const char* kc = (const char*)p.k_c + off * ROW_BYTES;
  const char* vc = (const char*)p.v_c + off * ROW_BYTES;
  const char* kn = view.new_row >= 0 ? (const char*)p.k_new + (int64_t)u * ROW_BYTES : nullptr;
  const char* vn = view.new_row >= 0 ? (const char*)p.v_new + (int64_t)u * ROW_BYTES : nullptr;
  // per-lane shared-memory offsets of the matrix loads: lanes 8i..8i+7 address the rows of the i-th 8x8 matrix
  const int mi = lane / 8, mr = lane % 8;
  const uint32_t k_lane = ((mi >> 1) * 8 + mr) * MT::PITCH + (mi & 1) * 16;  // keys (mi/2)*8.., d half mi%2
  const uint32_t v_lane = ((mi & 1) * 8 + mr) * MT::PITCH + (mi >> 1) * 16;  // keys (mi%2)*8.., column block mi/2

  {
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    float o[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;

    auto load_chunk = [&](int r, int buf) {
      const uint32_t kd = wsm_a + buf * 2 * MT::TILE, vd = kd + MT::TILE;
#pragma unroll
      for (int x = lane; x < 16 * LPR; x += 32) {
        const int rr = x / LPR, cc = x % LPR;
        const bool valid = r + rr < row_end;
        const int64_t src = (int64_t)(valid ? r + rr : r) * ROW_BYTES + cc * 16;  // row r itself is always valid
        // (the appended row comes from k_new / v_new, not from the cache row this block is writing)
        const bool fresh = valid && r + rr == view.new_row;
        cp_async16(kd + rr * MT::PITCH + cc * 16, fresh ? kn + cc * 16 : kc + src, valid);
        cp_async16(vd + rr * MT::PITCH + cc * 16, fresh ? vn + cc * 16 : vc + src, valid);
      }
    };
    if (row_begin + 16 * warp < row_end) load_chunk(row_begin + 16 * warp, 0);
    cp_async_commit();
    for (int it = 0;; ++it) {
      const int r = row_begin + 16 * (warp + kMmaWarps * it);
      if (r >= row_end) break;
      const int buf = it & 1;
      if (r + 16 * kMmaWarps < row_end) load_chunk(r + 16 * kMmaWarps, buf ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
      __syncwarp();
      const uint32_t kb = wsm_a + buf * 2 * MT::TILE, vb = kb + MT::TILE;

      float s[2][4];
#pragma unroll
      for (int b = 0; b < 2; ++b) s[b][0] = s[b][1] = s[b][2] = s[b][3] = 0.f;
#pragma unroll
      for (int c = 0; c < KC; ++c) {
        uint32_t kf[4];
        ldmatrix_x4(kb + k_lane + c * 32, kf);
        mma_bf16_16816(s[0], qa[c], kf[0], kf[1]);
        mma_bf16_16816(s[1], qa[c], kf[2], kf[3]);
      }
      // element j of block b: head hr + 8 * (j / 2), key r + 8 * b + 2 * t + (j & 1)
#pragma unroll
      for (int b = 0; b < 2; ++b)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          s[b][j] = (r + 8 * b + 2 * t + (j & 1) < row_end) ? s[b][j] * p.scale2 : -INFINITY;
      float f[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float mx = fmaxf(fmaxf(s[0][2 * e], s[0][2 * e + 1]), fmaxf(s[1][2 * e], s[1][2 * e + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mn = fmaxf(m[e], mx);  // finite: key r of the chunk is valid
        f[e] = fast_ex2(m[e] - mn);        // exp2(-inf) = 0 on the first chunk
        m[e] = mn;
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          s[b][2 * e] = fast_ex2(s[b][2 * e] - mn);
          s[b][2 * e + 1] = fast_ex2(s[b][2 * e + 1] - mn);
        }
        l[e] = l[e] * f[e] + ((s[0][2 * e] + s[0][2 * e + 1]) + (s[1][2 * e] + s[1][2 * e + 1]));
      }
      if (__any_sync(0xffffffffu, f[0] != 1.f || f[1] != 1.f)) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          o[nb][0] *= f[0]; o[nb][1] *= f[0];
          o[nb][2] *= f[1]; o[nb][3] *= f[1];
        }
      }
      uint32_t pa[4];
      pa[0] = pack_bf16x2(s[0][0], s[0][1]);
      pa[1] = pack_bf16x2(s[0][2], s[0][3]);
      pa[2] = pack_bf16x2(s[1][0], s[1][1]);
      pa[3] = pack_bf16x2(s[1][2], s[1][3]);
#pragma unroll
      for (int nb = 0; nb < NB; nb += 2) {
        uint32_t vf[4];
        ldmatrix_x4_trans(vb + v_lane + nb * 16, vf);
        mma_bf16_16816(o[nb], pa, vf[0], vf[1]);
        mma_bf16_16816(o[nb + 1], pa, vf[2], vf[3]);
      }
      __syncwarp();  // the buffer is refilled two iterations on
    }
    cp_async_wait<0>();
    __syncwarp();
    // the warp's state goes to its own (now idle) staging area: o[16][D + 8], then m[16], l[16]
    float* so = reinterpret_cast<float*>(wsm);
    float* sm = so + 16 * MT::OPITCH;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      l[e] += __shfl_xor_sync(0xffffffffu, l[e], 1);
      l[e] += __shfl_xor_sync(0xffffffffu, l[e], 2);
      if (t == 0) {
        sm[hr + 8 * e] = m[e];
        sm[16 + hr + 8 * e] = l[e];
      }
    }
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      *reinterpret_cast<float2*>(so + hr * MT::OPITCH + nb * 8 + 2 * t) = make_float2(o[nb][0], o[nb][1]);
      *reinterpret_cast<float2*>(so + (hr + 8) * MT::OPITCH + nb * 8 + 2 * t) = make_float2(o[nb][2], o[nb][3]);
    }
    __syncthreads();
    for (int x = threadIdx.x; x < p.g * D; x += kMmaWarps * 32) {
      const int i = x / D, c = x % D;
      float mw[kMmaWarps], M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kMmaWarps; ++w) {
        mw[w] = reinterpret_cast<const float*>(dsmem + w * MT::WARP)[16 * MT::OPITCH + i];
        M = fmaxf(M, mw[w]);
      }
      float Lsum = 0.f, O = 0.f;
#pragma unroll
      for (int w = 0; w < kMmaWarps; ++w) {
        const float* wo = reinterpret_cast<const float*>(dsmem + w * MT::WARP);
        const float fw = (mw[w] == -INFINITY) ? 0.f : exp2f(mw[w] - M);
        Lsum += wo[16 * MT::OPITCH + 16 + i] * fw;
        O += wo[i * MT::OPITCH + c] * fw;
      }
      float* dst = p.part + (((int64_t)bl * p.Hq + h * p.g + i) * p.slots + slot) * (D + 2);
      dst[c] = O;
      if (c == 0) {
        dst[D] = M;
        dst[D + 1] = Lsum;
      }
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(D) decode_merge_kernel(DecodeParams p) {
  // blockIdx.x enumerates the query heads of the selected layer(s)
  pdl_wait();
  pdl_go();
  int row;
  if (p.layer < 0) {
    row = blockIdx.x;
  } else {
    const int b = blockIdx.x / p.Hq, hq = blockIdx.x % p.Hq;
    row = (b * p.L + p.layer) * p.Hq + hq;
  }
  const int bl = row / p.Hq, hq = row % p.Hq;
  const int u = bl * p.Hkv + hq / p.g;
  // an appending call: the length the partial kernel worked with; the first head of the group makes it the segment's
  const int len = p.eff_len ? p.eff_len[u] : segment_rows(p, u);
  if (p.eff_len && hq % p.g == 0 && threadIdx.x == 0 && len > p.kept_len[u]) p.kept_len[u] = len;
  const int used = segment_blocks(p, len);
  const float* part = p.part + (int64_t)row * p.slots * (D + 2);
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

// Smallest share of a segment that a block takes. 512 rows when there are segments enough to fill the GPU (shorter
// shares leave a block's load pipeline no time to fill and cost more merge work: measured 5-8 % at 256 rows); a call
// with few segments (one layer of a long-context model: 8 segments) is bound by the latency of its longest block,
// and there shorter shares spread a segment over more blocks: 128 rows for the scalar kernel (one layer of the llava
// workload: 747 -> 488 us for the 32 layers of a step), 256 for the tensor-core kernel, whose four warps take 64
// rows per iteration (at 128 rows it lost more in merge work than it gained: long 429 -> 471 us, at 256: 426).
int min_share_rows(int n_sel, bool tensor_core_kernel) {
  return n_sel >= 64 ? kDecodeMinRows : (tensor_core_kernel ? 256 : 128);
}

// Blocks launched per segment (the grid is segments x this number, and a block whose share of its segment is empty
// returns at once). With segments enough to fill the GPU 8 is plenty, and the thousands of blocks that 32 per segment
// launched only to return cost a tenth of the call (batched 246 -> 219 us, qwen 26.6 -> 23.8); a long segment then
// simply gets longer shares. A call with few segments keeps 32 (scalar kernel) or 16 (tensor-core kernel).
int blocks_per_segment(int n_sel, bool tensor_core_kernel, int splits) {
  const int want = n_sel >= 64 ? 8 : (tensor_core_kernel ? 16 : kDecodeSlots);
  return splits < want ? splits : want;
}

// Block order of the grid. With many segments a segment's blocks follow one another (neighbouring blocks stream
// neighbouring rows); with fewer segments than SMs the grid is a wave or two, and then the blocks are ordered by slot so
// that every segment's last and shortest block is scheduled last.
int slot_order(int n_sel) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 1;
  return n_sel >= sms ? 1 : 0;
}

template <typename T, int D>
int run(const DecodeParams& p, const madakv_config&, cudaStream_t st) {
  const int n_sel = p.n_sel;
  // every host-side refusal comes before the first launch (an appending call changes the cache)
  const bool mma = sizeof(T) == 2 && p.g >= 3 && p.g <= 16;
  if (!mma && p.g > 8) return MADAKV_EUNSUPPORTED;
  if constexpr (sizeof(T) == 2) {
    if (mma && cudaFuncSetAttribute(decode_partial_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    MmaTile<D>::BYTES) != cudaSuccess)
      return MADAKV_ECUDA;
  }
  const dim3 grid((unsigned)n_sel * p.slots);  // one dimension: no 65535 limit on the number of segments
  if constexpr (sizeof(T) == 2) {
    if (mma) launch_pdl(decode_partial_mma_kernel<D>, grid, dim3(kMmaWarps * 32), MmaTile<D>::BYTES, st, p);
  }
  if (mma) {
  } else if (p.g == 1) launch_pdl(decode_partial_kernel<T, D, 1>, grid, dim3(NT), 0, st, p);
  else if (p.g == 2) launch_pdl(decode_partial_kernel<T, D, 2>, grid, dim3(NT), 0, st, p);
  else if (p.g <= 4) launch_pdl(decode_partial_kernel<T, D, 4>, grid, dim3(NT), 0, st, p);
  else launch_pdl(decode_partial_kernel<T, D, 8>, grid, dim3(NT), 0, st, p);
  // (the merge may be scheduled while the partial kernel runs; it waits for its completion before reading anything)
  launch_pdl(decode_merge_kernel<T, D>, dim3(n_sel * p.g), dim3(D), 0, st, p);
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
  p.eff_len = k_new ? reinterpret_cast<int32_t*>((char*)ws + wl.decode_len_off) : nullptr;
  p.ws = ws;
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = c.n_q_heads / c.n_kv_heads;
  p.layer = layer;
  p.n_sel = (layer < 0 ? c.batch * c.n_layers : c.batch) * c.n_kv_heads;
  const bool tc = c.dtype == MADAKV_BF16 && p.g >= 3 && p.g <= 16;
  p.slots = blocks_per_segment(p.n_sel, tc, wl.decode_splits);
  p.min_rows = min_share_rows(p.n_sel, tc);
  p.slot_fast = slot_order(p.n_sel);
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
  p.eff_len = nullptr;
  p.ws = nullptr;  // only an appending call reports through the workspace
  p.L = c.n_layers;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.g = c.n_q_heads / c.n_kv_heads;
  p.layer = layer;
  p.n_sel = (layer < 0 ? c.batch * c.n_layers : c.batch) * c.n_kv_heads;
  const bool tc = c.dtype == MADAKV_BF16 && p.g >= 3 && p.g <= 16;
  p.slots = blocks_per_segment(p.n_sel, tc, splits);  // what the kernels use of the (larger) documented bound
  p.min_rows = min_share_rows(p.n_sel, tc);
  p.slot_fast = slot_order(p.n_sel);
  p.scale2 = scale_of(c) * kLog2e;
  cudaStream_t st = (cudaStream_t)stream;
  if (c.dtype == MADAKV_F32) return c.head_dim == 64 ? run<float, 64>(p, c, st) : run<float, 128>(p, c, st);
  return c.head_dim == 64 ? run<__nv_bfloat16, 64>(p, c, st) : run<__nv_bfloat16, 128>(p, c, st);
}
