// Shared pieces of the tensor-core scoring kernels: PTX wrappers (mbarrier, TMA, tcgen05, TMEM loads, packed fp32
// arithmetic), the bounded wait, the exponent loops of the epilogue, and the host-side tensor-map encoder.
#pragma once

#include <cuda.h>
#include <cstdlib>
#include <type_traits>

#include "common.cuh"

namespace madakv {
namespace {

constexpr int kTileKeys = 128;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kEmptyMax = -1.0e30f;               // "no key seen yet" marker of a running maximum
constexpr long long kWaitCycles = 4000000000ll;     // ~2 s at B200 clocks: bound of every device-side wait

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a barrier phase (try_wait may suspend the thread for a while; this never does).
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Records a wait that ran out: the status word, and (for diagnosis) which wait it was.
enum { kSiteQEmpty = 1, kSiteStage = 2, kSiteQFull = 3, kSiteTEmpty = 4, kSiteFull = 5, kSiteTile = 6, kSiteFlag = 7,
       kSiteDrain = 8 };
__device__ __forceinline__ void give_up(volatile int* abort_flag, int32_t* status, int site) {
  *abort_flag = 1;
  if (atomicCAS(status, 0, (int)MADAKV_ETIMEOUT) == 0) status[1] = site | ((int)blockIdx.x << 8);
}
// Bounded wait. Returns false if the wait was abandoned (own timeout or another role's abort flag).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          int site) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 63) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        give_up(abort_flag, status, site);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// 5-D tiled TMA load into this CTA's shared memory, completion signalled on an mbarrier.
__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes packed densely
// (8-row groups 1024 bytes apart), descriptor version 1. Only the low word depends on the address: start address
// in 16-byte units (bits 0-13) and the unused leading byte offset (bit 16); the high word holds the stride byte
// offset (1024 >> 4), the version (bit 46) and SWIZZLE_128B (bits 61-63). Moving the start by x bytes (x a multiple
// of 16, same operand buffer) adds x >> 4 to the low word, which is all the MMA issue loop has to do per instruction.
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | (1u << 16); }
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_desc_lo, uint32_t b_desc_lo, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 da, db;\nsetp.ne.b32 p, %4, 0;\nmov.b64 da, {%1, %5};\nmov.b64 db, {%2, %5};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_desc_lo), "r"(b_desc_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// Issue a 16-column TMEM load of this thread's lane; the registers are valid only after tmem_ld_wait16 on them (the
// registers pass through that statement so that no use of them can be scheduled before the wait). The epilogue
// works on blocks of 16 window rows so that two blocks (one being processed, one in flight) fit the register budget.
#define MADAKV_R8(r, o) "+r"(r[o]), "+r"(r[o + 1]), "+r"(r[o + 2]), "+r"(r[o + 3]), "+r"(r[o + 4]), "+r"(r[o + 5]), \
                        "+r"(r[o + 6]), "+r"(r[o + 7])
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait16(uint32_t (&a)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : MADAKV_R8(a, 0), MADAKV_R8(a, 8) : : "memory");
}
// Ties 16 more registers to the wait before them (no instruction): the second half of a 32-column chunk.
__device__ __forceinline__ void tmem_ld_tie16(uint32_t (&a)[16]) {
  asm volatile("" : MADAKV_R8(a, 0), MADAKV_R8(a, 8) : : "memory");
}
#undef MADAKV_R8
__device__ __forceinline__ float warp_max(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
// packed pairs of fp32 (sm_100 f32x2 arithmetic): one instruction per two logits
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pack2u(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// three-input maximum (sm_100)
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Sum over the 32 lanes of 32 per-lane values, transposed: lane j returns the sum over all lanes of their v[j]. Five
// exchange rounds (31 shuffles) in registers; the order of the additions is fixed (a tree over lane pairs).
__device__ __forceinline__ float warp_rowsum32(float (&v)[32]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    const bool up = (lane & m) != 0;
#pragma unroll
    for (int i = 0; i < m; ++i) {
      const float keep = up ? v[i + m] : v[i];
      const float send = up ? v[i] : v[i + m];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, m);
    }
  }
  return v[0];
}
// (max, sum) merge of two partial softmax statistics in the log2 domain.
__device__ __forceinline__ void merge_stats(float& m, float& z, float mo, float zo) {
  const float mn = fmaxf(m, mo);
  z = z * ex2(m - mn) + zo * ex2(mo - mn);
  m = mn;
}

// exp2 of 16 scaled-and-shifted logits, added to 8 packed accumulators (acc2[i] += exp2(raw * scale - shift)), or
// all summed into one packed accumulator (phase 2: sum over window rows)
__device__ __forceinline__ void exp_accumulate16(const uint32_t (&raw)[16], uint64_t scale2x, const uint64_t* negshift2,
                                                 uint64_t* acc2) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float lo, hi;
    unpack2(fma2(pack2u(raw[2 * i], raw[2 * i + 1]), scale2x, negshift2[i]), lo, hi);
    acc2[i] = add2(acc2[i], pack2(ex2(lo), ex2(hi)));
  }
}
__device__ __forceinline__ uint64_t exp_sum16(const uint32_t (&raw)[16], uint64_t scale2x, const uint64_t* negshift2,
                                              uint64_t acc) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float lo, hi;
    unpack2(fma2(pack2u(raw[2 * i], raw[2 * i + 1]), scale2x, negshift2[i]), lo, hi);
    acc = add2(acc, pack2(ex2(lo), ex2(hi)));
  }
  return acc;
}
// logits of keys a window row may not see are replaced by a huge negative value
__device__ __forceinline__ void mask_block16(uint32_t (&raw)[16], int key, const int* vis) {
#pragma unroll
  for (int c = 0; c < 16; ++c)
    if (key >= vis[c]) raw[c] = __float_as_uint(kEmptyMax);
}
// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// [B, L, H, tokens, d] bf16 tensor with element strides -> 5-D map, box = {64, box_tokens, box_heads, 1, 1}.
bool make_map(CUtensorMap* map, const void* base, int d, int tokens, int heads, int L, int B, madakv_strides s,
              int box_tokens, int box_heads) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[5] = {(cuuint64_t)d, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)L, (cuuint64_t)B};
  // a dimension of extent 1 never advances; give it a harmless valid stride if the caller's is 0
  auto st = [&](int64_t v, int64_t fallback) { return (cuuint64_t)((v > 0 ? v : fallback) * 2); };
  const int64_t tok = s.token;
  const cuuint64_t strides[4] = {st(s.token, d), st(s.head, tok * tokens), st(s.layer, tok * tokens * heads),
                                 st(s.batch, tok * tokens * heads * L)};
  for (int i = 0; i < 4; ++i)
    if (strides[i] % 16 || strides[i] >= ((cuuint64_t)1 << 40)) return false;
  const cuuint32_t box[5] = {64, (cuuint32_t)box_tokens, (cuuint32_t)box_heads, 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace madakv
