// Stage 4a: per-head, per-modality top-budget selection (Section 3.3, the eviction step after Eq. 8).
//
//   seg_scan     one block: kept_len[u] = b_v + b_t and the exclusive scan seg_off (rows, with headroom)
//   select_unit  one block per unit: a 4-pass shared-memory radix select over the order-preserving bit pattern of
//                psi finds, for both modalities at once, the budget-th largest value and how many of its ties are
//                still needed; an ordered sweep then emits the kept positions in ascending order, giving ties to
//                the lowest positions (block-wide prefix scans provide the tie ranks and the output slots).
// Integer work only: results are bit-exact functions of (psi bits, mask, budgets).
#include "common.cuh"

namespace madakv {
namespace {

constexpr int NT = 256;
constexpr int ITEMS = 4;               // positions per thread per sweep step
constexpr int STEP = NT * ITEMS;       // 1024 positions per sweep step

struct SelParams {
  const float* psi;
  const uint8_t* mask;
  const int32_t* seq_len;
  const int32_t* budgets;
  int32_t* kept_len;
  int64_t* seg_off;
  int32_t* kept_idx;
  int64_t capacity;
  void* ws;
  int32_t* seq_nv;  // ws: visual-token count of every sequence
  int units, L, Hkv, n_max, mpa, headroom;
};

// One block per sequence: number of visual tokens among the first seq_len[b] positions.
__global__ void __launch_bounds__(1024) count_visual_kernel(SelParams p) {
  __shared__ int s_cnt;
  const int b = blockIdx.x;
  const int n = min(p.seq_len[b], p.n_max);
  const uint8_t* mask = p.mask + (int64_t)b * p.n_max;
  if (threadIdx.x == 0) s_cnt = 0;
  __syncthreads();
  int c = 0;
  for (int i = threadIdx.x; i < n; i += 1024) c += mask[i] ? 1 : 0;
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
  if ((threadIdx.x & 31) == 0) atomicAdd(&s_cnt, c);
  __syncthreads();
  if (threadIdx.x == 0) p.seq_nv[b] = p.mpa ? s_cnt : 0;
}

__global__ void __launch_bounds__(1024) seg_scan_kernel(SelParams p) {
  __shared__ long long warp_tot[32];
  __shared__ long long carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < p.units; base += 1024) {
    const int u = base + threadIdx.x;
    long long v = 0;
    if (u < p.units) {
      const int b = u / (p.Hkv * p.L);
      const int n = min(p.seq_len[b], p.n_max);
      const int n_v = p.seq_nv[b];
      const int len = (p.mpa ? min(max(p.budgets[2 * u], 0), n_v) : 0) + min(max(p.budgets[2 * u + 1], 0), n - n_v);
      p.kept_len[u] = len;
      v = (long long)len + p.headroom;
    }
    long long incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long t = __shfl_up_sync(0xffffffffu, incl, off);
      if ((threadIdx.x & 31) >= off) incl += t;
    }
    if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = incl;
    __syncthreads();
    long long wbase = 0;
    for (int i = 0; i < (int)(threadIdx.x >> 5); ++i) wbase += warp_tot[i];
    const long long excl = carry + wbase + incl - v;
    if (u < p.units) p.seg_off[u] = excl;
    __syncthreads();
    if (threadIdx.x == 1023) carry = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    p.seg_off[p.units] = carry;
    if (carry > p.capacity) set_status(p.ws, MADAKV_ECAPACITY);
  }
}

// Exclusive block scan of a packed pair of 16-bit counters (each total <= STEP < 65536).
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  uint32_t incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, off);
    if ((threadIdx.x & 31) >= off) incl += t;
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = incl;
  __syncthreads();
  uint32_t wbase = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < NT / 32; ++i) {
    const uint32_t t = warp_tot[i];
    if (i < (int)(threadIdx.x >> 5)) wbase += t;
    tot += t;
  }
  *total = tot;
  return wbase + incl - v;
}

__global__ void __launch_bounds__(NT) select_unit_kernel(SelParams p) {
  __shared__ unsigned int cnt[2][256];
  __shared__ uint32_t s_prefix[2];
  __shared__ unsigned int s_above[2];
  __shared__ uint32_t warp_tot[NT / 32];

  const int u = blockIdx.x;
  const int b = u / (p.Hkv * p.L);
  const int n = min(p.seq_len[b], p.n_max);
  const float* psi = p.psi + (int64_t)u * p.n_max;
  const uint8_t* mask = p.mask + (int64_t)b * p.n_max;
  const int64_t off0 = p.seg_off[u];
  if (off0 + p.kept_len[u] + p.headroom > p.capacity) return;  // seg_scan has raised MADAKV_ECAPACITY
  const int want[2] = {p.mpa ? max(p.budgets[2 * u], 0) : 0, max(p.budgets[2 * u + 1], 0)};

  if (threadIdx.x < 2) {
    s_prefix[threadIdx.x] = 0;
    s_above[threadIdx.x] = 0;
  }
  // radix select: after the 4 passes s_prefix[m] is the want[m]-th largest key of modality m (if that many exist)
  // and s_above[m] counts the keys strictly above it
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_round = (n + 31) & ~31;  // whole warps run every iteration (the match below is a warp-wide call)
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int x = threadIdx.x; x < 512; x += NT) (&cnt[0][0])[x] = 0;
    __syncthreads();
    const uint32_t pre0 = s_prefix[0], pre1 = s_prefix[1];
    for (int i = threadIdx.x; i < n_round; i += NT) {
      int bucket = -1;
      if (i < n) {
        const uint32_t key = psi_key(psi[i]);
        const int m = (p.mpa && mask[i]) ? 0 : 1;
        if ((key & himask) == (m == 0 ? pre0 : pre1)) bucket = m * 256 + (int)((key >> shift) & 255u);
      }
      // lanes that hit the same bucket are counted by one of them: importance values cluster in a few exponent
      // buckets, and per-lane atomics on them would serialise
      const unsigned int peers = __match_any_sync(0xffffffffu, bucket);
      if (bucket >= 0 && lane == __ffs(peers) - 1) atomicAdd(&(&cnt[0][0])[bucket], (unsigned int)__popc(peers));
    }
    __syncthreads();
    if (warp < 2) {
      // warp m walks modality m's buckets from the top; lane j owns buckets 8j..8j+7
      const int m = warp;
      unsigned int cs[8], lc = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        cs[j] = cnt[m][lane * 8 + j];
        lc += cs[j];
      }
      unsigned int sc = lc;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_down_sync(0xffffffffu, sc, off);
        if (lane + off < 32) sc += t;
      }
      unsigned int above = s_above[m] + (sc - lc);
      int found = -1;
#pragma unroll
      for (int j = 7; j >= 0; --j) {
        if (found < 0) {
          if (above + cs[j] >= (unsigned int)want[m] || (lane == 0 && j == 0)) found = j;
          else above += cs[j];
        }
      }
      const unsigned int hit = __ballot_sync(0xffffffffu, found >= 0);  // lane 0 always hits
      if (lane == 31 - __clz(hit)) {
        s_above[m] = above;
        s_prefix[m] |= (uint32_t)(lane * 8 + found) << shift;
      }
    }
    __syncthreads();
  }
  const uint32_t thr[2] = {s_prefix[0], s_prefix[1]};
  // ties at the threshold value that are still needed (all of them if the modality has fewer tokens than wanted)
  const int ties[2] = {max(want[0] - (int)s_above[0], 0), max(want[1] - (int)s_above[1], 0)};

  // ordered sweep
  int tie_run[2] = {0, 0};  // threshold-valued keys met so far, per modality
  int out_run = 0;          // kept positions emitted so far
  for (int base = 0; base < n; base += STEP) {
    uint32_t key[ITEMS];
    int mod[ITEMS];
    uint32_t eq_pack = 0;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      const int i = base + threadIdx.x * ITEMS + j;
      key[j] = 0;
      mod[j] = -1;
      if (i < n) {
        key[j] = psi_key(psi[i]);
        mod[j] = (p.mpa && mask[i]) ? 0 : 1;
        if (key[j] == thr[mod[j]]) eq_pack += mod[j] == 0 ? 1u : 0x10000u;
      }
    }
    uint32_t eq_total;
    uint32_t eq_before = block_excl_scan(eq_pack, warp_tot, &eq_total);
    int rank[2] = {tie_run[0] + (int)(eq_before & 0xffffu), tie_run[1] + (int)(eq_before >> 16)};
    uint32_t keep_bits = 0, keep_cnt = 0;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      if (mod[j] < 0) continue;
      const int m = mod[j];
      bool keep = false;
      if (want[m] > 0) {
        if (key[j] > thr[m]) keep = true;
        else if (key[j] == thr[m]) {
          keep = rank[m] < ties[m];
          rank[m] += 1;
        }
      }
      if (keep) {
        keep_bits |= 1u << j;
        keep_cnt += 1;
      }
    }
    uint32_t keep_total;
    const uint32_t slot = block_excl_scan(keep_cnt, warp_tot, &keep_total);
    int o = out_run + (int)slot;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j)
      if (keep_bits & (1u << j)) p.kept_idx[off0 + o++] = base + threadIdx.x * ITEMS + j;
    tie_run[0] += (int)(eq_total & 0xffffu);
    tie_run[1] += (int)(eq_total >> 16);
    out_run += (int)keep_total;
  }
}

}  // namespace

int launch_select(const madakv_config& c, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                  const int32_t* budgets, int32_t* kept_len, int64_t* seg_off, int32_t* kept_idx, int64_t capacity,
                  void* ws, cudaStream_t st) {
  SelParams p;
  p.psi = psi;
  p.mask = mask;
  p.seq_len = seq_len;
  p.budgets = budgets;
  p.kept_len = kept_len;
  p.seg_off = seg_off;
  p.kept_idx = kept_idx;
  p.capacity = capacity;
  p.ws = ws;
  p.units = c.batch * c.n_layers * c.n_kv_heads;
  p.L = c.n_layers;
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.mpa = c.mpa;
  p.headroom = c.max_new_tokens;
  p.seq_nv = reinterpret_cast<int32_t*>((char*)ws + ws_layout(c).seq_nv_off);
  count_visual_kernel<<<c.batch, 1024, 0, st>>>(p);
  seg_scan_kernel<<<1, 1024, 0, st>>>(p);
  select_unit_kernel<<<p.units, NT, 0, st>>>(p);
  return launch_status();
}

}  // namespace madakv
