// Stage 4a: per-head, per-modality top-budget selection (Section 3.3, the eviction step after Eq. 8).
//
//   seg_scan     one block: visual-token count of every sequence, kept_len[u] = b_v + b_t and the exclusive scan
//                seg_off (rows, with headroom)
//   select_unit  one block per unit: a three- or four-pass shared-memory radix select over the order-preserving bit pattern of
//                psi finds, for both modalities at once, the budget-th largest value and how many of its ties are
//                still needed; an ordered sweep then emits the kept positions in ascending order, giving ties to
//                the lowest positions (block-wide prefix scans provide the tie ranks and the output slots).
//                A thread owns KPT consecutive positions and keeps their keys in registers from the first pass to
//                the sweep (sequences longer than one chunk are re-read from L2 chunk by chunk).
// Two options outside the paper: with pooling the ranking key of a position is the maximum of the keys of the
// positions around it (a maximum of fp32 values is exact, so nothing changes for the integer results); with
// forced retention the proxy tokens are emitted by the sweep without taking part in the ranking, and the wanted
// counts shrink by their number.
// Integer work only: results are bit-exact functions of (psi bits, mask, budgets).
#include "common.cuh"

namespace madakv {
namespace {

constexpr int NT = 256;
constexpr int KPT = 32;                // consecutive positions per thread
constexpr int CHUNK = NT * KPT;        // 8192 positions per chunk
constexpr unsigned int kFull = 0xffffffffu;
// A radix digit has DIG bits: 10 for configs whose sequences are longer than one chunk (they are re-read from L2 in
// every pass, and the 30 bits in which importance values differ at most then take three passes instead of four),
// 8 for those that sit in registers (the larger histograms only cost there). Bucket b of a modality sits at word
// b + b / kPerLane, so that the lanes of the walking warp (lane j owns buckets kPerLane * j ..) read 32 different banks.

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
  int32_t* seq_wv;  // ws: visual tokens among the proxy tokens of every sequence (forced retention)
  int units, B, L, Hkv, n_max, mpa, headroom, keep_window, window, pool_r;  // pool_r: (pool_kernel - 1) / 2
};

__global__ void __launch_bounds__(1024) seg_scan_kernel(SelParams p) {
  __shared__ long long warp_tot[32];
  __shared__ long long carry;
  __shared__ int s_cnt, s_wcnt;
  // visual tokens among the first seq_len[b] positions of every sequence
  for (int b = 0; b < p.B; ++b) {
    const int n = clamped_len(p.seq_len, b, p.n_max);
    const uint8_t* mask = p.mask + (int64_t)b * p.n_max;
    const int wfrom = p.keep_window ? max(n - p.window, 0) : n;  // first proxy token retained unconditionally
    if (threadIdx.x == 0) s_cnt = s_wcnt = 0;
    __syncthreads();
    int c = 0, cw = 0;  // visual tokens, visual proxy tokens
    if (p.mpa) {
      int done = 0;
      if ((reinterpret_cast<uintptr_t>(mask) & 15) == 0) {  // 16 mask bytes per load
        const int n16 = n >> 4;
        for (int i = threadIdx.x; i < n16; i += 1024) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask) + i);
          c += __popc(nonzero_bytes(v.x) | (nonzero_bytes(v.y) << 4) | (nonzero_bytes(v.z) << 8) | (nonzero_bytes(v.w) << 12));
        }
        done = n16 << 4;
      }
      for (int i = done + threadIdx.x; i < n; i += 1024) c += mask[i] ? 1 : 0;
      for (int i = wfrom + threadIdx.x; i < n; i += 1024) cw += mask[i] ? 1 : 0;  // (no proxy tokens: wfrom = n)
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      c += __shfl_xor_sync(kFull, c, off);
      cw += __shfl_xor_sync(kFull, cw, off);
    }
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&s_cnt, c);
    if ((threadIdx.x & 31) == 0 && cw) atomicAdd(&s_wcnt, cw);
    __syncthreads();
    if (threadIdx.x == 0) {
      p.seq_nv[b] = s_cnt;
      p.seq_wv[b] = s_wcnt;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();  // also orders the seq_nv stores before the loads below (same block)
  for (int base = 0; base < p.units; base += 1024) {
    const int u = base + threadIdx.x;
    long long v = 0;
    if (u < p.units) {
      const int b = u / (p.Hkv * p.L);
      const int n = clamped_len(p.seq_len, b, p.n_max);
      const int n_v = p.seq_nv[b];
      const int lo_v = p.seq_wv[b], lo_t = (p.keep_window ? min(p.window, n) : 0) - lo_v;  // proxy tokens kept anyway
      const int len = (p.mpa ? min(max(p.budgets[2 * u], lo_v), n_v) : 0) + min(max(p.budgets[2 * u + 1], lo_t), n - n_v);
      p.kept_len[u] = len;
      v = (long long)len + p.headroom;
    }
    long long incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const long long t = __shfl_up_sync(kFull, incl, off);
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

// Exclusive block scan of a packed pair of 16-bit counters (each total <= CHUNK < 65536).
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  uint32_t incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, incl, off);
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

constexpr int kMaxPoolR = 7;  // pool_kernel <= 15

// Keys of KPT consecutive positions from pos0. valid: positions that take part in the ranking (inside the sequence
// and not retained unconditionally); forced: proxy tokens retained unconditionally (positions wfrom .. n-1);
// vis: visual tokens. kPool is the variant for the two options outside the paper: the key of a position is the maximum
// over the 2 * pool_r + 1 positions around it (pool_r may be 0), and the proxy tokens from wfrom on are forced; without
// kPool neither exists and the code is the plain paper-literal selection.
template <bool kVec, bool kPool>
__device__ __forceinline__ void load_chunk(const float* psi, const uint8_t* mask, int n, int pos0, int mpa, int wfrom,
                                           int pool_r, uint32_t (&key)[KPT], uint32_t& valid, uint32_t& vis,
                                           uint32_t& forced) {
  valid = 0;
  vis = 0;
  forced = 0;
  if (kPool) {
    uint32_t e[KPT + 2 * kMaxPoolR];  // keys of positions pos0 - 7 .. pos0 + KPT + 6 (0 outside the sequence)
#pragma unroll
    for (int x = 0; x < KPT + 2 * kMaxPoolR; ++x) {
      const int pos = pos0 - kMaxPoolR + x;
      e[x] = (pos >= 0 && pos < n) ? psi_key(__ldg(psi + pos)) : 0u;
    }
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      uint32_t m = e[j + kMaxPoolR];
#pragma unroll
      for (int d = 1; d <= kMaxPoolR; ++d)
        if (d <= pool_r) m = max(m, max(e[j + kMaxPoolR - d], e[j + kMaxPoolR + d]));
      key[j] = pos0 + j < n ? m : 0u;
      if (pos0 + j < n) valid |= 1u << j;
    }
  } else if (kVec && pos0 + KPT <= n) {
#pragma unroll
    for (int j = 0; j < KPT; j += 4) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(psi + pos0 + j));
      key[j] = psi_key(v.x);
      key[j + 1] = psi_key(v.y);
      key[j + 2] = psi_key(v.z);
      key[j + 3] = psi_key(v.w);
    }
    valid = 0xffffffffu;
  } else {
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      key[j] = 0;
      if (pos0 + j < n) {
        key[j] = psi_key(__ldg(psi + pos0 + j));
        valid |= 1u << j;
      }
    }
  }
  if (mpa) {
    if (kVec && pos0 + KPT <= n && (reinterpret_cast<uintptr_t>(mask + pos0) & 15) == 0) {  // 16 mask bytes per load
#pragma unroll
      for (int j = 0; j < KPT; j += 16) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask + pos0 + j));
        vis |= (nonzero_bytes(v.x) | (nonzero_bytes(v.y) << 4) | (nonzero_bytes(v.z) << 8) | (nonzero_bytes(v.w) << 12)) << j;
      }
    } else {
#pragma unroll
      for (int j = 0; j < KPT; ++j)
        if (pos0 + j < n && __ldg(mask + pos0 + j)) vis |= 1u << j;
    }
  }
  if (kPool && pos0 + KPT > wfrom) {  // proxy tokens retained unconditionally: out of the ranking, into the output
#pragma unroll
    for (int j = 0; j < KPT; ++j)
      if (pos0 + j >= wfrom && pos0 + j < n) forced |= 1u << j;
    valid &= ~forced;
  }
}

// The radix digits are taken from t = kmax - key, starting at the highest bit in which the unit's keys differ
// (kmax, kmin: largest and smallest key of the unit): importance values share their sign and most exponent bits,
// so digits of the raw key would put nearly all keys into a handful of buckets and serialise the shared atomics.
// Ascending t is descending importance.
template <bool kVec, bool kPool, int DIG>
__global__ void __launch_bounds__(NT) select_unit_kernel(SelParams p) {
  constexpr int kDigitBits = DIG, kBuckets = 1 << DIG, kPerLane = kBuckets / 32, kCntWords = kBuckets + 32;
  auto cnt_slot = [](uint32_t digit) { return (int)(digit + digit / kPerLane); };
  __shared__ unsigned int cnt[2][kCntWords];
  __shared__ uint32_t s_prefix[2];
  __shared__ unsigned int s_above[2];
  __shared__ uint32_t warp_tot[NT / 32];
  __shared__ uint32_t s_red[2][NT / 32];

  const int u = blockIdx.x;
  const int b = u / (p.Hkv * p.L);
  const int n = clamped_len(p.seq_len, b, p.n_max);
  const float* psi = p.psi + (int64_t)u * p.n_max;
  const uint8_t* mask = p.mask + (int64_t)b * p.n_max;
  const int64_t off0 = p.seg_off[u];
  if (off0 + p.kept_len[u] + p.headroom > p.capacity) return;  // seg_scan has raised MADAKV_ECAPACITY
  // proxy tokens retained unconditionally (none without cfg->keep_window): they are emitted by the sweep and the
  // ranking only has to find the rest of each modality's budget
  const int wfrom = kPool && p.keep_window ? max(n - p.window, 0) : n;
  const int lo_v = kPool ? p.seq_wv[b] : 0, lo_t = (n - wfrom) - lo_v;
  const int want0 = p.mpa ? max(p.budgets[2 * u] - lo_v, 0) : 0, want1 = max(p.budgets[2 * u + 1] - lo_t, 0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = (n + CHUNK - 1) / CHUNK;

  // range of the unit's keys (the chunk stays in registers when there is only one)
  uint32_t key[KPT], valid = 0, vis = 0, forced = 0;
  uint32_t kmax = 0, kmin = 0xffffffffu;
  for (int c = 0; c < chunks; ++c) {
    load_chunk<kVec, kPool>(psi, mask, n, c * CHUNK + (int)threadIdx.x * KPT, p.mpa, wfrom, p.pool_r, key, valid, vis, forced);
#pragma unroll
    for (int j = 0; j < KPT; ++j)
      if ((valid >> j) & 1u) {
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
  if (threadIdx.x < 2) {
    s_prefix[threadIdx.x] = 0;
    s_above[threadIdx.x] = 0;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NT / 32; ++i) {
    kmax = max(kmax, s_red[0][i]);
    kmin = min(kmin, s_red[1][i]);
  }
  if (kmin > kmax) kmin = kmax;  // no keys at all
  const int top = 32 - __clz(kmax - kmin);  // significant bits of t; 0 when all keys are equal
  if (chunks == 1) {
#pragma unroll
    for (int j = 0; j < KPT; ++j) key[j] = (valid >> j) & 1u ? kmax - key[j] : 0xffffffffu;
  }

  // radix select: when all bits of t are resolved, s_prefix[m] is the t of the want[m]-th largest key of modality m
  // (if that many exist) and s_above[m] counts the keys strictly above it. `rem` counts the bits not yet resolved.
  for (int rem = top; rem > 0;) {
    const int bits = min(rem, kDigitBits), shift = rem - bits;
    const uint32_t dmask = (1u << bits) - 1u;
    for (int x = threadIdx.x; x < 2 * kCntWords; x += NT) (&cnt[0][0])[x] = 0;
    __syncthreads();
    const uint32_t pre0 = s_prefix[0], pre1 = s_prefix[1];
    for (int c = 0; c < chunks; ++c) {
      if (chunks > 1) {
        load_chunk<kVec, kPool>(psi, mask, n, c * CHUNK + (int)threadIdx.x * KPT, p.mpa, wfrom, p.pool_r, key, valid, vis, forced);
#pragma unroll
        for (int j = 0; j < KPT; ++j) key[j] = (valid >> j) & 1u ? kmax - key[j] : 0xffffffffu;
      }
#pragma unroll
      for (int j = 0; j < KPT; ++j) {  // (a position outside the ranking holds all ones: no prefix equals its shifted t)
        const int m = (vis >> j) & 1u ? 0 : 1;
        if ((key[j] >> rem) == (m == 0 ? pre0 : pre1)) atomicAdd(&cnt[m][cnt_slot((key[j] >> shift) & dmask)], 1u);
      }
    }
    __syncthreads();
    if (warp < 2) {
      // warp m walks modality m's buckets in ascending digit order: a prefix scan of the lanes' totals tells which
      // lane holds the bucket that takes the running count to `want` (lane 31 if none does), and that lane alone
      // walks its buckets
      const int m = warp;
      const unsigned int want = (unsigned int)(m == 0 ? want0 : want1);
      unsigned int lc = 0;
#pragma unroll 8
      for (int i = 0; i < kPerLane; ++i) lc += cnt[m][cnt_slot(lane * kPerLane + i)];
      unsigned int sc = lc;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_up_sync(kFull, sc, off);
        if (lane >= off) sc += t;
      }
      unsigned int above = s_above[m] + (sc - lc);
      const unsigned int hit = __ballot_sync(kFull, above + lc >= want || lane == 31);
      if (lane == __ffs(hit) - 1) {
        int found = kPerLane - 1;
        for (int i = 0; i < kPerLane; ++i) {
          const unsigned int ci = cnt[m][cnt_slot(lane * kPerLane + i)];
          if (above + ci >= want || i == kPerLane - 1) {
            found = i;
            break;
          }
          above += ci;
        }
        // buckets beyond the pass's digit range are empty; landing there means "fewer keys than wanted"
        s_above[m] = above;
        s_prefix[m] = (s_prefix[m] << bits) | min((uint32_t)(lane * kPerLane + found), dmask);
      }
    }
    __syncthreads();
    rem = shift;
  }
  const uint32_t thr0 = s_prefix[0], thr1 = s_prefix[1];
  // ties at the threshold value that are still needed (all of them if the modality has fewer tokens than wanted)
  const int ties0 = max(want0 - (int)s_above[0], 0), ties1 = max(want1 - (int)s_above[1], 0);

  // ordered sweep: a thread's positions are consecutive, threads and chunks follow in position order
  int tie_run0 = 0, tie_run1 = 0;  // threshold-valued keys met in earlier chunks, per modality
  int out_run = 0;                 // kept positions emitted by earlier chunks
  for (int c = 0; c < chunks; ++c) {
    const int pos0 = c * CHUNK + (int)threadIdx.x * KPT;
    if (chunks > 1) {
      load_chunk<kVec, kPool>(psi, mask, n, pos0, p.mpa, wfrom, p.pool_r, key, valid, vis, forced);
#pragma unroll
      for (int j = 0; j < KPT; ++j) key[j] = (valid >> j) & 1u ? kmax - key[j] : 0xffffffffu;
    }
    uint32_t eq_bits = 0, gt_bits = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      const bool v = (vis >> j) & 1u;
      const uint32_t thr = v ? thr0 : thr1;
      // (thresholds are below 2^31; a position outside the ranking holds all ones and is neither equal nor smaller)
      if (key[j] == thr) eq_bits |= 1u << j;
      if (key[j] < thr && (v ? want0 : want1) > 0) gt_bits |= 1u << j;  // smaller t: larger importance
    }
    const uint32_t eq_pack = (uint32_t)__popc(eq_bits & vis) | ((uint32_t)__popc(eq_bits & ~vis) << 16);
    uint32_t eq_total;
    const uint32_t eq_before = block_excl_scan(eq_pack, warp_tot, &eq_total);
    // a threshold-valued key is kept while its rank among the modality's ties (in position order) is below ties[m]
    const int room0 = ties0 - (tie_run0 + (int)(eq_before & 0xffffu));
    const int room1 = ties1 - (tie_run1 + (int)(eq_before >> 16));
    uint32_t keep_bits = kPool ? (gt_bits | forced) : gt_bits;
    {
      uint32_t ev = eq_bits & vis, et = eq_bits & ~vis;
      for (int k = 0; k < room0 && ev && want0 > 0; ++k) {  // lowest positions first
        keep_bits |= ev & (0u - ev);
        ev &= ev - 1;
      }
      for (int k = 0; k < room1 && et && want1 > 0; ++k) {
        keep_bits |= et & (0u - et);
        et &= et - 1;
      }
    }
    uint32_t keep_total;
    const uint32_t slot = block_excl_scan((uint32_t)__popc(keep_bits), warp_tot, &keep_total);
    int o = out_run + (int)slot;
    while (keep_bits) {
      const int j = __ffs(keep_bits) - 1;
      keep_bits &= keep_bits - 1;
      p.kept_idx[off0 + o++] = pos0 + j;
    }
    tie_run0 += (int)(eq_total & 0xffffu);
    tie_run1 += (int)(eq_total >> 16);
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
  p.B = c.batch;
  p.L = c.n_layers;
  p.Hkv = c.n_kv_heads;
  p.n_max = c.max_seq_len;
  p.mpa = c.mpa;
  p.headroom = c.max_new_tokens;
  p.seq_nv = reinterpret_cast<int32_t*>((char*)ws + ws_layout(c).seq_nv_off);
  p.seq_wv = p.seq_nv + c.batch;
  p.keep_window = c.keep_window;
  p.window = c.window;
  p.pool_r = (c.pool_kernel - 1) / 2;
  seg_scan_kernel<<<1, 1024, 0, st>>>(p);
  // 16-byte loads of psi need every unit's row (n_max floats apart) to start on a 16-byte boundary
  const bool wide = c.max_seq_len > CHUNK;  // 10-bit digits when sequences can be longer than one chunk
  if (c.pool_kernel > 1 || c.keep_window) {
    if (wide) select_unit_kernel<false, true, 10><<<p.units, NT, 0, st>>>(p);
    else select_unit_kernel<false, true, 8><<<p.units, NT, 0, st>>>(p);
  } else if (c.max_seq_len % 4 == 0) {
    if (wide) select_unit_kernel<true, false, 10><<<p.units, NT, 0, st>>>(p);
    else select_unit_kernel<true, false, 8><<<p.units, NT, 0, st>>>(p);
  } else {
    if (wide) select_unit_kernel<false, false, 10><<<p.units, NT, 0, st>>>(p);
    else select_unit_kernel<false, false, 8><<<p.units, NT, 0, st>>>(p);
  }
  return launch_status();
}

}  // namespace madakv
