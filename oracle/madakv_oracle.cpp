// madakv_oracle.cpp — TEST INFRASTRUCTURE, not product code.
//
// A plain, slow CPU restatement of the MadaKV eviction pass (arXiv 2506.15724, Section 3), written from the
// paper's equations and used only to check the CUDA library and as the timed CPU baseline. It shares no code,
// header, table or constant generator with the CUDA path. Floating point is fp64 throughout; inputs are the
// stored fp32 / bf16 bits. No blocking, fusion or reordering beyond what the equations state; the only
// parallelism is a thread per independent (sequence, layer, KV head) unit.
//
// Parity status of each function:
//   mo_score     Eq. 7 + softmax of Eq. 5          pinned (closed forms, textbook softmax, worked 16-token case)
//   mo_allocate  Eq. 6, 8, 9, 10, 11                pinned piecewise (subset brute force, closed-form scalars,
//                                                   worked case); the way Eq. 8 and Eq. 10-11 are composed where
//                                                   the paper's units disagree is a stated reading: parity unpinned
//   mo_select    top-budget per modality            pinned (full-sort brute force, worked case); score pooling and
//                                                   forced retention of the window are readings of this build, not
//                                                   of the paper (it defines neither): parity unpinned by the paper,
//                                                   pinned against a library maximum filter and worked cases
//   mo_compact   row gather                         pinned (definition)
//   mo_decode    Eq. 4 + Eq. 5                      pinned (library attention, worked case)
//
// Layouts are dense: q_win [B,L,Hq,w,d], k/v [B,L,Hkv,n_max,d], psi [B,L,Hkv,n_max], mask [B,n_max].
// unit u = (b*L + l)*Hkv + h. Modality index 0 = visual (mask 1), 1 = text (mask 0).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

typedef unsigned __int128 u128;

inline double load_elem(const void* base, int dtype, int64_t idx) {
  if (dtype == 0) return (double)((const float*)base)[idx];
  uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;  // bf16 = upper half of an fp32
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

template <class F>
void for_units(int64_t n_units, int threads, F f) {
  int hw = (int)std::thread::hardware_concurrency();
  if (threads <= 0) threads = hw > 0 ? hw : 1;
  if ((int64_t)threads > n_units) threads = (int)std::max<int64_t>(1, n_units);
  if (threads == 1) {
    for (int64_t u = 0; u < n_units; ++u) f(u);
    return;
  }
  std::vector<std::thread> pool;
  for (int t = 0; t < threads; ++t)
    pool.emplace_back([=]() {
      for (int64_t u = t; u < n_units; u += threads) f(u);
    });
  for (auto& th : pool) th.join();
}

// Fixed-point image of an importance value: floor(x * 2^32) for x > 0, else 0 (NaN counts as 0).
inline uint64_t fix32(float x) {
  if (!(x > 0.0f)) return 0;
  return (uint64_t)((double)x * 4294967296.0);
}

// Sort key "psi descending, position ascending".
struct Cand {
  float psi;
  int32_t pos;
};
inline bool before(const Cand& a, const Cand& b) {
  float pa = a.psi > 0.0f ? a.psi : 0.0f, pb = b.psi > 0.0f ? b.psi : 0.0f;
  if (pa != pb) return pa > pb;
  return a.pos < b.pos;
}

}  // namespace

extern "C" {

int mo_hardware_threads() { return (int)std::thread::hardware_concurrency(); }

// Eq. 7: psi(i) = sum_{j in P} alpha_{j->i}, alpha = softmax over keys of scale * q_j . k_i (Eq. 5), summed over
// the g query heads that share KV head h. Window row r is the query at position n - w + r.
// lse (may be null) receives log sum_i exp(s_{r,i}) per query head and row; rows at negative positions get -inf.
int mo_score(int dtype, int B, int L, int Hq, int Hkv, int d, int n_max, int w, int causal, double scale,
             const void* q_win, const void* k, const int32_t* seq_len, double* psi, double* lse, int threads) {
  if (Hkv <= 0 || Hq % Hkv) return 1;
  const int g = Hq / Hkv;
  for_units((int64_t)B * L * Hkv, threads, [=](int64_t u) {
    const int h = (int)(u % Hkv), l = (int)((u / Hkv) % L), b = (int)(u / ((int64_t)Hkv * L));
    const int n = seq_len[b];
    double* out = psi + u * n_max;
    for (int i = 0; i < n_max; ++i) out[i] = 0.0;
    std::vector<double> s(n > 0 ? n : 1), kd((size_t)(n > 0 ? n : 1) * d);
    const int64_t kbase = u * (int64_t)n_max * d;
    for (int64_t x = 0; x < (int64_t)n * d; ++x) kd[x] = load_elem(k, dtype, kbase + x);
    for (int qh = h * g; qh < (h + 1) * g; ++qh) {
      for (int r = 0; r < w; ++r) {
        const int pos = n - w + r;
        const int64_t row = (((int64_t)b * L + l) * Hq + qh) * w + r;
        if (pos < 0) {
          if (lse) lse[row] = -std::numeric_limits<double>::infinity();
          continue;
        }
        const int visible = causal ? pos + 1 : n;
        std::vector<double> qd(d);
        for (int c = 0; c < d; ++c) qd[c] = load_elem(q_win, dtype, row * d + c);
        double m = -std::numeric_limits<double>::infinity();
        for (int i = 0; i < visible; ++i) {
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += qd[c] * kd[(int64_t)i * d + c];
          s[i] = scale * acc;
          m = std::max(m, s[i]);
        }
        double z = 0.0;
        for (int i = 0; i < visible; ++i) z += std::exp(s[i] - m);
        for (int i = 0; i < visible; ++i) out[i] += std::exp(s[i] - m) / z;
        if (lse) lse[row] = m + std::log(z);
      }
    }
  });
  return 0;
}

// Eq. 9 for one modality, exactly as a minimum over subsets can be evaluated: take candidates in descending psi
// and stop at the first prefix whose mass reaches theta * total. Fixed-point masses, 128-bit comparison
//   prefix * 2^32 >= floor(theta * 2^32) * total.
static int32_t topp_count(std::vector<Cand>& c, float theta) {
  std::sort(c.begin(), c.end(), before);
  u128 total = 0;
  for (auto& e : c) total += fix32(e.psi);
  double th = theta < 0.0f ? 0.0 : (theta > 1.0f ? 1.0 : (double)theta);
  const uint64_t theta_fix = (uint64_t)(th * 4294967296.0);
  const u128 need = (u128)theta_fix * total;
  if (need == 0) return 0;
  u128 prefix = 0;
  for (size_t j = 0; j < c.size(); ++j) {
    prefix += fix32(c[j].psi);
    if ((prefix << 32) >= need) return (int32_t)(j + 1);
  }
  return (int32_t)c.size();
}

// The same count with fp64 sums and comparison (used by the tests to show the fixed-point rule is the fp64 rule
// away from exact threshold hits).
int32_t mo_topp_count_f64(const double* psi, int n, double theta) {
  std::vector<double> v(psi, psi + n);
  std::sort(v.begin(), v.end(), [](double a, double b) { return a > b; });
  double total = 0.0;
  for (double x : v) total += x;
  if (!(theta * total > 0.0)) return 0;
  double prefix = 0.0;
  for (int j = 0; j < n; ++j) {
    prefix += v[j];
    if (prefix >= theta * total) return j + 1;
  }
  return n;
}

// Stages 2-3. Eq. 6 (masses), Eq. 8 (ratio and, after the layer recurrence, integer budgets), Eq. 9 (demand),
// Eq. 10-11 (layer compensation). hcc_mode: 0 off, 1 divide by H*(L-l), 2 divide by (L-l) as printed, 3 as 1 with
// every layer but the last keeping what Eq. 9 asks for (then Eq. 11 is "what is left over the layers left" and the
// last layer, budgeted by Eq. 8, spends the remainder: the total stays L*H*phi^1).
// keep_window (not in the paper): the proxy tokens (the last min(window, n) positions) are always retained, so a
// head's budgets are floored at the window's token counts per modality: with lo_v, lo_t those counts and
// P' = max(Phi^l, lo_v + lo_t), the visual budget of Eq. 8 is brought into [lo_v, P' - lo_t] and the text budget is
// P' minus it. Masses, preferences, Eq. 9 and Eq. 10-11 are untouched.
int mo_allocate(int B, int L, int Hkv, int n_max, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                const int32_t* budget, float theta, int mpa, int hcc_mode, int keep_window, int window, double* mass,
                double* pref, int32_t* demand, double* phi, int32_t* budgets, int threads) {
  const int64_t units = (int64_t)B * L * Hkv;
  for_units(units, threads, [=](int64_t u) {
    const int b = (int)(u / ((int64_t)Hkv * L));
    const int n = seq_len[b];
    const float* p = psi + u * n_max;
    const uint8_t* mk = mask + (int64_t)b * n_max;
    std::vector<Cand> cv, ct;
    uint64_t W[2] = {0, 0};
    for (int i = 0; i < n; ++i) {
      const int m = mk[i] ? 0 : 1;
      W[m] += fix32(p[i]);  // Eq. 6
      (m == 0 ? cv : ct).push_back(Cand{p[i], i});
    }
    mass[u * 2 + 0] = (double)W[0] / 4294967296.0;
    mass[u * 2 + 1] = (double)W[1] / 4294967296.0;
    const uint64_t tot = W[0] + W[1];
    pref[u * 2 + 0] = tot ? (double)W[0] / (double)tot : 0.0;  // Eq. 8: w_v / (w_v + w_t)
    pref[u * 2 + 1] = tot ? (double)W[1] / (double)tot : 0.0;
    demand[u * 2 + 0] = topp_count(cv, theta);  // Eq. 9
    demand[u * 2 + 1] = topp_count(ct, theta);
  });
  for (int b = 0; b < B; ++b) {
    const int n = seq_len[b];
    int n_v = 0;
    for (int i = 0; i < n; ++i) n_v += mask[(int64_t)b * n_max + i] ? 1 : 0;
    const int n_t = n - n_v;
    int lo_v = 0, lo_t = 0;  // window tokens per modality (forced retention), 0 without keep_window
    if (keep_window)
      for (int i = std::max(0, n - window); i < n; ++i) (mask[(int64_t)b * n_max + i] ? lo_v : lo_t) += 1;
    const double lo = n >= 1 ? 1.0 : 0.0, hi = (double)n;
    double ph = (double)budget[b];  // phi^1
    for (int l = 1; l <= L; ++l) {
      phi[(int64_t)b * L + (l - 1)] = ph;
      double Phi = std::floor(ph + 0.5);
      Phi = std::min(std::max(Phi, lo), hi);
      int64_t dem = 0;
      for (int h = 0; h < Hkv; ++h) {
        const int64_t u = ((int64_t)b * L + (l - 1)) * Hkv + h;
        dem += (int64_t)demand[u * 2] + demand[u * 2 + 1];
        int32_t bv, bt;
        const int32_t P = std::max((int32_t)Phi, lo_v + lo_t);
        if (mpa) {
          bv = (int32_t)std::floor(pref[u * 2] * Phi + 0.5);  // Eq. 8, rounded half up
          bv = std::min(std::max(bv, lo_v), P - lo_t);         // forced retention of the window (no-op without it)
          bt = P - bv;
          if (bv > n_v) { bt += bv - n_v; bv = n_v; }
          if (bt > n_t) { bv = std::min(n_v, bv + (bt - n_t)); bt = n_t; }
        } else {
          bv = 0;
          bt = std::min(P, n);
        }
        if (hcc_mode == 3 && l < L) {  // the layer keeps its demand (k_m <= n_m by construction)
          bv = mpa ? std::max(demand[u * 2], lo_v) : 0;
          bt = mpa ? std::max(demand[u * 2 + 1], lo_t)
                   : std::min(std::max(demand[u * 2] + demand[u * 2 + 1], lo_v + lo_t), n);
        }
        budgets[u * 2] = bv;
        budgets[u * 2 + 1] = bt;
      }
      if (l < L) {
        const double K = (double)dem - (double)Hkv * ph;  // Eq. 10
        double next = ph;
        if (hcc_mode == 1 || hcc_mode == 3) next = ph - K / (double)((int64_t)Hkv * (L - l));  // Eq. 11, per-head units
        if (hcc_mode == 2) next = ph - K / (double)(L - l);                    // Eq. 11 as printed
        ph = std::min(std::max(next, lo), hi);
      }
    }
  }
  return 0;
}

// Stage 4a: keep, of each modality, the budgeted number of highest-scoring tokens; list them by position.
// Two options the paper does not have (both off by default):
//   pool_kernel p (odd): tokens are ranked by the maximum of psi over the p positions centred on them (positions
//     outside the sequence do not count) instead of psi itself: a token next to a strongly attended one is kept with
//     it. Only the ranking uses the pooled score.
//   keep_window: the last min(window, n) positions are kept whatever their score; they count towards their
//     modality's budget, and a budget smaller than their number is raised to it.
// Returns 5 if a segment would not fit into `capacity` rows (that segment and all later ones are not written).
int mo_select(int B, int L, int Hkv, int n_max, const float* psi, const uint8_t* mask, const int32_t* seq_len,
              const int32_t* budgets, int mpa, int headroom, int keep_window, int window, int pool_kernel,
              int32_t* kept_len, int64_t* seg_off, int32_t* kept_idx, int64_t capacity) {
  const int64_t units = (int64_t)B * L * Hkv;
  int64_t off = 0;
  for (int64_t u = 0; u < units; ++u) {
    const int b = (int)(u / ((int64_t)Hkv * L));
    const int n = seq_len[b];
    const float* p = psi + u * n_max;
    const uint8_t* mk = mask + (int64_t)b * n_max;
    const int r = (pool_kernel - 1) / 2;
    std::vector<Cand> c[2];  // candidates by score
    std::vector<int32_t> keep;
    int forced[2] = {0, 0}, count[2] = {0, 0};
    for (int i = 0; i < n; ++i) {
      const int m = (mpa && mk[i]) ? 0 : 1;
      count[m] += 1;
      if (keep_window && i >= n - window) {  // a proxy token: kept unconditionally
        keep.push_back(i);
        forced[m] += 1;
        continue;
      }
      float pooled = p[i];
      for (int j = std::max(0, i - r); j <= std::min(n - 1, i + r); ++j) pooled = std::max(pooled, p[j]);
      c[m].push_back(Cand{pooled, i});
    }
    for (int m = 0; m < 2; ++m) {
      std::sort(c[m].begin(), c[m].end(), before);
      const int want = std::min<int>(std::max<int>(budgets[u * 2 + m], forced[m]), count[m]);
      for (int j = 0; j < want - forced[m]; ++j) keep.push_back(c[m][j].pos);
    }
    std::sort(keep.begin(), keep.end());
    seg_off[u] = off;
    kept_len[u] = (int32_t)keep.size();
    if (off + (int64_t)keep.size() + headroom > capacity) return 5;
    for (size_t j = 0; j < keep.size(); ++j) kept_idx[off + (int64_t)j] = keep[j];
    off += (int64_t)keep.size() + headroom;
  }
  seg_off[units] = off;
  return 0;
}

// Stage 4b: bit copies of the kept rows.
int mo_compact(int elem_bytes, int B, int L, int Hkv, int d, int n_max, const void* k, const void* v,
               const int32_t* kept_idx, const int64_t* seg_off, const int32_t* kept_len, void* k_c, void* v_c) {
  const int64_t units = (int64_t)B * L * Hkv;
  const size_t row = (size_t)d * elem_bytes;
  for (int64_t u = 0; u < units; ++u)
    for (int j = 0; j < kept_len[u]; ++j) {
      const int64_t src = (u * n_max + kept_idx[seg_off[u] + j]) * (int64_t)row;
      const int64_t dst = (seg_off[u] + j) * (int64_t)row;
      std::memcpy((char*)k_c + dst, (const char*)k + src, row);
      std::memcpy((char*)v_c + dst, (const char*)v + src, row);
    }
  return 0;
}

// Stage 5: Eq. 4 (append one row per KV head when k_new is given) and Eq. 5 over each segment.
// layer = -1 runs every layer. out [B,L,Hq,d] fp64, lse [B,L,Hq] fp64 or null. Returns 5 when an append
// does not fit (segment left unchanged).
int mo_decode(int dtype, int B, int L, int Hq, int Hkv, int d, double scale, int layer, const void* q,
              const void* k_new, const void* v_new, void* k_c, void* v_c, const int64_t* seg_off,
              int32_t* kept_len, double* out, double* lse, int threads) {
  const int g = Hq / Hkv;
  const size_t eb = dtype == 0 ? 4 : 2;
  std::vector<int> rcs((size_t)B * L * Hkv, 0);
  int* rcp = rcs.data();
  for_units((int64_t)B * L * Hkv, threads, [=](int64_t u) {
    const int h = (int)(u % Hkv), l = (int)((u / Hkv) % L), b = (int)(u / ((int64_t)Hkv * L));
    if (layer >= 0 && l != layer) return;
    if (k_new) {
      if (seg_off[u] + kept_len[u] + 1 > seg_off[u + 1]) {
        rcp[u] = 5;
      } else {
        const int64_t dst = (seg_off[u] + kept_len[u]) * (int64_t)d * eb;
        std::memcpy((char*)k_c + dst, (const char*)k_new + u * (int64_t)d * eb, d * eb);  // Eq. 4
        std::memcpy((char*)v_c + dst, (const char*)v_new + u * (int64_t)d * eb, d * eb);
        kept_len[u] += 1;
      }
    }
    const int len = kept_len[u];
    std::vector<double> s(len > 0 ? len : 1), p(len > 0 ? len : 1), qd(d);
    for (int qh = h * g; qh < (h + 1) * g; ++qh) {
      const int64_t row = ((int64_t)b * L + l) * Hq + qh;
      for (int c = 0; c < d; ++c) qd[c] = load_elem(q, dtype, row * d + c);
      double m = -std::numeric_limits<double>::infinity();
      for (int j = 0; j < len; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += qd[c] * load_elem(k_c, dtype, (seg_off[u] + j) * d + c);
        s[j] = scale * acc;
        m = std::max(m, s[j]);
      }
      double z = 0.0;
      for (int j = 0; j < len; ++j) z += std::exp(s[j] - m);
      for (int j = 0; j < len; ++j) p[j] = std::exp(s[j] - m) / z;  // softmax weights of Eq. 5
      for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int j = 0; j < len; ++j) acc += p[j] * load_elem(v_c, dtype, (seg_off[u] + j) * d + c);
        out[row * d + c] = len > 0 ? acc : 0.0;
      }
      if (lse) lse[row] = len > 0 ? m + std::log(z) : -std::numeric_limits<double>::infinity();
    }
  });
  int rc = 0;
  for (int x : rcs) rc = x ? x : rc;
  return rc;
}

}  // extern "C"
