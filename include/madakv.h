/*
 * madakv.h — C ABI of the MadaKV prefill-to-decode KV-cache eviction pass for NVIDIA B200 (sm_100a).
 *
 * The pass follows arXiv 2506.15724 (MadaKV), Section 3:
 *   stage 1  madakv_score        importance psi(i) of every cached key under the proxy-token window   (Eq. 7, scale of Eq. 5)
 *   stage 2  madakv_allocate     modality preference w_v, w_t and per-head modality budgets            (Eq. 6, Eq. 8)
 *   stage 3  madakv_allocate     sparsity counts k_v, k_t, layer compensation K^l and phi^{l+1}        (Eq. 9, Eq. 10, Eq. 11)
 *   stage 4  madakv_select       per-head, per-modality eviction: keep the budgeted top-psi tokens     (Section 3.3, text after Eq. 8)
 *            madakv_compact      gather the kept K/V rows into a ragged per-head cache
 *   stage 5  madakv_decode_attn  cache append and decode attention over the ragged cache                (Eq. 4, Eq. 5)
 *
 * General rules for every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller (the only host pointers are `cfg` and the
 *     `size_t* / int32_t*` result arguments of madakv_workspace_bytes / madakv_poll_status). The library allocates no
 *     device memory, keeps no state between calls other than what lives in the caller's buffers, and only
 *     enqueues work on `stream`.
 *   - Return value: MADAKV_OK or a host-detected error (null or misaligned pointer, bad shape, unsupported
 *     dtype/head_dim, workspace or capacity too small). Host-detected errors are raised before any kernel launch.
 *   - Conditions only the device can see (a ragged segment that would overflow its capacity, a bounded wait that
 *     expired) set a status word at the head of the workspace; the offending write is skipped, never performed out
 *     of bounds. madakv_poll_status reads that word (it is the only call that synchronises the stream).
 *   - Layouts: the innermost dimension (head_dim) is contiguous; all other strides are passed in ELEMENTS through
 *     madakv_strides. Every row (head_dim elements) must start on a 16-byte boundary.
 *   - Notation: B sequences, L layers, H_q query heads, H_kv KV heads, g = H_q / H_kv, d = head_dim, n_max =
 *     max_seq_len, w = window. A "unit" is one (sequence b, layer l, KV head h); its flat index is
 *     u = (b * L + l) * H_kv + h. Modality index 0 = visual, 1 = text.
 */
#ifndef MADAKV_H_
#define MADAKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum madakv_status {
  MADAKV_OK = 0,
  MADAKV_EINVAL = 1,       /* null pointer, bad struct_size, bad flag value                         */
  MADAKV_ESHAPE = 2,       /* non-positive or inconsistent dimension, H_q not a multiple of H_kv     */
  MADAKV_EALIGN = 3,       /* a pointer or stride breaks the 16-byte row alignment rule              */
  MADAKV_EWORKSPACE = 4,   /* workspace smaller than madakv_workspace_bytes reports                   */
  MADAKV_ECAPACITY = 5,    /* ragged cache capacity exceeded (host- or device-detected)              */
  MADAKV_EUNSUPPORTED = 6, /* dtype / head_dim / window*g outside the supported set                  */
  MADAKV_ECUDA = 7,        /* a CUDA runtime call failed (launch configuration, missing sm_100 device) */
  MADAKV_ETIMEOUT = 8,     /* device-detected: a bounded wait inside a kernel ran out                */
  MADAKV_ESTATIC = 9       /* madakv_decode_attn_static only: the problem needs more than its built-in scratch */
} madakv_status;

enum { MADAKV_F32 = 0, MADAKV_BF16 = 1 };

/* Layer-compensation modes (Eq. 10-11). phi^l is a per-head token budget; H below means KV heads.
 *   OFF      phi^l = phi^1 for every layer (ablation "without HCC", Table 3)
 *   PAPER    phi^{l+1} = phi^l - K^l / (H * (L - l)); the factor H reconciles Eq. 8 (phi^l per head) with Eq. 10
 *            (K^l summed over heads)
 *   LITERAL  phi^{l+1} = phi^l - K^l / (L - l), Eq. 11 exactly as printed
 *   DEMAND   phi as in PAPER, but every layer except the last keeps what Eq. 9 asks for (budgets = demand) instead
 *            of Eq. 8's split of phi^l. K^l is then what the layer overspent, Eq. 11 reads "what is left, over the
 *            layers left", and the last layer (Eq. 8 at phi^L) spends the remainder: the total over all layers
 *            stays L * H * phi^1 up to rounding and the clamps. One reading of "exceeded its budget" under Eq. 10. */
enum { MADAKV_HCC_OFF = 0, MADAKV_HCC_PAPER = 1, MADAKV_HCC_LITERAL = 2, MADAKV_HCC_DEMAND = 3 };

typedef struct madakv_config {
  uint32_t struct_size;     /* sizeof(madakv_config), checked                                            */
  int32_t dtype;            /* MADAKV_F32 or MADAKV_BF16: element type of q, K, V, the ragged cache, out   */
  int32_t batch;            /* B                                                                          */
  int32_t n_layers;         /* L                                                                          */
  int32_t n_q_heads;        /* H_q                                                                        */
  int32_t n_kv_heads;       /* H_kv, divides H_q                                                          */
  int32_t head_dim;         /* d, 64 or 128                                                               */
  int32_t max_seq_len;      /* n_max: row count of the token dimension of K, V, psi, mask                  */
  int32_t window;           /* w = |P|, the proxy tokens are the last w prompt positions (Section 3.3)     */
  int32_t causal;           /* 1: window query at position p sees keys 0..p; 0: every window query sees all */
  int32_t mpa;              /* 1: Eq. 8 modality split; 0: one budget per head, modality ignored (Table 3) */
  int32_t hcc_mode;         /* MADAKV_HCC_*                                                               */
  int32_t max_new_tokens;   /* rows of headroom left after every ragged segment for Eq. 4 appends          */
  float theta;              /* threshold of Eq. 9, 0 <= theta <= 1                                        */
  float softmax_scale;      /* 0 means 1/sqrt(head_dim) (Eq. 5)                                           */
  /* Two options of the selection step that the paper does not have (it defines no pooling and says nothing about
   * retaining the proxy tokens); both are off in the paper-literal setting 0 / 1.                                 */
  int32_t keep_window;      /* 1: the proxy tokens (the last min(w, seq_len) positions) are always kept; budgets
                               are floored at their number per modality (madakv_allocate, madakv_select)          */
  int32_t pool_kernel;      /* odd, 1..15. p > 1: stage 4a ranks tokens by the maximum of psi over the p positions
                               centred on them (inside the sequence) instead of psi itself. 1 = no pooling        */
} madakv_config;

/* Strides in elements of a [B, L, H, tokens, d] tensor; d is contiguous. */
typedef struct madakv_strides {
  int64_t batch, layer, head, token;
} madakv_strides;

/* Bytes of caller-provided scratch every other call expects in `ws` (a device buffer, 256-byte aligned).
 * The first 256 bytes hold the device status word and counters; the caller zeroes the buffer once after
 * allocating it (cudaMemsetAsync) and may then reuse it across calls on one stream. Two calls that run
 * concurrently on different streams need separate workspaces.                                             */
int madakv_workspace_bytes(const madakv_config* cfg, size_t* bytes_out);

/* Stage 1 (Eq. 7 with the softmax of Eq. 5). For unit (b,l,h) and key i < seq_len[b]:
 *   psi[u][i] = sum over the g query heads of the KV group and over window rows r of
 *               softmax_i( scale * q_win[b,l,hq,r,:] . k[b,l,h,i,:] )
 * Window row r stands at absolute position seq_len[b] - w + r; rows with a negative position are skipped; with
 * cfg->causal the row sees keys 0..position. psi[u][i] = 0 for i >= seq_len[b]. Accumulation is fp32.
 *   q_win   [B, L, H_q, w, d]  dtype, strides sq
 *   k       [B, L, H_kv, n_max, d] dtype, strides sk
 *   seq_len [B] int32, 0 <= seq_len[b] <= n_max (device data: a value outside the range is used as the nearest
 *           bound, in every call that takes seq_len)
 *   lse     [B, L, H_q, w] fp32, natural-log sum-exp of every window row's scaled logits. The call computes
 *           these values and stores them here when `lse` is non-null (may be null).
 *   psi     [B, L, H_kv, n_max] fp32, contiguous, written in full
 * Deterministic: a fixed reduction order, no floating-point atomics.
 * The scoring kernels are persistent grids sized to the whole device. One of them (bf16, g * w <= 64, sequences too
 * long for a thread-block cluster's tensor memory) lets a CTA wait, bounded, for results of other CTAs of the same
 * launch: give this call the device to itself. If kernels of another stream keep part of its grid from being
 * scheduled, the wait runs out and the call reports MADAKV_ETIMEOUT through the status word instead of scores
 * (nothing hangs, the workspace stays usable).                                                              */
int madakv_score(const madakv_config* cfg, const void* q_win, madakv_strides sq, const void* k, madakv_strides sk,
                 const int32_t* seq_len, float* lse, float* psi, void* ws, size_t ws_bytes, void* stream);

/* Stage 1 in a single pass (Eq. 7), for callers that already hold the softmax normalisers: the attention of the
 * prompt's last w queries was computed during prefill (Eq. 5), and its log-sum-exp per row is what a fused attention
 * kernel keeps anyway. Same arguments and result as madakv_score, except that
 *   lse     [B, L, H_q, w] fp32 is an INPUT: the natural-log sum-exp of every window row's scaled logits over the
 *           keys the row sees (what madakv_score stores in its `lse`); -inf for a row that sees no key.
 * psi[u][i] = sum over the group's heads and window rows of exp( scale * q.k_i - lse ). K is read once and nothing
 * is reduced over keys, so the result is only as good as the normalisers supplied. Layer by layer use: pass a
 * config with n_layers = 1 and pointers to that layer's slices.                                             */
int madakv_score_lse(const madakv_config* cfg, const void* q_win, madakv_strides sq, const void* k, madakv_strides sk,
                     const int32_t* seq_len, const float* lse, float* psi, void* ws, size_t ws_bytes, void* stream);

/* Stages 2-3 (Eq. 6, 8, 9, 10, 11). All sums of psi are taken exactly, in 2^-32 fixed point:
 *   Q(x) = floor(x * 2^32) for x > 0, else 0;   W_m = sum_{i in X_m} Q(psi[u][i])                 (Eq. 6)
 *   pref[u][m] = W_m / (W_v + W_t)  (0 if the denominator is 0)                                    (Eq. 8 ratio)
 *   demand[u][m] = smallest c such that the c largest Q of modality m sum to >= theta * W_m,
 *                  0 when theta * W_m = 0                                                          (Eq. 9)
 *   per sequence, l = 1..L (fp64): Phi^l = clamp(floor(phi^l + 1/2), 1, n);
 *                  K^l = sum_h (k_v + k_t) - H * phi^l;                                             (Eq. 10)
 *                  phi^{l+1} per cfg->hcc_mode, clamped to [1, n];  phi^1 = budget[b]               (Eq. 11)
 *   budgets[u][0] = floor(pref_v * Phi^l + 1/2), budgets[u][1] = Phi^l - budgets[u][0]; a modality with fewer
 *                  tokens than its share passes the surplus to the other one (both capped by their token counts).
 *                  With cfg->mpa = 0: budgets[u] = {0, min(Phi^l, n)}.
 *                  With cfg->keep_window: lo_v, lo_t = visual / text tokens among the last min(w, n) positions,
 *                  P' = max(Phi^l, lo_v + lo_t); the visual budget above is first brought into [lo_v, P' - lo_t] and
 *                  the text budget is P' minus it (mpa = 0: {0, min(P', n)}). Nothing else changes.
 *   psi [B,L,H_kv,n_max] fp32; mask [B,n_max] uint8 (1 = visual token); seq_len [B]; budget [B] int32 >= 1
 *   mass, pref [B,L,H_kv,2] fp64 (mass = W_m / 2^32); demand, budgets [B,L,H_kv,2] int32; phi [B,L] fp64      */
int madakv_allocate(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                    const int32_t* budget, double* mass, double* pref, int32_t* demand, double* phi, int32_t* budgets,
                    void* ws, size_t ws_bytes, void* stream);

/* Stages 2-3 for ONE layer of a layer-by-layer pass (the order Section 3.3 implies: a layer is evicted right after
 * its prefill and the budget state goes on to the next layer, Eq. 11). cfg->n_layers = L is the real depth and
 * `layer` in [0, L) the layer at hand; the per-layer arrays hold that layer only:
 *   psi [B,H_kv,n_max]; mass, pref [B,H_kv,2] fp64; demand, budgets [B,H_kv,2] int32
 *   phi [B,L] fp64 is the state carried between calls: layer 0 sets phi[b][0] = budget[b]; every call reads
 *   phi[b][layer] and, when layer + 1 < L, writes phi[b][layer + 1]  (Eq. 10-11).
 * Called for layer = 0 .. L-1 in order it produces exactly the phi, mass, pref, demand and budgets that
 * madakv_allocate produces for the stacked arrays. For stages 1 and 4 of such a pass give madakv_score_lse (or
 * madakv_score), madakv_select and madakv_compact a config with n_layers = 1 and that layer's slices.        */
int madakv_allocate_layer(const madakv_config* cfg, int32_t layer, const float* psi, const uint8_t* mask,
                          const int32_t* seq_len, const int32_t* budget, double* mass, double* pref, int32_t* demand,
                          double* phi, int32_t* budgets, void* ws, size_t ws_bytes, void* stream);

/* The part of madakv_allocate_layer that does not depend on the budget state: mass, pref and demand of one layer
 * (Eq. 6, the ratio of Eq. 8, Eq. 9) from that layer's psi. Only Eq. 10-11 chain the layers together, so a caller
 * that keeps several layers in flight runs this call for layer l + 1 while layer l is still being allocated, and
 * then calls madakv_allocate_layer with psi = NULL, which takes mass, pref and demand as given and does the rest
 * (Phi^l, phi^{l+1}, budgets). The two calls together write exactly what madakv_allocate_layer alone writes.
 *   psi [B,H_kv,n_max]; mass, pref [B,H_kv,2] fp64; demand [B,H_kv,2] int32 (cfg as for madakv_allocate_layer)   */
int madakv_demand_layer(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                        double* mass, double* pref, int32_t* demand, void* ws, size_t ws_bytes, void* stream);

/* Stage 4a (Section 3.3: modality-specific eviction for each head). For every unit keep, of each modality m,
 * the budgets[u][m] tokens with the largest psi (equal psi: the lower position wins) and list the kept positions
 * in ascending order:
 *   kept_len[u] = budgets[u][0] + budgets[u][1]
 *   seg_off[u]  = sum_{u' < u} (kept_len[u'] + cfg->max_new_tokens), seg_off has B*L*H_kv + 1 entries (rows)
 *   kept_idx[seg_off[u] + j], j < kept_len[u]: the j-th kept position
 * With cfg->mpa = 0 the mask is ignored and budgets[u][1] positions are kept. A segment that would end beyond
 * `capacity` rows is not written and sets MADAKV_ECAPACITY in the status word.
 * Options outside the paper: with cfg->pool_kernel = p > 1 "largest psi" reads "largest max of psi over positions
 * i - (p-1)/2 .. i + (p-1)/2 inside the sequence" (only this ranking uses the pooled value). With cfg->keep_window
 * the last min(w, seq_len) positions are kept whatever their score; they count towards their modality's budget, a
 * budget smaller than their number acts as that number, and kept_len counts accordingly.                     */
int madakv_select(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                  const int32_t* budgets, int32_t* kept_len, int64_t* seg_off, int32_t* kept_idx, int64_t capacity,
                  void* ws, size_t ws_bytes, void* stream);

/* Stage 4b: k_c[seg_off[u] + j, :] = k[b,l,h, kept_idx[seg_off[u] + j], :] and the same for v (bit copies).
 *   k, v [B,L,H_kv,n_max,d] dtype with strides skv; k_c, v_c [capacity, d] dtype, contiguous.             */
int madakv_compact(const madakv_config* cfg, const void* k, const void* v, madakv_strides skv, const int32_t* kept_idx,
                   const int64_t* seg_off, const int32_t* kept_len, void* k_c, void* v_c, int64_t capacity,
                   void* ws, size_t ws_bytes, void* stream);

/* Stage 5 (Eq. 4-5). For every unit of layer `layer` (all layers when layer = -1):
 *   if k_new is non-null: row kept_len[u] of the segment := k_new[b,l,h,:] / v_new[b,l,h,:], kept_len[u] += 1
 *                         (a full segment is left unchanged and sets MADAKV_ECAPACITY)              (Eq. 4)
 *   out[b,l,hq,:] = softmax( scale * q[b,l,hq,:] . K_seg^T ) V_seg for the g query heads of the group (Eq. 5)
 *   q, out [B,L,H_q,d] dtype contiguous; k_new, v_new [B,L,H_kv,d] dtype contiguous or both null;
 *   lse_out [B,L,H_q] fp32 or null. An empty segment gives out = 0, lse = -inf.
 * Accumulation is fp32; out is rounded to dtype once. With bf16 and 3 <= g <= 16 the products run on the tensor
 * cores and the softmax weights enter the P V product rounded to bf16 (the denominator stays fp32).
 * Supported: g <= 8 for fp32, g <= 16 for bf16; beyond that MADAKV_EUNSUPPORTED.                           */
int madakv_decode_attn(const madakv_config* cfg, int32_t layer, const void* q, const void* k_new, const void* v_new,
                       void* k_c, void* v_c, const int64_t* seg_off, int32_t* kept_len, int64_t capacity, void* out,
                       float* lse_out, void* ws, size_t ws_bytes, void* stream);

/* Decode attention for callers that cannot allocate device memory. (No counterpart in the paper: this is the
 * attention of Eq. 5 exactly as madakv_decode_attn computes it, packaged for a different kind of caller.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits, for example a plug-in called in the middle of an
 * inference engine's step, whose memory pool is owned by the host application, or a real-time loop in which an
 * allocation (which may synchronise the whole device) would break the latency budget. Such a caller has buffers
 * for its inputs and outputs but nowhere to put the split partials the attention kernels exchange, and
 * madakv_decode_attn asks for a workspace. This variant keeps those partials in a fixed array that is part of the
 * library image: MADAKV_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library, held until the
 * process exits. It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Arguments are those of madakv_decode_attn without k_new / v_new (no append, kept_len is only read), without the
 * workspace, and with read-only caches. Same layouts, same result bits as madakv_decode_attn on the same inputs.
 *   - Limit: B * L * H_q * ceil((n_max + max_new_tokens) / 256) * (d + 2) * 4 bytes must not exceed
 *     MADAKV_STATIC_SCRATCH_BYTES; a larger problem returns MADAKV_ESTATIC before anything is launched.
 *   - The first call on each device looks up the device address of the built-in array (a host-side query, no
 *     allocation) with that device current; make that first call outside any stream capture.
 *   - All calls on one device share the one array. Nothing in it has to start at zero (every partial that is read
 *     was written earlier in the same call), but two calls whose kernels overlap on the GPU (different streams, or
 *     different host threads) race on it: serialise them.                                                  */
#define MADAKV_STATIC_SCRATCH_BYTES (16u << 20)
int madakv_decode_attn_static(const madakv_config* cfg, int32_t layer, const void* q, const void* k_c, const void* v_c,
                              const int64_t* seg_off, const int32_t* kept_len, int64_t capacity, void* out,
                              float* lse_out, void* stream);

/* Synchronises `stream`, copies the device status word (a madakv_status) to *status_out and clears it. */
int madakv_poll_status(void* ws, void* stream, int32_t* status_out);

const char* madakv_status_string(int status);

/* Library version, bumped when the ABI changes. 2: madakv_score_lse, madakv_allocate_layer and MADAKV_HCC_DEMAND added
 * (nothing that version 1 had was changed). 3: madakv_config grew by keep_window and pool_kernel (struct_size is
 * checked: a caller built against version 2 gets MADAKV_EINVAL, not a misread struct). 4: madakv_demand_layer
 * added, madakv_allocate_layer accepts psi = NULL (nothing that version 3 had was changed). */
int madakv_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MADAKV_H_ */
