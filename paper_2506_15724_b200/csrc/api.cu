// C-ABI entry points: argument checks, then stage launchers. No entry point allocates or synchronises, except
// madakv_poll_status, which synchronises the stream to read the device status word.
#include "common.cuh"

using namespace madakv;

extern "C" {

int madakv_abi_version(void) { return 4; }

const char* madakv_status_string(int s) {
  switch (s) {
    case MADAKV_OK: return "ok";
    case MADAKV_EINVAL: return "invalid argument";
    case MADAKV_ESHAPE: return "bad shape";
    case MADAKV_EALIGN: return "misaligned pointer or stride";
    case MADAKV_EWORKSPACE: return "workspace too small";
    case MADAKV_ECAPACITY: return "ragged cache capacity exceeded";
    case MADAKV_EUNSUPPORTED: return "unsupported dtype, head_dim or window";
    case MADAKV_ECUDA: return "CUDA runtime error";
    case MADAKV_ETIMEOUT: return "bounded device wait expired";
    case MADAKV_ESTATIC: return "problem exceeds the built-in scratch of madakv_decode_attn_static";
    default: return "unknown status";
  }
}

int madakv_workspace_bytes(const madakv_config* cfg, size_t* bytes_out) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!bytes_out) return MADAKV_EINVAL;
  *bytes_out = ws_layout(*cfg).total;
  return MADAKV_OK;
}

int madakv_score(const madakv_config* cfg, const void* q_win, madakv_strides sq, const void* k, madakv_strides sk,
                 const int32_t* seq_len, float* lse, float* psi, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!q_win || !k || !seq_len || !psi) return MADAKV_EINVAL;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(psi) || ((uintptr_t)seq_len & 3) || ((uintptr_t)lse & 3))
    return MADAKV_EALIGN;
  if (!strides_ok(*cfg, sq) || !strides_ok(*cfg, sk)) return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_score(*cfg, q_win, sq, k, sk, seq_len, lse, psi, ws, (cudaStream_t)stream);
}

int madakv_score_lse(const madakv_config* cfg, const void* q_win, madakv_strides sq, const void* k, madakv_strides sk,
                     const int32_t* seq_len, const float* lse, float* psi, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!q_win || !k || !seq_len || !lse || !psi) return MADAKV_EINVAL;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(psi) || ((uintptr_t)seq_len & 3) || ((uintptr_t)lse & 3))
    return MADAKV_EALIGN;
  if (!strides_ok(*cfg, sq) || !strides_ok(*cfg, sk)) return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_score_lse(*cfg, q_win, sq, k, sk, seq_len, lse, psi, ws, (cudaStream_t)stream);
}

int madakv_allocate(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                    const int32_t* budget, double* mass, double* pref, int32_t* demand, double* phi, int32_t* budgets,
                    void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!psi || !mask || !seq_len || !budget || !mass || !pref || !demand || !phi || !budgets) return MADAKV_EINVAL;
  if (!aligned16(psi) || ((uintptr_t)mass & 7) || ((uintptr_t)pref & 7) || ((uintptr_t)phi & 7) ||
      ((uintptr_t)demand & 7) || ((uintptr_t)budgets & 7) || ((uintptr_t)seq_len & 3) || ((uintptr_t)budget & 3))
    return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_allocate(*cfg, psi, mask, seq_len, budget, mass, pref, demand, phi, budgets, ws, (cudaStream_t)stream);
}

int madakv_allocate_layer(const madakv_config* cfg, int32_t layer, const float* psi, const uint8_t* mask,
                          const int32_t* seq_len, const int32_t* budget, double* mass, double* pref, int32_t* demand,
                          double* phi, int32_t* budgets, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (layer < 0 || layer >= cfg->n_layers) return MADAKV_ESHAPE;
  // psi may be null: mass, pref and demand of the layer then come from madakv_demand_layer
  if (!mask || !seq_len || !budget || !mass || !pref || !demand || !phi || !budgets) return MADAKV_EINVAL;
  if (!aligned16(psi) || ((uintptr_t)mass & 7) || ((uintptr_t)pref & 7) || ((uintptr_t)phi & 7) ||
      ((uintptr_t)demand & 7) || ((uintptr_t)budgets & 7) || ((uintptr_t)seq_len & 3) || ((uintptr_t)budget & 3))
    return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_allocate_layer(*cfg, layer, psi, mask, seq_len, budget, mass, pref, demand, phi, budgets, ws,
                               (cudaStream_t)stream);
}

int madakv_demand_layer(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                        double* mass, double* pref, int32_t* demand, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!psi || !mask || !seq_len || !mass || !pref || !demand) return MADAKV_EINVAL;
  if (!aligned16(psi) || ((uintptr_t)mass & 7) || ((uintptr_t)pref & 7) || ((uintptr_t)demand & 7) ||
      ((uintptr_t)seq_len & 3))
    return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_demand_layer(*cfg, psi, mask, seq_len, mass, pref, demand, ws, (cudaStream_t)stream);
}

int madakv_select(const madakv_config* cfg, const float* psi, const uint8_t* mask, const int32_t* seq_len,
                  const int32_t* budgets, int32_t* kept_len, int64_t* seg_off, int32_t* kept_idx, int64_t capacity,
                  void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!psi || !mask || !seq_len || !budgets || !kept_len || !seg_off || !kept_idx) return MADAKV_EINVAL;
  if (capacity <= 0) return MADAKV_ECAPACITY;
  if (!aligned16(psi) || ((uintptr_t)budgets & 7) || ((uintptr_t)kept_len & 3) || ((uintptr_t)seg_off & 7) ||
      ((uintptr_t)kept_idx & 3) || ((uintptr_t)seq_len & 3))
    return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_select(*cfg, psi, mask, seq_len, budgets, kept_len, seg_off, kept_idx, capacity, ws,
                       (cudaStream_t)stream);
}

int madakv_compact(const madakv_config* cfg, const void* k, const void* v, madakv_strides skv, const int32_t* kept_idx,
                   const int64_t* seg_off, const int32_t* kept_len, void* k_c, void* v_c, int64_t capacity, void* ws,
                   size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!k || !v || !kept_idx || !seg_off || !kept_len || !k_c || !v_c) return MADAKV_EINVAL;
  if (capacity <= 0) return MADAKV_ECAPACITY;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_c) || !aligned16(v_c) || ((uintptr_t)kept_idx & 3) ||
      ((uintptr_t)seg_off & 7) || ((uintptr_t)kept_len & 3))
    return MADAKV_EALIGN;
  if (!strides_ok(*cfg, skv)) return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_compact(*cfg, k, v, skv, kept_idx, seg_off, kept_len, k_c, v_c, capacity, ws, (cudaStream_t)stream);
}

int madakv_decode_attn(const madakv_config* cfg, int32_t layer, const void* q, const void* k_new, const void* v_new,
                       void* k_c, void* v_c, const int64_t* seg_off, int32_t* kept_len, int64_t capacity, void* out,
                       float* lse_out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!q || !k_c || !v_c || !seg_off || !kept_len || !out) return MADAKV_EINVAL;
  if ((k_new == nullptr) != (v_new == nullptr)) return MADAKV_EINVAL;
  if (layer < -1 || layer >= cfg->n_layers) return MADAKV_ESHAPE;
  if (capacity <= 0) return MADAKV_ECAPACITY;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_c) || !aligned16(v_c) ||
      !aligned16(out) || ((uintptr_t)seg_off & 7) || ((uintptr_t)kept_len & 3) || ((uintptr_t)lse_out & 3))
    return MADAKV_EALIGN;
  if ((rc = check_ws(*cfg, ws, ws_bytes))) return rc;
  return launch_decode(*cfg, layer, q, k_new, v_new, k_c, v_c, seg_off, kept_len, capacity, out, lse_out, ws,
                       (cudaStream_t)stream);
}

int madakv_poll_status(void* ws, void* stream, int32_t* status_out) {
  if (!ws || !status_out) return MADAKV_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MADAKV_ECUDA;
  int32_t s = 0;
  if (cudaMemcpyAsync(&s, ws, sizeof(s), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MADAKV_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MADAKV_ECUDA;
  if (s != 0 && cudaMemsetAsync(ws, 0, sizeof(s), st) != cudaSuccess) return MADAKV_ECUDA;
  *status_out = s;
  return MADAKV_OK;
}

}  // extern "C"
