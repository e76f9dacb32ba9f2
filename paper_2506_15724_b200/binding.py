"""Thin ctypes binding of libmadakv.so: the same names as include/madakv.h, argument marshalling only.

Every step of the eviction pass runs in the library's CUDA kernels; PyTorch is used for device memory and streams.
There is no CPU fallback: importing this module without the built library, or calling it without a CUDA device,
raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmadakv.so")

MADAKV_F32, MADAKV_BF16 = 0, 1
HCC_OFF, HCC_PAPER, HCC_LITERAL, HCC_DEMAND = 0, 1, 2, 3
STATUS_NAMES = ["OK", "EINVAL", "ESHAPE", "EALIGN", "EWORKSPACE", "ECAPACITY", "EUNSUPPORTED", "ECUDA", "ETIMEOUT",
                "ESTATIC"]
(OK, EINVAL, ESHAPE, EALIGN, EWORKSPACE, ECAPACITY, EUNSUPPORTED, ECUDA, ETIMEOUT, ESTATIC) = range(10)
STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = [
    "madakv_abi_version", "madakv_status_string", "madakv_workspace_bytes", "madakv_score", "madakv_score_lse",
    "madakv_allocate", "madakv_allocate_layer", "madakv_demand_layer",
    "madakv_select", "madakv_compact", "madakv_decode_attn", "madakv_decode_attn_static", "madakv_poll_status",
]


class MadakvConfig(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("dtype", ctypes.c_int32), ("batch", ctypes.c_int32),
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("max_seq_len", ctypes.c_int32), ("window", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("mpa", ctypes.c_int32), ("hcc_mode", ctypes.c_int32),
        ("max_new_tokens", ctypes.c_int32), ("theta", ctypes.c_float), ("softmax_scale", ctypes.c_float),
        ("keep_window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
    ]


class MadakvStrides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int64), ("layer", ctypes.c_int64), ("head", ctypes.c_int64),
                ("token", ctypes.c_int64)]


class MadakvError(RuntimeError):
    def __init__(self, where, code):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where} failed: MADAKV_{name}")


_lib = None


def lib():
    """The loaded C-ABI library (loaded once). Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2506_15724_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        cfgp = ctypes.POINTER(MadakvConfig)
        L.madakv_abi_version.restype = ctypes.c_int
        L.madakv_status_string.restype = ctypes.c_char_p
        L.madakv_status_string.argtypes = [ctypes.c_int]
        L.madakv_workspace_bytes.argtypes = [cfgp, ctypes.POINTER(sz)]
        L.madakv_score.argtypes = [cfgp, vp, MadakvStrides, vp, MadakvStrides, vp, vp, vp, vp, sz, vp]
        L.madakv_score_lse.argtypes = [cfgp, vp, MadakvStrides, vp, MadakvStrides, vp, vp, vp, vp, sz, vp]
        L.madakv_allocate.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.madakv_allocate_layer.argtypes = [cfgp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.madakv_demand_layer.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.madakv_select.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
        L.madakv_compact.argtypes = [cfgp, vp, vp, MadakvStrides, vp, vp, vp, vp, vp, i64, vp, sz, vp]
        L.madakv_decode_attn.argtypes = [cfgp, i32, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp]
        L.madakv_decode_attn_static.argtypes = [cfgp, i32, vp, vp, vp, vp, vp, i64, vp, vp, vp]
        L.madakv_poll_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        for f in EXPORTS:
            if f not in ("madakv_status_string",):
                getattr(L, f).restype = ctypes.c_int
        _lib = L
    return _lib


def make_config(dtype, batch, n_layers, n_q_heads, n_kv_heads, head_dim, max_seq_len, window, causal=1, mpa=1,
                hcc_mode=HCC_PAPER, max_new_tokens=0, theta=0.5, softmax_scale=0.0, keep_window=0, pool_kernel=1):
    code = {torch.float32: MADAKV_F32, torch.bfloat16: MADAKV_BF16}.get(dtype, dtype)
    return MadakvConfig(ctypes.sizeof(MadakvConfig), code, batch, n_layers, n_q_heads, n_kv_heads, head_dim,
                        max_seq_len, window, causal, mpa, hcc_mode, max_new_tokens, theta, softmax_scale, keep_window,
                        pool_kernel)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _strides5(t):
    assert t.dim() == 5 and t.stride(4) == 1, "expected [B, L, H, tokens, d] with contiguous d"
    return MadakvStrides(t.stride(0), t.stride(1), t.stride(2), t.stride(3))


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(where, rc):
    if rc != 0:
        raise MadakvError(where, rc)


def madakv_workspace_bytes(cfg):
    out = ctypes.c_size_t(0)
    _check("madakv_workspace_bytes", lib().madakv_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)))
    return out.value


def new_workspace(cfg, device="cuda"):
    """A zeroed device workspace of the size the library asks for."""
    return torch.zeros(madakv_workspace_bytes(cfg), dtype=torch.uint8, device=device)


def madakv_score(cfg, q_win, k, seq_len, lse, psi, ws):
    _check("madakv_score", lib().madakv_score(ctypes.byref(cfg), _ptr(q_win), _strides5(q_win), _ptr(k), _strides5(k),
                                              _ptr(seq_len), _ptr(lse), _ptr(psi), _ptr(ws), ws.numel(), _stream()))


def madakv_score_lse(cfg, q_win, k, seq_len, lse, psi, ws):
    _check("madakv_score_lse", lib().madakv_score_lse(ctypes.byref(cfg), _ptr(q_win), _strides5(q_win), _ptr(k),
                                                      _strides5(k), _ptr(seq_len), _ptr(lse), _ptr(psi), _ptr(ws),
                                                      ws.numel(), _stream()))


def madakv_allocate(cfg, psi, mask, seq_len, budget, mass, pref, demand, phi, budgets, ws):
    _check("madakv_allocate", lib().madakv_allocate(ctypes.byref(cfg), _ptr(psi), _ptr(mask), _ptr(seq_len),
                                                    _ptr(budget), _ptr(mass), _ptr(pref), _ptr(demand), _ptr(phi),
                                                    _ptr(budgets), _ptr(ws), ws.numel(), _stream()))


def madakv_demand_layer(cfg, psi, mask, seq_len, mass, pref, demand, ws):
    _check("madakv_demand_layer", lib().madakv_demand_layer(ctypes.byref(cfg), _ptr(psi), _ptr(mask), _ptr(seq_len),
                                                            _ptr(mass), _ptr(pref), _ptr(demand), _ptr(ws), ws.numel(),
                                                            _stream()))


def madakv_allocate_layer(cfg, layer, psi, mask, seq_len, budget, mass, pref, demand, phi, budgets, ws):
    """psi may be None: mass, pref and demand then come from madakv_demand_layer."""
    _check("madakv_allocate_layer", lib().madakv_allocate_layer(ctypes.byref(cfg), int(layer), _ptr(psi), _ptr(mask),
                                                                _ptr(seq_len), _ptr(budget), _ptr(mass), _ptr(pref),
                                                                _ptr(demand), _ptr(phi), _ptr(budgets), _ptr(ws),
                                                                ws.numel(), _stream()))


def madakv_select(cfg, psi, mask, seq_len, budgets, kept_len, seg_off, kept_idx, ws):
    _check("madakv_select", lib().madakv_select(ctypes.byref(cfg), _ptr(psi), _ptr(mask), _ptr(seq_len), _ptr(budgets),
                                                _ptr(kept_len), _ptr(seg_off), _ptr(kept_idx), kept_idx.numel(),
                                                _ptr(ws), ws.numel(), _stream()))


def madakv_compact(cfg, k, v, kept_idx, seg_off, kept_len, k_c, v_c, ws):
    assert k.stride() == v.stride()
    _check("madakv_compact", lib().madakv_compact(ctypes.byref(cfg), _ptr(k), _ptr(v), _strides5(k), _ptr(kept_idx),
                                                  _ptr(seg_off), _ptr(kept_len), _ptr(k_c), _ptr(v_c), k_c.shape[0],
                                                  _ptr(ws), ws.numel(), _stream()))


def madakv_decode_attn(cfg, layer, q, k_new, v_new, k_c, v_c, seg_off, kept_len, out, lse_out, ws):
    _check("madakv_decode_attn", lib().madakv_decode_attn(ctypes.byref(cfg), layer, _ptr(q), _ptr(k_new), _ptr(v_new),
                                                          _ptr(k_c), _ptr(v_c), _ptr(seg_off), _ptr(kept_len),
                                                          k_c.shape[0], _ptr(out), _ptr(lse_out), _ptr(ws),
                                                          ws.numel(), _stream()))


def madakv_decode_attn_static(cfg, layer, q, k_c, v_c, seg_off, kept_len, out, lse_out):
    """Decode attention without a workspace: the library's built-in scratch is used, nothing is allocated. For
    callers that may not allocate device memory; calls must not overlap on the GPU (they share the scratch)."""
    _check("madakv_decode_attn_static", lib().madakv_decode_attn_static(ctypes.byref(cfg), layer, _ptr(q), _ptr(k_c),
                                                                        _ptr(v_c), _ptr(seg_off), _ptr(kept_len),
                                                                        k_c.shape[0], _ptr(out), _ptr(lse_out),
                                                                        _stream()))


def madakv_poll_status(ws):
    out = ctypes.c_int32(0)
    _check("madakv_poll_status", lib().madakv_poll_status(_ptr(ws), _stream(), ctypes.byref(out)))
    return out.value


def madakv_status_string(code):
    return lib().madakv_status_string(code).decode()


class EvictionBuffers:
    """Device tensors the five calls write (allocated once through torch; no arithmetic here)."""

    def __init__(self, cfg, capacity_rows, device="cuda", want_lse=False):
        B, L, Hq, Hkv = cfg.batch, cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads
        d, n = cfg.head_dim, cfg.max_seq_len
        units = B * L * Hkv
        dt = torch.float32 if cfg.dtype == MADAKV_F32 else torch.bfloat16
        z = lambda shape, dtype: torch.zeros(shape, dtype=dtype, device=device)  # noqa: E731
        self.cfg = cfg
        self.ws = new_workspace(cfg, device)
        self.psi = z((B, L, Hkv, n), torch.float32)
        self.lse = z((B, L, Hq, cfg.window), torch.float32) if want_lse else None
        self.mass = z((B, L, Hkv, 2), torch.float64)
        self.pref = z((B, L, Hkv, 2), torch.float64)
        self.demand = z((B, L, Hkv, 2), torch.int32)
        self.phi = z((B, L), torch.float64)
        self.budgets = z((B, L, Hkv, 2), torch.int32)
        self.kept_len = z((units,), torch.int32)
        self.seg_off = z((units + 1,), torch.int64)
        self.kept_idx = torch.full((capacity_rows,), -1, dtype=torch.int32, device=device)
        self.k_c = z((capacity_rows, d), dt)
        self.v_c = z((capacity_rows, d), dt)
        self.out = z((B, L, Hq, d), dt)
        self.lse_dec = z((B, L, Hq), torch.float32)

    def run_eviction(self, q_win, k, v, mask, seq_len, budget):
        """Stages 1-4, enqueued on the current stream."""
        c = self.cfg
        madakv_score(c, q_win, k, seq_len, self.lse, self.psi, self.ws)
        madakv_allocate(c, self.psi, mask, seq_len, budget, self.mass, self.pref, self.demand, self.phi, self.budgets,
                        self.ws)
        madakv_select(c, self.psi, mask, seq_len, self.budgets, self.kept_len, self.seg_off, self.kept_idx, self.ws)
        madakv_compact(c, k, v, self.kept_idx, self.seg_off, self.kept_len, self.k_c, self.v_c, self.ws)

    def run_decode(self, q, k_new=None, v_new=None, layer=-1):
        madakv_decode_attn(self.cfg, layer, q, k_new, v_new, self.k_c, self.v_c, self.seg_off, self.kept_len, self.out,
                           self.lse_dec, self.ws)
