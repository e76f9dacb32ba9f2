"""ctypes front end of the C++ oracle (``madakv_oracle.cpp``): TEST INFRASTRUCTURE, not product code.

Arrays are numpy, dense, in the layouts the C++ file documents. bf16 tensors are passed as ``uint16`` bit patterns
(``dtype=1``), fp32 as ``float32`` (``dtype=0``). Every function returns new arrays; nothing here depends on the
CUDA library.
"""
import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "madakv_oracle.cpp")
_LIB = os.path.join(_HERE, "libmadakv_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with g++ (no fast-math, no FMA contraction) and return the path of the library."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread", "-o", _LIB, _SRC]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.mo_topp_count_f64.restype = ctypes.c_int32
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a)
    assert a.dtype == dt, (a.dtype, dt)
    return a


def _elem(dtype):
    return np.float32 if dtype == 0 else np.uint16


def hardware_threads():
    return int(_load().mo_hardware_threads())


def score(dtype, q_win, k, seq_len, causal=1, scale=None, threads=0, want_lse=False):
    """Eq. 7. q_win [B,L,Hq,w,d], k [B,L,Hkv,n_max,d] -> psi [B,L,Hkv,n_max] float64 (and lse [B,L,Hq,w])."""
    q_win, k = _c(q_win, _elem(dtype)), _c(k, _elem(dtype))
    B, L, Hq, w, d = q_win.shape
    Hkv, n_max = k.shape[2], k.shape[3]
    seq_len = _c(seq_len, np.int32)
    psi = np.zeros((B, L, Hkv, n_max), np.float64)
    lse = np.zeros((B, L, Hq, w), np.float64) if want_lse else None
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    rc = _load().mo_score(dtype, B, L, Hq, Hkv, d, n_max, w, int(causal), ctypes.c_double(scale), _p(q_win), _p(k),
                          _p(seq_len), _p(psi), _p(lse), threads)
    assert rc == 0, rc
    return (psi, lse) if want_lse else psi


def allocate(psi, mask, seq_len, budget, theta, mpa=1, hcc_mode=1, keep_window=0, window=0, threads=0):
    """Eq. 6, 8, 9, 10, 11. psi [B,L,Hkv,n_max] float32 -> dict(mass, pref, demand, phi, budgets).
    keep_window (with the window size): budgets floored at the proxy tokens' counts per modality."""
    psi = _c(psi, np.float32)
    B, L, Hkv, n_max = psi.shape
    mask, seq_len, budget = _c(mask, np.uint8), _c(seq_len, np.int32), _c(budget, np.int32)
    out = dict(
        mass=np.zeros((B, L, Hkv, 2), np.float64),
        pref=np.zeros((B, L, Hkv, 2), np.float64),
        demand=np.zeros((B, L, Hkv, 2), np.int32),
        phi=np.zeros((B, L), np.float64),
        budgets=np.zeros((B, L, Hkv, 2), np.int32),
    )
    rc = _load().mo_allocate(B, L, Hkv, n_max, _p(psi), _p(mask), _p(seq_len), _p(budget), ctypes.c_float(theta),
                             int(mpa), int(hcc_mode), int(keep_window), int(window), _p(out["mass"]), _p(out["pref"]),
                             _p(out["demand"]), _p(out["phi"]), _p(out["budgets"]), threads)
    assert rc == 0, rc
    return out


def select(psi, mask, seq_len, budgets, mpa=1, headroom=0, capacity=None, keep_window=0, window=0, pool_kernel=1):
    """Stage 4a. Returns (rc, kept_len [units], seg_off [units+1], kept_idx [capacity]); rc 5 = capacity exceeded.
    pool_kernel (odd): rank by the maximum of psi over that many positions; keep_window: the last `window` positions
    of every sequence are always kept."""
    assert pool_kernel >= 1 and pool_kernel % 2 == 1
    psi = _c(psi, np.float32)
    B, L, Hkv, n_max = psi.shape
    units = B * L * Hkv
    budgets = _c(budgets, np.int32)
    if capacity is None:
        capacity = int(budgets.reshape(units, 2).sum()) + units * (headroom + (window if keep_window else 0))
    kept_len = np.zeros(units, np.int32)
    seg_off = np.zeros(units + 1, np.int64)
    kept_idx = np.full(max(capacity, 1), -1, np.int32)
    rc = _load().mo_select(B, L, Hkv, n_max, _p(psi), _p(_c(mask, np.uint8)), _p(_c(seq_len, np.int32)), _p(budgets),
                           int(mpa), int(headroom), int(keep_window), int(window), int(pool_kernel), _p(kept_len),
                           _p(seg_off), _p(kept_idx), ctypes.c_int64(capacity))
    return rc, kept_len, seg_off, kept_idx


def compact(dtype, k, v, kept_idx, seg_off, kept_len, capacity):
    """Stage 4b. k, v [B,L,Hkv,n_max,d] -> k_c, v_c [capacity, d] (zero where no row was written)."""
    k, v = _c(k, _elem(dtype)), _c(v, _elem(dtype))
    B, L, Hkv, n_max, d = k.shape
    k_c = np.zeros((capacity, d), _elem(dtype))
    v_c = np.zeros((capacity, d), _elem(dtype))
    rc = _load().mo_compact(k.itemsize, B, L, Hkv, d, n_max, _p(k), _p(v), _p(_c(kept_idx, np.int32)),
                            _p(_c(seg_off, np.int64)), _p(_c(kept_len, np.int32)), _p(k_c), _p(v_c))
    assert rc == 0, rc
    return k_c, v_c


def decode(dtype, q, k_new, v_new, k_c, v_c, seg_off, kept_len, Hkv, layer=-1, scale=None, threads=0):
    """Stage 5 (Eq. 4-5). q [B,L,Hq,d]; k_c, v_c, kept_len are updated IN PLACE when k_new is given.
    Returns (rc, out [B,L,Hq,d] float64, lse [B,L,Hq] float64)."""
    q = _c(q, _elem(dtype))
    B, L, Hq, d = q.shape
    assert k_c.flags.c_contiguous and v_c.flags.c_contiguous and kept_len.dtype == np.int32
    if k_new is not None:
        k_new, v_new = _c(k_new, _elem(dtype)), _c(v_new, _elem(dtype))
    out = np.zeros((B, L, Hq, d), np.float64)
    lse = np.zeros((B, L, Hq), np.float64)
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    rc = _load().mo_decode(dtype, B, L, Hq, Hkv, d, ctypes.c_double(scale), int(layer), _p(q), _p(k_new), _p(v_new),
                           _p(k_c), _p(v_c), _p(_c(seg_off, np.int64)), _p(kept_len), _p(out), _p(lse), threads)
    return rc, out, lse


def topp_count_f64(psi, theta):
    psi = _c(psi, np.float64)
    return int(_load().mo_topp_count_f64(_p(psi), int(psi.size), ctypes.c_double(theta)))
