"""Shared plumbing of the GPU parity tests: tensor <-> numpy conversion and stage-by-stage comparison."""
import numpy as np
import torch

import oracle
from paper_2506_15724_b200 import binding as mk


def to_np(t):
    """torch tensor -> numpy array the oracle accepts (bf16 as uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def dcode(wl):
    return 0 if wl.dtype == "f32" else 1


def config_of(wl, **kw):
    args = dict(dtype=wl.torch_dtype, batch=wl.B, n_layers=wl.L, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.d,
                max_seq_len=wl.n, window=wl.w, max_new_tokens=wl.max_new_tokens, theta=wl.theta)
    args.update(kw)
    return mk.make_config(**args)


def capacity_of(wl, per_unit=None):
    per_unit = wl.n if per_unit is None else per_unit
    return wl.units * (min(per_unit, wl.n) + wl.max_new_tokens)


def psi_close(got, want, rtol, atol=1e-9):
    """Relative agreement of importance scores; returns the worst relative error for reporting."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    err = np.abs(got - want)
    ok = err <= rtol * np.abs(want) + atol
    assert ok.all(), f"psi mismatch: worst abs {err.max():.3e}, {np.count_nonzero(~ok)} bad"
    denom = np.maximum(np.abs(want), 1e-30)
    return float((err / denom)[np.abs(want) > 1e-6].max(initial=0.0))


def oracle_stages_from(wl, cfg, psi32, mask, seq_len, budget, k, v):
    """Oracle stages 2-4 run on a given fp32 psi (numpy inputs). Returns dict of numpy results."""
    al = oracle.allocate(psi32, mask, seq_len, budget, float(np.float32(cfg.theta)), mpa=cfg.mpa, hcc_mode=cfg.hcc_mode)
    cap = capacity_of(wl)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi32, mask, seq_len, al["budgets"], mpa=cfg.mpa,
                                                    headroom=cfg.max_new_tokens, capacity=cap)
    assert rc == 0
    k_c, v_c = oracle.compact(dcode(wl), k, v, kept_idx, seg_off, kept_len, cap)
    al.update(kept_len=kept_len, seg_off=seg_off, kept_idx=kept_idx, k_c=k_c, v_c=v_c, capacity=cap)
    return al


def assert_segments_equal(kept_len, seg_off, got, want, what):
    """Compare ragged arrays on the rows that belong to segments (headroom rows are unspecified)."""
    for u in range(kept_len.shape[0]):
        a, b = int(seg_off[u]), int(seg_off[u]) + int(kept_len[u])
        assert np.array_equal(got[a:b], want[a:b]), f"{what}: unit {u} differs"
