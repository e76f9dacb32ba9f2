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
    al = oracle.allocate(psi32, mask, seq_len, budget, float(np.float32(cfg.theta)), mpa=cfg.mpa, hcc_mode=cfg.hcc_mode,
                         keep_window=cfg.keep_window, window=cfg.window)
    cap = capacity_of(wl)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi32, mask, seq_len, al["budgets"], mpa=cfg.mpa,
                                                    headroom=cfg.max_new_tokens, capacity=cap,
                                                    keep_window=cfg.keep_window, window=cfg.window,
                                                    pool_kernel=cfg.pool_kernel)
    assert rc == 0
    k_c, v_c = oracle.compact(dcode(wl), k, v, kept_idx, seg_off, kept_len, cap)
    al.update(kept_len=kept_len, seg_off=seg_off, kept_idx=kept_idx, k_c=k_c, v_c=v_c, capacity=cap)
    return al


def assert_segments_equal(kept_len, seg_off, got, want, what):
    """Compare ragged arrays on the rows that belong to segments (headroom rows are unspecified)."""
    for u in range(kept_len.shape[0]):
        a, b = int(seg_off[u]), int(seg_off[u]) + int(kept_len[u])
        assert np.array_equal(got[a:b], want[a:b]), f"{what}: unit {u} differs"


def _fix32(x):
    """floor(x * 2^32) of fp32 scores as Python-exact uint64 (the fixed-point image both sides sum, Eq. 6 / Eq. 9)."""
    x = np.asarray(x, np.float32)
    return np.where(x > 0, np.floor(x.astype(np.float64) * 4294967296.0), 0.0).astype(np.uint64)


def eq9_prefix_is_at_threshold(psi_m, theta, count, rtol=1e-5):
    """True if the mass of the `count` largest scores of one modality lies within rtol (relative) of theta * total:
    the one situation in which two correct evaluations of Eq. 9 on scores that differ in the last bits may disagree."""
    f = np.sort(_fix32(psi_m))[::-1]
    total = int(f.sum(dtype=np.uint64))
    need = int(np.float64(np.float32(theta)) * 4294967296.0) * total  # scaled by 2^32, as the prefix below
    pre = int(f[:count].sum(dtype=np.uint64)) << 32
    return abs(pre - need) <= rtol * need


def compare_with_pure_oracle(wl, cfg, want_psi, got, mask, seq_len, budget, tie_rtol=1e-5):
    """The CUDA pipeline's results `got` (numpy: demand, phi, budgets, kept_len, seg_off, kept_idx) against the
    pure-oracle pipeline on the oracle's own scores `want_psi` (float64 [B,L,Hkv,n]).

    Integer results must be identical except where the scores are tied within `tie_rtol`:
      - a demand (Eq. 9) may differ only if the prefix mass at that count is within tie_rtol of theta * W_m; from the
        first such layer of a sequence on, phi (Eq. 11) and with it the budgets of the later layers may differ;
      - with equal Phi^l a budget (Eq. 8) may differ only if pref_v * Phi^l is within tie_rtol (relative) of a rounding
        boundary (x.5);
      - given the budgets the CUDA path arrived at, its kept set may differ from the oracle's selection on the oracle's
        scores only in positions whose score is within tie_rtol (relative) of the last kept score of that modality.
    Nothing is skipped silently: the returned dict counts every use of a tie rule."""
    psi32 = np.ascontiguousarray(want_psi, np.float32)
    theta = float(np.float32(cfg.theta))
    assert cfg.keep_window == 0 and cfg.pool_kernel == 1, "the tie rules are written for the paper-literal selection"
    pure = oracle.allocate(psi32, mask, seq_len, budget, theta, mpa=cfg.mpa, hcc_mode=cfg.hcc_mode)
    B, L, H, n = psi32.shape
    stats = dict(units=B * L * H, demand_ties=0, budget_rounding_ties=0, units_after_a_demand_tie=0, kept_ties=0,
                 units_with_kept_ties=0)
    diverged_at = np.full(B, L, np.int64)  # first layer of the sequence with a tied demand
    dd = np.argwhere(pure["demand"] != got["demand"])
    for b, l, h, m in dd.tolist():
        sel = (mask[b, : seq_len[b]] != 0) if m == 0 else (mask[b, : seq_len[b]] == 0)
        if not cfg.mpa:
            sel = np.ones(seq_len[b], bool)
        c = int(min(pure["demand"][b, l, h, m], got["demand"][b, l, h, m]))
        assert abs(int(pure["demand"][b, l, h, m]) - int(got["demand"][b, l, h, m])) == 1, (b, l, h, m)
        assert eq9_prefix_is_at_threshold(psi32[b, l, h, : seq_len[b]][sel], theta, c, tie_rtol), \
            f"Eq. 9 count differs away from the threshold: unit {(b, l, h)}, modality {m}"
        stats["demand_ties"] += 1
        diverged_at[b] = min(diverged_at[b], l)
    for b in range(B):
        upto = min(L, int(diverged_at[b]) + 1)  # phi^1 .. phi^{l*} are functions of identical demands
        assert np.array_equal(pure["phi"][b, :upto], got["phi"][b, :upto]), f"phi of sequence {b}"
        stats["units_after_a_demand_tie"] += (L - upto) * H
        for l in range(upto):
            for h in range(H):
                if np.array_equal(pure["budgets"][b, l, h], got["budgets"][b, l, h]):
                    continue
                Phi = min(max(np.floor(pure["phi"][b, l] + 0.5), 1.0), float(seq_len[b]))
                x = pure["pref"][b, l, h, 0] * Phi
                assert abs(x - np.floor(x) - 0.5) <= tie_rtol * max(x, 1.0), f"budget of unit {(b, l, h)}"
                assert np.abs(pure["budgets"][b, l, h] - got["budgets"][b, l, h]).max() == 1
                stats["budget_rounding_ties"] += 1
    # selection on the oracle's scores with the budgets the CUDA path used
    cap = int(got["seg_off"][-1])
    rc, kept_len, seg_off, kept_idx = oracle.select(psi32, mask, seq_len, got["budgets"], mpa=cfg.mpa,
                                                    headroom=cfg.max_new_tokens, capacity=max(cap, 1))
    assert rc == 0
    assert np.array_equal(kept_len, got["kept_len"]) and np.array_equal(seg_off, got["seg_off"])
    psi_u = psi32.reshape(B * L * H, n)
    agreed = np.ones(B * L * H, bool)
    for u in range(B * L * H):
        a0, a1 = int(seg_off[u]), int(seg_off[u]) + int(kept_len[u])
        want_set, got_set = kept_idx[a0:a1], got["kept_idx"][a0:a1]
        if np.array_equal(want_set, got_set):
            continue
        agreed[u] = False
        b = u // (L * H)
        diff = np.setxor1d(want_set, got_set)
        assert np.all(np.diff(got_set) > 0), f"kept positions of unit {u} are not ascending"
        for i in diff.tolist():
            m = mask[b, i] if cfg.mpa else 0
            same = want_set[(mask[b, want_set] == m)] if cfg.mpa else want_set
            kth = float(psi_u[u, same].min())
            assert abs(float(psi_u[u, i]) - kth) <= tie_rtol * kth, f"unit {u}: position {i} is no tie of the last kept score"
        stats["kept_ties"] += int(diff.size)
        stats["units_with_kept_ties"] += 1
    return stats, agreed, pure
