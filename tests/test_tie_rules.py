"""The tie rules of the end-to-end comparison (tests/helpers.compare_with_pure_oracle), checked on the CPU with the
oracle alone: results computed from the oracle's own scores pass with no tie counted; results computed from scores
perturbed in the last bits pass only where the rule allows it; a planted mistake (a wrong kept position, a wrong
budget, a demand off by one away from the threshold) is rejected."""
import numpy as np
import pytest

import oracle
from paper_2506_15724_b200 import binding as bc
from paper_2506_15724_b200 import synth
from helpers import compare_with_pure_oracle, to_np


def _case():
    wl = synth.scaled(synth.CONFIGS["tiny"], B=2, L=3, Hq=4, Hkv=2, n=389, w=8, budget=40, theta=0.3)
    inp = synth.make_inputs(wl, want_v=False)
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    psi = oracle.score(0, to_np(inp["q_win"]), to_np(inp["k"]), sl)
    cfg = bc.make_config(0, wl.B, wl.L, wl.Hq, wl.Hkv, wl.d, wl.n, wl.w, max_new_tokens=wl.max_new_tokens,
                         theta=wl.theta)
    return wl, cfg, psi, mask, sl, bud


def _pipeline(cfg, psi32, mask, sl, bud):
    al = oracle.allocate(psi32, mask, sl, bud, float(np.float32(cfg.theta)))
    rc, kept_len, seg_off, kept_idx = oracle.select(psi32, mask, sl, al["budgets"], headroom=cfg.max_new_tokens)
    assert rc == 0
    return dict(demand=al["demand"], phi=al["phi"], budgets=al["budgets"], kept_len=kept_len, seg_off=seg_off,
                kept_idx=kept_idx)


def test_identical_results_use_no_tie_rule():
    wl, cfg, psi, mask, sl, bud = _case()
    got = _pipeline(cfg, psi.astype(np.float32), mask, sl, bud)
    stats, agreed, _ = compare_with_pure_oracle(wl, cfg, psi, got, mask, sl, bud)
    assert agreed.all()
    assert all(stats[k] == 0 for k in ("demand_ties", "budget_rounding_ties", "kept_ties", "units_after_a_demand_tie"))


def test_a_swap_at_the_last_kept_score_passes_only_within_the_tie_window():
    wl, cfg, psi, mask, sl, bud = _case()
    psi32 = psi.astype(np.float32)
    got = _pipeline(cfg, psi32, mask, sl, bud)
    u = 3
    b = u // (wl.L * wl.Hkv)
    a0, a1 = int(got["seg_off"][u]), int(got["seg_off"][u]) + int(got["kept_len"][u])
    kept = got["kept_idx"][a0:a1]
    pu = psi32.reshape(wl.units, wl.n)[u]
    text_kept = kept[mask[b, kept] == 0]
    last = text_kept[np.argmin(pu[text_kept])]  # the lowest-scoring kept text position
    cand = np.setdiff1d(np.nonzero(mask[b, : sl[b]] == 0)[0], kept)
    runner_up = cand[np.argmax(pu[cand])]  # the best evicted text position
    swapped = np.sort(np.concatenate([kept[kept != last], [runner_up]])).astype(np.int32)
    bad = {k: v.copy() for k, v in got.items()}
    bad["kept_idx"][a0:a1] = swapped
    # the two scores differ by far more than 1e-5 relative on random data: rejected
    assert abs(pu[runner_up] - pu[last]) > 1e-4 * pu[last]
    with pytest.raises(AssertionError):
        compare_with_pure_oracle(wl, cfg, psi, bad, mask, sl, bud)
    # with the runner-up's score moved to within 1e-6 relative of the last kept score the same swap is a tie
    psi_tied = psi.copy()
    psi_tied.reshape(wl.units, wl.n)[u, runner_up] = float(pu[last]) * (1.0 - 1e-6)
    base = _pipeline(cfg, psi_tied.astype(np.float32), mask, sl, bud)
    b0, b1 = int(base["seg_off"][u]), int(base["seg_off"][u]) + int(base["kept_len"][u])
    kept = base["kept_idx"][b0:b1]  # (the moved score may have changed the budgets a little: take the sets anew)
    assert last in kept and runner_up not in kept
    tied = {k: v.copy() for k, v in base.items()}
    tied["kept_idx"][b0:b1] = np.sort(np.concatenate([kept[kept != last], [runner_up]])).astype(np.int32)
    stats, agreed, _ = compare_with_pure_oracle(wl, cfg, psi_tied, tied, mask, sl, bud)
    assert stats["kept_ties"] == 2 and stats["units_with_kept_ties"] == 1 and not agreed[u]


def test_planted_mistakes_in_budgets_and_demands_are_rejected():
    wl, cfg, psi, mask, sl, bud = _case()
    got = _pipeline(cfg, psi.astype(np.float32), mask, sl, bud)
    bad = {k: v.copy() for k, v in got.items()}
    bad["demand"][0, 1, 0, 1] += 1  # Eq. 9 off by one, nowhere near the threshold
    with pytest.raises(AssertionError):
        compare_with_pure_oracle(wl, cfg, psi, bad, mask, sl, bud)
    bad = {k: v.copy() for k, v in got.items()}
    bad["budgets"][1, 0, 1] += np.array([1, -1], np.int32)  # Eq. 8 split moved by one token, no rounding boundary near
    with pytest.raises(AssertionError):
        compare_with_pure_oracle(wl, cfg, psi, bad, mask, sl, bud)
    bad = {k: v.copy() for k, v in got.items()}
    bad["phi"][0, 2] += 0.25  # Eq. 11 wrong
    with pytest.raises(AssertionError):
        compare_with_pure_oracle(wl, cfg, psi, bad, mask, sl, bud)
