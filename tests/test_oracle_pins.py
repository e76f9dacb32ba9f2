"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA library).

Each oracle function is checked against something other than itself: a case worked by hand from the paper's
equations (tests/golden), closed forms, invariants, a library attention routine, or brute force on tiny inputs.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _hand():
    with open(os.path.join(GOLDEN, "handworked_16.json")) as f:
        return json.load(f)


def _hand_inputs(h):
    a = np.array(h["a"], np.float64)
    q = np.zeros((1, 1, 1, 2, 64), np.float32)
    q[..., 0] = 8.0
    k = np.zeros((1, 1, 1, 16, 64), np.float32)
    k[0, 0, 0, :, 0] = np.log(a).astype(np.float32)
    v = np.zeros((1, 1, 1, 16, 64), np.float32)
    v[0, 0, 0, :, 0] = np.arange(16)
    return q, k, v, np.array([h["mask"]], np.uint8), np.array([16], np.int32)


# ---------------------------------------------------------------- stage 1: Eq. 7


def test_score_handworked_case():
    h = _hand()
    q, k, _, _, sl = _hand_inputs(h)
    psi = oracle.score(0, q, k, sl, causal=1, scale=1 / 8)
    np.testing.assert_allclose(psi[0, 0, 0] * 160, h["psi_times_160_causal"], rtol=1e-6)
    psi = oracle.score(0, q, k, sl, causal=0, scale=1 / 8)
    np.testing.assert_allclose(psi[0, 0, 0] * 20, h["psi_times_20_noncausal"], rtol=1e-6)


@pytest.mark.parametrize("g", [1, 3])
def test_score_identical_keys_closed_form(g):
    # all keys equal => every visible key gets 1/(pos+1) from the window row at position pos
    B, L, Hkv, n, w, d = 1, 2, 2, 37, 5, 64
    rng = np.random.RandomState(0)
    q = rng.randn(B, L, Hkv * g, w, d).astype(np.float32)
    k = np.broadcast_to(rng.randn(1, 1, 1, 1, d), (B, L, Hkv, n, d)).astype(np.float32).copy()
    psi = oracle.score(0, q, k, np.array([n], np.int32))
    want = np.zeros(n)
    for r in range(w):
        pos = n - w + r
        want[: pos + 1] += g / (pos + 1)
    np.testing.assert_allclose(psi, np.broadcast_to(want, psi.shape), rtol=1e-12)


def test_score_rows_sum_to_one_and_dominant_key():
    B, L, Hq, Hkv, n, w, d = 2, 1, 4, 2, 50, 4, 64
    rng = np.random.RandomState(1)
    q = rng.randn(B, L, Hq, w, d).astype(np.float32)
    k = rng.randn(B, L, Hkv, n, d).astype(np.float32)
    sl = np.array([50, 33], np.int32)
    psi = oracle.score(0, q, k, sl)
    assert (psi >= 0).all()
    np.testing.assert_allclose(psi.sum(-1), (Hq // Hkv) * w, rtol=1e-12)  # each softmax row sums to 1
    assert (psi[1, :, :, 33:] == 0).all()
    # one key with a huge logit for every row takes (almost) all the mass of the rows that see it
    k2, q2 = k.copy(), q.copy()
    k2[0, 0, 0, 10] = 0
    q2[0, 0, 0:2, :, 0] = 5.0
    k2[0, 0, 0, 10, 0] = 400.0
    psi2 = oracle.score(0, q2, k2, sl)
    assert abs(psi2[0, 0, 0, 10] - 2 * w) < 1e-9


@pytest.mark.parametrize("causal", [0, 1])
def test_score_matches_library_attention(causal):
    # alpha rows are what a library attention returns for V = identity; psi is their column sum over the group
    B, L, Hq, Hkv, n, w, d = 1, 2, 6, 2, 45, 7, 64
    g = Hq // Hkv
    rng = np.random.RandomState(2)
    q = rng.randn(B, L, Hq, w, d).astype(np.float32)
    k = rng.randn(B, L, Hkv, n, d).astype(np.float32)
    psi, lse = oracle.score(0, q, k, np.array([n], np.int32), causal=causal, want_lse=True)
    tq = torch.from_numpy(q).double()
    tk = torch.from_numpy(k).double().repeat_interleave(g, dim=2)
    pos = torch.arange(n - w, n).view(w, 1)
    allow = (torch.arange(n).view(1, n) <= pos) if causal else torch.ones(w, n, dtype=torch.bool)
    eye = torch.eye(n, dtype=torch.float64).expand(B, L, Hq, n, n)
    alpha = torch.nn.functional.scaled_dot_product_attention(tq, tk, eye, attn_mask=allow)
    want = alpha.view(B, L, Hkv, g, w, n).sum((3, 4)).numpy()
    np.testing.assert_allclose(psi, want, rtol=1e-10, atol=1e-14)
    logits = (tq @ tk.transpose(-1, -2)) / math.sqrt(d)
    want_lse = torch.logsumexp(logits.masked_fill(~allow, -math.inf), -1).numpy()
    np.testing.assert_allclose(lse, want_lse, rtol=1e-12)


def test_score_single_row_is_textbook_softmax_bf16_bits():
    # w = 1, g = 1: psi is one softmax row; inputs given as bf16 bit patterns
    n, d = 29, 128
    rng = np.random.RandomState(3)
    tq = torch.from_numpy(rng.randn(1, 1, 1, 1, d).astype(np.float32)).bfloat16()
    tk = torch.from_numpy(rng.randn(1, 1, 1, n, d).astype(np.float32)).bfloat16()
    psi = oracle.score(1, tq.view(torch.int16).numpy().view(np.uint16), tk.view(torch.int16).numpy().view(np.uint16),
                       np.array([n], np.int32))
    s = (tk.double()[0, 0, 0] @ tq.double()[0, 0, 0, 0]) / math.sqrt(d)
    np.testing.assert_allclose(psi[0, 0, 0], torch.softmax(s, 0).numpy(), rtol=1e-12)


def test_score_short_sequence_skips_rows_before_position_zero():
    n, w, d = 3, 5, 64
    rng = np.random.RandomState(4)
    q = rng.randn(1, 1, 1, w, d).astype(np.float32)
    k = rng.randn(1, 1, 1, n, d).astype(np.float32)
    psi, lse = oracle.score(0, q, k, np.array([n], np.int32), want_lse=True)
    assert abs(psi.sum() - n) < 1e-12  # only the 3 rows at positions 0, 1, 2 exist
    assert np.isneginf(lse[0, 0, 0, :2]).all()
    # the same as a 3-row window made of the last three queries
    np.testing.assert_allclose(psi, oracle.score(0, q[:, :, :, 2:], k, np.array([n], np.int32)), rtol=1e-15)
    assert psi[0, 0, 0, 0] > 1.0  # the row at position 0 sees only key 0


# ---------------------------------------------------------------- stages 2-3: Eq. 6, 8, 9, 10, 11


def test_allocate_handworked_case():
    h = _hand()
    q, k, _, mask, sl = _hand_inputs(h)
    psi = oracle.score(0, q, k, sl, scale=1 / 8).astype(np.float32)
    psi2 = np.concatenate([psi, psi], axis=1)  # L = 2 with identical layers
    for theta, key in ((0.5, "theta_0p5"), (0.9, "theta_0p9")):
        al = oracle.allocate(psi2, mask, sl, np.array([h["budget"]], np.int32), theta, hcc_mode=1)
        assert al["demand"][0, 0, 0].tolist() == [h[key]["k_v"], h[key]["k_t"]]
        np.testing.assert_allclose(al["mass"][0, 0, 0], [h["w_v"], h["w_t"]], rtol=1e-6)
        np.testing.assert_allclose(al["pref"][0, 0, 0], [h["pref_v"], h["pref_t"]], rtol=1e-6)
        assert al["budgets"][0, 0, 0].tolist() == [h["b_v"], h["b_t"]]
        if theta == 0.5:
            assert al["phi"][0].tolist() == [8.0, h["phi2_L2_H1_theta_0p5"]]


@pytest.mark.parametrize("mode,key", [(1, "paper"), (2, "literal"), (0, "off")])
def test_allocate_layer_recurrence_closed_form(mode, key):
    with open(os.path.join(GOLDEN, "hcc_uniform.json")) as f:
        gold = json.load(f)
    n, H, L = gold["n_v"] + gold["n_t"], gold["H"], gold["L"]
    mask = np.zeros((1, n), np.uint8)
    mask[0, 3 : 3 + gold["n_v"]] = 1
    psi = np.full((1, L, H, n), 1.0 / 16, np.float32)
    al = oracle.allocate(psi, mask, np.array([n], np.int32), np.array([gold["budget"]], np.int32), gold["theta"],
                         hcc_mode=mode)
    assert (al["demand"] == np.array(gold["demand"])).all()
    assert al["phi"][0].tolist() == gold[key]["phi"]
    for l in range(L):
        for hh in range(H):
            assert al["budgets"][0, l, hh].tolist() == gold[key]["budgets"][l]


def _subset_min_count(vals, theta_num, theta_den):
    """Eq. 9 by definition: smallest |C| over ALL subsets C with sum(C) >= theta * total (exact integers)."""
    total = sum(vals)
    if theta_num * total == 0:
        return 0
    for size in range(1, len(vals) + 1):
        for c in itertools.combinations(vals, size):
            if sum(c) * theta_den >= theta_num * total:
                return size
    return len(vals)


def test_topp_count_equals_subset_brute_force():
    rng = np.random.RandomState(5)
    for trial in range(40):
        n = int(rng.randint(2, 15))
        ints = rng.randint(0, 64, size=n)  # psi = ints / 1024: exact in fp32 and in 2^-32 fixed point
        mask = (rng.rand(1, n) < 0.5).astype(np.uint8)
        psi = (ints / 1024.0).astype(np.float32).reshape(1, 1, 1, n)
        for num, den in ((1, 4), (1, 2), (3, 4), (1, 1), (0, 1)):
            al = oracle.allocate(psi, mask, np.array([n], np.int32), np.array([4], np.int32), num / den)
            for m, val in enumerate((1, 0)):
                vals = [int(x) for x in ints[mask[0] == val]]
                assert al["demand"][0, 0, 0, m] == _subset_min_count(vals, num, den), (trial, ints, mask, num, den)


def test_topp_count_limits_monotonicity_and_fp64_agreement():
    rng = np.random.RandomState(6)
    n = 300
    psi = rng.lognormal(0, 1.5, size=(1, 1, 1, n)).astype(np.float32)
    psi /= psi.sum()
    mask = (rng.rand(1, n) < 0.6).astype(np.uint8)
    sl, bud = np.array([n], np.int32), np.array([50], np.int32)
    prev = np.zeros(2, np.int64)
    for theta in (0.0, 1e-6, 0.1, 0.3, 0.5, 0.7, 0.9, 0.99, 1.0):
        dem = oracle.allocate(psi, mask, sl, bud, theta)["demand"][0, 0, 0]
        assert (dem >= prev).all()  # monotone in theta
        prev = dem
        for m, val in enumerate((1, 0)):
            sub = psi[0, 0, 0][mask[0] == val].astype(np.float64)
            if 0.0 < theta < 1.0:
                assert dem[m] == oracle.topp_count_f64(sub, np.float32(theta))
            if theta == 0.0:
                assert dem[m] == 0
            if theta == 1e-6:
                assert dem[m] == 1
            if theta == 1.0:
                assert dem[m] <= sub.size and dem[m] >= np.count_nonzero(sub >= 2.0 ** -32)


def test_allocate_invariants_and_mask_swap():
    rng = np.random.RandomState(7)
    B, L, H, n = 2, 5, 3, 120
    psi = rng.lognormal(0, 1, size=(B, L, H, n)).astype(np.float32)
    psi /= psi.sum(-1, keepdims=True) / 8.0
    mask = (rng.rand(B, n) < 0.7).astype(np.uint8)
    sl = np.array([120, 77], np.int32)
    psi[1, :, :, 77:] = 0
    bud = np.array([30, 20], np.int32)
    al = oracle.allocate(psi, mask, sl, bud, 0.4)
    np.testing.assert_allclose(al["pref"].sum(-1), 1.0, rtol=1e-15)  # preferences sum to 1 per head
    for b in range(B):
        np.testing.assert_allclose(al["mass"][b].sum(-1), psi[b, :, :, : sl[b]].astype(np.float64).sum(-1), rtol=1e-6)
        n_v = int(mask[b, : sl[b]].sum())
        for l in range(L):
            Phi = min(max(math.floor(al["phi"][b, l] + 0.5), 1), sl[b])
            # per-head budgets sum to the layer budget H * Phi^l after compensation
            assert al["budgets"][b, l].sum() == H * Phi
            assert (al["budgets"][b, l].sum(-1) == Phi).all()
            assert (al["budgets"][b, l, :, 0] <= n_v).all() and (al["budgets"][b, l, :, 1] <= sl[b] - n_v).all()
    sw = oracle.allocate(psi, 1 - mask, sl, bud, 0.4)
    np.testing.assert_array_equal(sw["pref"], al["pref"][..., ::-1])
    np.testing.assert_array_equal(sw["demand"], al["demand"][..., ::-1])
    off = oracle.allocate(psi, mask, sl, bud, 0.4, hcc_mode=0)
    assert (off["phi"] == bud[:, None]).all()
    nompa = oracle.allocate(psi, mask, sl, bud, 0.4, mpa=0)
    assert (nompa["budgets"][..., 0] == 0).all()
    np.testing.assert_array_equal(nompa["phi"], al["phi"])


def test_allocate_demand_mode_conserves_the_total_budget():
    """Mode DEMAND (each layer but the last keeps what Eq. 9 asks for, phi follows Eq. 10-11 in per-head units): by
    induction phi^{l+1} * H * (L - l) = L * H * B - (spent so far), so with the last layer budgeted by Eq. 8 the total
    kept over all layers is L * H * B up to the rounding of the last Phi. Random scores, demands well inside the
    clamps."""
    rng = np.random.RandomState(5)
    B, L, H, n = 2, 6, 3, 400
    psi = rng.gamma(0.6, 1.0, size=(B, L, H, n)).astype(np.float32)
    mask = (rng.rand(B, n) < 0.5).astype(np.uint8)
    sl = np.array([n, n - 37], np.int32)
    bud = np.array([120, 90], np.int32)
    al = oracle.allocate(psi, mask, sl, bud, 0.55, hcc_mode=3)
    pa = oracle.allocate(psi, mask, sl, bud, 0.55, hcc_mode=1)
    np.testing.assert_array_equal(al["demand"], pa["demand"])
    for b in range(B):
        assert al["phi"][b, 0] == bud[b]
        assert (al["phi"][b] > 1).all() and (al["phi"][b] < sl[b]).all()  # no clamp was hit
        np.testing.assert_array_equal(al["budgets"][b, : L - 1], al["demand"][b, : L - 1])
        spent = 0
        for l in range(L - 1):  # the recurrence, re-derived from its meaning: what is left over the layers left
            spent += int(al["demand"][b, l].sum())
            want = (L * H * int(bud[b]) - spent) / (H * (L - 1 - l))
            assert abs(al["phi"][b, l + 1] - want) < 1e-9 * want
        Phi_last = math.floor(al["phi"][b, L - 1] + 0.5)
        assert al["budgets"][b, L - 1].sum() == H * Phi_last
        total = spent + int(al["budgets"][b, L - 1].sum())
        assert abs(total - L * H * int(bud[b])) <= H / 2 + 1e-9


def test_allocate_surplus_spills_to_other_modality():
    n = 40
    mask = np.zeros((1, n), np.uint8)
    mask[0, :3] = 1  # only 3 visual tokens but they hold most of the mass
    psi = np.full((1, 1, 1, n), 0.01, np.float32)
    psi[0, 0, 0, :3] = 1.0
    al = oracle.allocate(psi, mask, np.array([n], np.int32), np.array([20], np.int32), 0.5)
    assert al["budgets"][0, 0, 0].tolist() == [3, 17]
    al = oracle.allocate(psi, 1 - mask, np.array([n], np.int32), np.array([20], np.int32), 0.5)
    assert al["budgets"][0, 0, 0].tolist() == [17, 3]
    al = oracle.allocate(psi, mask, np.array([n], np.int32), np.array([100], np.int32), 0.5)
    assert al["budgets"][0, 0, 0].tolist() == [3, 37]  # budget clamped to n


# ---------------------------------------------------------------- stage 4: selection and compaction


def test_select_handworked_case():
    h = _hand()
    q, k, _, mask, sl = _hand_inputs(h)
    psi = oracle.score(0, q, k, sl, scale=1 / 8).astype(np.float32)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, np.array([[[[h["b_v"], h["b_t"]]]]], np.int32))
    assert rc == 0 and kept_len.tolist() == [8] and seg_off.tolist() == [0, 8]
    assert kept_idx[:8].tolist() == h["kept_idx"]


def test_select_equals_full_sort_brute_force():
    rng = np.random.RandomState(8)
    B, L, H, n = 2, 2, 3, 97
    psi = rng.randint(0, 12, size=(B, L, H, n)).astype(np.float32) / 16  # many exact ties
    mask = (rng.rand(B, n) < 0.5).astype(np.uint8)
    sl = np.array([97, 60], np.int32)
    budgets = rng.randint(0, 40, size=(B, L, H, 2)).astype(np.int32)
    headroom = 3
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, budgets, headroom=headroom)
    assert rc == 0
    u = 0
    for b in range(B):
        for l in range(L):
            for hh in range(H):
                keep = []
                for m, val in enumerate((1, 0)):
                    pos = np.nonzero(mask[b, : sl[b]] == val)[0]
                    order = np.lexsort((pos, -psi[b, l, hh, pos]))  # psi descending, then position ascending
                    keep += pos[order][: budgets[b, l, hh, m]].tolist()
                keep = sorted(keep)
                got = kept_idx[seg_off[u] : seg_off[u] + kept_len[u]].tolist()
                assert got == keep
                assert seg_off[u + 1] - seg_off[u] == len(keep) + headroom
                evicted = sorted(set(range(sl[b])) - set(keep))
                assert len(evicted) + len(keep) == sl[b]
                u += 1
    # budget >= token count keeps everything (identity); mpa = 0 ignores the mask
    big = np.full((B, L, H, 2), 1000, np.int32)
    rc, kl, so, ki = oracle.select(psi, mask, sl, big)
    assert kl.reshape(B, -1)[0].tolist() == [97] * (L * H) and ki[:97].tolist() == list(range(97))
    one = np.zeros((B, L, H, 2), np.int32)
    one[..., 1] = 5
    rc, kl, so, ki = oracle.select(psi, mask, sl, one, mpa=0)
    order = np.lexsort((np.arange(97), -psi[0, 0, 0]))
    assert ki[:5].tolist() == sorted(order[:5].tolist())
    # too small a capacity is reported, not overrun
    rc, *_ = oracle.select(psi, mask, sl, budgets, headroom=headroom, capacity=10)
    assert rc == 5


def test_pooling_and_window_retention_handworked_case():
    # options this build adds to the paper's selection step (the paper defines neither): values worked by hand
    with open(os.path.join(GOLDEN, "pooling_window_16.json")) as f:
        g = json.load(f)
    h = _hand()
    q, k, _, mask, sl = _hand_inputs(h)
    psi = oracle.score(0, q, k, sl, scale=1 / 8).astype(np.float32)
    bud8 = np.array([[[[3, 5]]]], np.int32)

    def kept(budgets, **kw):
        rc, kl, so, ki = oracle.select(psi, mask, sl, budgets, **kw)
        assert rc == 0
        return ki[: kl[0]].tolist()

    assert kept(bud8, pool_kernel=3) == g["kept_pool3"]
    assert kept(bud8, pool_kernel=3, keep_window=1, window=2) == g["kept_pool3_keep_window"]
    assert kept(bud8, keep_window=1, window=2) == g["kept_pool1_keep_window"]
    assert kept(bud8) == h["kept_idx"]  # both options off: the base case
    for budget, key in ((2, "budget_2_keep_window"), (1, "budget_1_keep_window")):
        al = oracle.allocate(psi, mask, sl, np.array([budget], np.int32), 0.5, keep_window=1, window=2)
        assert al["budgets"][0, 0, 0].tolist() == [g[key]["b_v"], g[key]["b_t"]]
        assert kept(al["budgets"], keep_window=1, window=2) == g[key]["kept"]
    al = oracle.allocate(psi, mask, sl, np.array([2], np.int32), 0.5)
    assert al["budgets"][0, 0, 0].tolist() == [g["budget_2_no_keep"]["b_v"], g["budget_2_no_keep"]["b_t"]]
    assert kept(al["budgets"]) == g["budget_2_no_keep"]["kept"]
    al8 = oracle.allocate(psi, mask, sl, np.array([8], np.int32), 0.5, keep_window=1, window=2)
    assert al8["budgets"][0, 0, 0].tolist() == [g["budget_8"]["b_v"], g["budget_8"]["b_t"]]


@pytest.mark.parametrize("pool", [1, 3, 7, 15])
@pytest.mark.parametrize("keep", [0, 1])
def test_pooled_selection_equals_library_maximum_filter_and_full_sort(pool, keep):
    # the ranking score against scipy's maximum filter (positions outside the sequence do not count: fill with -inf),
    # the choice against a full sort, the forced window positions against their definition
    from scipy.ndimage import maximum_filter1d

    rng = np.random.RandomState(80 + pool)
    B, L, H, n, w = 2, 2, 2, 131, 9
    psi = (rng.randint(1, 40, size=(B, L, H, n)) / 64).astype(np.float32)  # many exact ties
    mask = (rng.rand(B, n) < 0.6).astype(np.uint8)
    sl = np.array([131, 77], np.int32)
    budgets = rng.randint(0, 50, size=(B, L, H, 2)).astype(np.int32)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, budgets, headroom=2, keep_window=keep, window=w,
                                                    pool_kernel=pool)
    assert rc == 0
    u = 0
    for b in range(B):
        nb = int(sl[b])
        win = set(range(max(0, nb - w), nb)) if keep else set()
        for l in range(L):
            for hh in range(H):
                pooled = maximum_filter1d(psi[b, l, hh, :nb].astype(np.float64), size=pool, mode="constant", cval=-np.inf)
                assert (pooled >= psi[b, l, hh, :nb]).all()
                want = set(win)
                for m, val in enumerate((1, 0)):
                    pos = np.nonzero(mask[b, :nb] == val)[0]
                    forced = [x for x in pos.tolist() if x in win]
                    free = np.array([x for x in pos.tolist() if x not in win], np.int64)
                    take = min(max(int(budgets[b, l, hh, m]), len(forced)), pos.size) - len(forced)
                    order = np.lexsort((free, -pooled[free])) if free.size else np.zeros(0, np.int64)
                    want |= set(free[order][:take].tolist())
                got = kept_idx[seg_off[u]: seg_off[u] + kept_len[u]].tolist()
                assert got == sorted(want), (b, l, hh)
                assert win <= set(got)
                u += 1


def test_window_retention_floors_budgets_and_changes_nothing_else():
    rng = np.random.RandomState(81)
    B, L, H, n, w = 2, 4, 3, 150, 12
    psi = rng.rand(B, L, H, n).astype(np.float32)
    mask = (rng.rand(B, n) < 0.5).astype(np.uint8)
    sl = np.array([150, 90], np.int32)
    bud = np.array([10, 30], np.int32)
    for mpa in (1, 0):
        for mode in (0, 1, 2, 3):
            base = oracle.allocate(psi, mask, sl, bud, 0.3, mpa=mpa, hcc_mode=mode)
            kw = oracle.allocate(psi, mask, sl, bud, 0.3, mpa=mpa, hcc_mode=mode, keep_window=1, window=w)
            for key in ("mass", "pref", "demand", "phi"):
                assert np.array_equal(base[key], kw[key]), key
            for b in range(B):
                nb = int(sl[b])
                win = mask[b, nb - w: nb]
                lo = np.array([int(win.sum()), int(w - win.sum())]) if mpa else np.array([0, w])
                assert (kw["budgets"][b] >= lo).all()
                # a head's total: the layer budget, or the window size where that is larger
                if mode != 3:
                    Phi = np.clip(np.floor(base["phi"][b] + 0.5), 1, nb).astype(np.int64)
                    tot = np.maximum(Phi, w)[:, None]
                    assert (kw["budgets"][b].sum(-1) == np.broadcast_to(tot, (L, H))).all()
                # where the base budgets already cover the window nothing changes
                same = (base["budgets"][b] >= lo).all(-1)
                assert np.array_equal(kw["budgets"][b][same], base["budgets"][b][same])
            rc, kl, so, ki = oracle.select(psi, mask, sl, kw["budgets"], mpa=mpa, keep_window=1, window=w)
            assert rc == 0 and np.array_equal(kl, kw["budgets"].reshape(-1, 2).sum(-1))


def test_compact_is_row_gather():
    rng = np.random.RandomState(9)
    B, L, H, n, d = 1, 2, 2, 31, 64
    k = rng.randn(B, L, H, n, d).astype(np.float32)
    v = rng.randn(B, L, H, n, d).astype(np.float32)
    psi = rng.rand(B, L, H, n).astype(np.float32)
    mask = (rng.rand(B, n) < 0.5).astype(np.uint8)
    budgets = np.full((B, L, H, 2), 4, np.int32)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, np.array([n], np.int32), budgets, headroom=2)
    k_c, v_c = oracle.compact(0, k, v, kept_idx, seg_off, kept_len, int(seg_off[-1]))
    kf, vf = k.reshape(-1, n, d), v.reshape(-1, n, d)
    for u in range(B * L * H):
        idx = kept_idx[seg_off[u] : seg_off[u] + kept_len[u]]
        np.testing.assert_array_equal(k_c[seg_off[u] : seg_off[u] + kept_len[u]], kf[u][idx])
        np.testing.assert_array_equal(v_c[seg_off[u] : seg_off[u] + kept_len[u]], vf[u][idx])
        assert (k_c[seg_off[u] + kept_len[u] : seg_off[u + 1]] == 0).all()


# ---------------------------------------------------------------- stage 5: Eq. 4-5


def test_decode_handworked_case():
    h = _hand()
    q, k, v, mask, sl = _hand_inputs(h)
    kept = np.array(h["kept_idx"], np.int32)
    k_c, v_c = oracle.compact(0, k, v, kept, np.array([0, 8], np.int64), np.array([8], np.int32), 8)
    qd = np.zeros((1, 1, 1, 64), np.float32)
    qd[..., 0] = 8.0
    kl = np.array([8], np.int32)
    rc, out, lse = oracle.decode(0, qd, None, None, k_c, v_c, np.array([0, 8], np.int64), kl, Hkv=1, scale=1 / 8)
    assert rc == 0 and abs(out[0, 0, 0, 0] - h["decode_o0"]) < 1e-6 and (out[0, 0, 0, 1:] == 0).all()
    assert abs(lse[0, 0, 0] - math.log(31.0)) < 1e-6


def test_decode_matches_library_attention_with_append_and_gqa():
    rng = np.random.RandomState(10)
    B, L, Hq, Hkv, d = 2, 2, 6, 2, 64
    g = Hq // Hkv
    units = B * L * Hkv
    lens = rng.randint(0, 20, size=units).astype(np.int32)
    lens[3] = 0
    headroom = 2
    seg_off = np.concatenate([[0], np.cumsum(lens + headroom)]).astype(np.int64)
    cap = int(seg_off[-1])
    k_c = rng.randn(cap, d).astype(np.float32)
    v_c = rng.randn(cap, d).astype(np.float32)
    q = rng.randn(B, L, Hq, d).astype(np.float32)
    kn = rng.randn(B, L, Hkv, d).astype(np.float32)
    vn = rng.randn(B, L, Hkv, d).astype(np.float32)
    for step in range(3):  # third append must overflow the 2 rows of headroom
        k_before, len_before = k_c.copy(), lens.copy()
        rc, out, lse = oracle.decode(0, q, kn, vn, k_c, v_c, seg_off, lens, Hkv=Hkv)
        if step < 2:
            assert rc == 0 and (lens == len_before + 1).all()
        else:
            assert rc == 5 and (lens == len_before).all() and (k_c == k_before).all()
        for u in range(units):
            b, l, hh = u // (L * Hkv), (u // Hkv) % L, u % Hkv
            if step < 2:
                np.testing.assert_array_equal(k_c[seg_off[u] + lens[u] - 1], kn[b, l, hh])  # Eq. 4
            ks = torch.from_numpy(k_c[seg_off[u] : seg_off[u] + lens[u]]).double()
            vs = torch.from_numpy(v_c[seg_off[u] : seg_off[u] + lens[u]]).double()
            qq = torch.from_numpy(q[b, l, hh * g : (hh + 1) * g]).double()
            want = torch.nn.functional.scaled_dot_product_attention(qq[None], ks[None], vs[None])[0]
            np.testing.assert_allclose(out[b, l, hh * g : (hh + 1) * g], want.numpy(), rtol=1e-10, atol=1e-12)
    # an empty segment without append gives zeros and -inf
    lens0 = np.zeros(units, np.int32)
    rc, out, lse = oracle.decode(0, q, None, None, k_c, v_c, seg_off, lens0, Hkv=Hkv)
    assert rc == 0 and (out == 0).all() and np.isneginf(lse).all()
    # layer selection touches only that layer
    lens1 = lens.copy()
    rc, out1, _ = oracle.decode(0, q, None, None, k_c, v_c, seg_off, lens1, Hkv=Hkv, layer=1)
    assert (out1[:, 0] == 0).all() and np.abs(out1[:, 1]).sum() > 0


def test_full_budget_pipeline_equals_full_cache_attention():
    # budget >= n: eviction is the identity, so decode equals attention over the whole prompt
    from paper_2506_15724_b200 import synth

    wl = synth.scaled(synth.CONFIGS["tiny"], n=384, budget=10_000)
    inp = synth.make_inputs(wl)
    q, k, v = inp["q_win"].numpy(), inp["k"].numpy(), inp["v"].numpy()
    mask, sl = inp["mask"].numpy(), inp["seq_len"].numpy()
    psi = oracle.score(0, q, k, sl).astype(np.float32)
    al = oracle.allocate(psi, mask, sl, inp["budget"].numpy(), 0.5)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"])
    assert (kept_len == wl.n).all()
    k_c, v_c = oracle.compact(0, k, v, kept_idx, seg_off, kept_len, int(seg_off[-1]))
    dq, _, _ = synth.make_decode_step(wl, 0)
    rc, out, _ = oracle.decode(0, dq.numpy(), None, None, k_c, v_c, seg_off, kept_len, Hkv=wl.Hkv)
    want = torch.nn.functional.scaled_dot_product_attention(
        dq.double().unsqueeze(-2), torch.from_numpy(k).double(), torch.from_numpy(v).double()).squeeze(-2)
    np.testing.assert_allclose(out, want.numpy(), rtol=1e-10, atol=1e-12)


def test_planted_needles_survive_eviction():
    from paper_2506_15724_b200 import synth

    wl = synth.CONFIGS["tiny"]
    inp = synth.make_inputs(wl)
    mask, sl = inp["mask"].numpy(), inp["seq_len"].numpy()
    psi = oracle.score(0, inp["q_win"].numpy(), inp["k"].numpy(), sl).astype(np.float32)
    al = oracle.allocate(psi, mask, sl, inp["budget"].numpy(), wl.theta)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"])
    needles = set(synth.needle_positions(wl, mask)[0].reshape(-1).tolist())
    for u in range(wl.units):
        assert needles <= set(kept_idx[seg_off[u] : seg_off[u] + kept_len[u]].tolist())
