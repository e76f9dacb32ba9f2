"""GPU parity: every stage of the CUDA library against the CPU oracle, element by element, through the C ABI.

Staged tests feed each CUDA stage the ORACLE's output of the stage before, so integer results must be bit-exact.
End-to-end tests run the CUDA pipeline on its own outputs and re-run each oracle stage on what the CUDA stage before
it produced; scores are compared within the stated tolerance, everything downstream exactly.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15724_b200 import binding as mk
from paper_2506_15724_b200 import synth
from helpers import (assert_segments_equal, capacity_of, compare_with_pure_oracle, config_of, dcode, oracle_stages_from,
                     psi_close, to_np)

pytestmark = pytest.mark.gpu

PSI_RTOL = 1e-3      # the stated bar for scores and preferences (fp32 accumulation)
PSI_RTOL_SEEN = 2e-5  # what this implementation is expected to reach; a regression beyond it fails too
DEC_ATOL = {"bf16": 2e-2, "f32": 2e-5}

TINY = synth.CONFIGS["tiny"]
SHAPES = {
    "tiny": TINY,
    "tiny_gqa_ragged": synth.scaled(TINY, B=3, L=2, Hq=6, Hkv=2, n=389, w=5, budget=60, theta=0.3),
    "bf16_d128": synth.scaled(TINY, dtype="bf16", L=3, Hq=4, Hkv=4, d=128, n=1100, w=32, budget=200, theta=0.3,
                              n_needles=8),
    "bf16_gqa7": synth.scaled(TINY, dtype="bf16", L=2, Hq=14, Hkv=2, d=128, n=700, w=32, budget=150, theta=0.3),
    # twelve query heads per KV head: both row halves of the decode kernel's 16-row tensor-core tile are live
    "bf16_gqa12": synth.scaled(TINY, dtype="bf16", B=2, L=2, Hq=12, Hkv=1, d=128, n=900, w=8, budget=300, theta=0.3),
    "bf16_d64_long_window": synth.scaled(TINY, dtype="bf16", L=1, Hq=8, Hkv=2, d=64, n=2500, w=64, budget=300,
                                         theta=0.2),
    "f32_d128": synth.scaled(TINY, L=2, Hq=2, Hkv=1, d=128, n=450, w=8, budget=100),
    # shapes the tensor-core scoring path takes (bf16, g * w <= 64)
    "tc_d64_r24": synth.scaled(TINY, dtype="bf16", B=2, L=2, Hq=6, Hkv=2, d=64, n=700, w=8, budget=90, theta=0.4),
    "tc_d128_r64": synth.scaled(TINY, dtype="bf16", L=2, Hq=4, Hkv=2, d=128, n=1500, w=32, budget=250, theta=0.3),
    "tc_d128_r40": synth.scaled(TINY, dtype="bf16", L=1, Hq=2, Hkv=2, d=128, n=900, w=40, budget=120, theta=0.3),
    "tc_d64_r64_b3": synth.scaled(TINY, dtype="bf16", B=3, L=2, Hq=2, Hkv=2, d=64, n=2100, w=64, budget=333,
                                  theta=0.3),
    # many short sequences: work items of one to four tiles follow one another (accumulator slots and K stages
    # come round again within a few tiles)
    # 8192 keys x 32 rows: a unit needs the TMEM of a 4-CTA cluster (ragged batch: shorter sequences use fewer tiles)
    "tc_cluster4": synth.scaled(TINY, dtype="bf16", B=2, L=2, Hq=3, Hkv=3, d=128, n=8192, w=32, budget=900, theta=0.3,
                                n_needles=8),
    "tc_short_seqs": synth.scaled(TINY, dtype="bf16", B=5, L=3, Hq=4, Hkv=4, d=128, n=389, w=8, budget=40, theta=0.3),
}


def make_case(wl, ragged=True):
    inp = synth.make_inputs(wl, device="cpu")
    if ragged and wl.B > 1:  # shorten all but the first sequence; the tail of the window must stay text
        sl = inp["seq_len"].clone()
        for b in range(1, wl.B):
            sl[b] = max(wl.w // 2, wl.n - 97 * b - 1)
        inp["seq_len"] = sl
    return inp


def dev(inp):
    return {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items()}


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("path", ["auto", "twophase"])
def test_score_matches_oracle(name, causal, path, monkeypatch):
    # "auto": the library's own choice (for bf16 shapes with g * w <= 64 the TMEM-resident cluster kernel when a unit
    # fits); "twophase": the two-phase tensor-core kernel is forced where a tensor-core path applies
    if path == "twophase":
        if not name.startswith("tc_"):
            pytest.skip("no tensor-core path for this shape")
        monkeypatch.setenv("MADAKV_SCORE_PATH", "twophase")
    wl = SHAPES[name]
    inp = make_case(wl)
    cfg = config_of(wl, causal=causal)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl), want_lse=True)
    buf.psi.fill_(7.0)  # the call must overwrite every element, padding included
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    want, want_lse = oracle.score(dcode(wl), to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["seq_len"]),
                                  causal=causal, want_lse=True)
    got = buf.psi.cpu().numpy()
    worst = psi_close(got, want, PSI_RTOL)
    assert worst < PSI_RTOL_SEEN, worst
    for b in range(wl.B):
        assert (got[b, :, :, int(inp["seq_len"][b]):] == 0).all()
    lse = buf.lse.cpu().numpy().astype(np.float64)
    fin = np.isfinite(want_lse)
    assert (np.isneginf(lse) == ~fin).all()
    np.testing.assert_allclose(lse[fin], want_lse[fin], rtol=0, atol=2e-5)
    # run to run bit-identical (fixed reduction order)
    again = torch.empty_like(buf.psi)
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], None, again, buf.ws)
    assert torch.equal(again, buf.psi)


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_single_pass_score_with_given_lse(name, causal, path, monkeypatch):
    # madakv_score_lse gets the oracle's log-sum-exps (rounded to fp32) and must reproduce the oracle's psi; "auto"
    # takes the tensor-core kernel for the bf16 shapes, "generic" the fp32 kernel for all
    if path == "generic":
        monkeypatch.setenv("MADAKV_SCORE_PATH", "generic")
    wl = SHAPES[name]
    inp = make_case(wl)
    cfg = config_of(wl, causal=causal)
    g = dev(inp)
    want, want_lse = oracle.score(dcode(wl), to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["seq_len"]),
                                  causal=causal, want_lse=True)
    lse = torch.from_numpy(want_lse.astype(np.float32)).cuda()
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    buf.psi.fill_(7.0)  # the call must overwrite every element, padding included
    mk.madakv_score_lse(cfg, g["q_win"], g["k"], g["seq_len"], lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    got = buf.psi.cpu().numpy()
    assert psi_close(got, want, PSI_RTOL) < PSI_RTOL_SEEN
    for b in range(wl.B):
        assert (got[b, :, :, int(inp["seq_len"][b]):] == 0).all()
    # and it agrees with the two-pass call's own normalisers fed back in
    two = mk.EvictionBuffers(cfg, capacity_of(wl), want_lse=True)
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], two.lse, two.psi, two.ws)
    mk.madakv_score_lse(cfg, g["q_win"], g["k"], g["seq_len"], two.lse, buf.psi, buf.ws)
    assert psi_close(buf.psi.cpu().numpy(), two.psi.cpu().numpy().astype(np.float64), 1e-4) < 1e-4


@pytest.mark.parametrize("lag", ["8", "9", "40", "1000"])
def test_tensor_core_score_item_interleaving(lag, monkeypatch):
    # many more work items than the phase-1 lead: exercises the interleaved phase-2 / phase-1 item order and the
    # waits between CTAs; the result may not depend on the lead (fixed reduction order)
    wl = synth.scaled(TINY, dtype="bf16", B=2, L=3, Hq=8, Hkv=8, d=128, n=4096, w=32, budget=500, n_needles=8)
    inp = make_case(wl)
    cfg = config_of(wl)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl), want_lse=True)
    monkeypatch.setenv("MADAKV_SCORE_PATH", "twophase")  # the kernel with the item schedule
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    base = buf.psi.clone()
    monkeypatch.setenv("MADAKV_SCORE_LAG", lag)
    buf.psi.fill_(-1.0)
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert torch.equal(buf.psi, base)
    want = oracle.score(1, to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["seq_len"]))
    assert psi_close(buf.psi.cpu().numpy(), want, PSI_RTOL) < PSI_RTOL_SEEN
    monkeypatch.setenv("MADAKV_SCORE_PATH", "generic")
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert psi_close(buf.psi.cpu().numpy(), want, PSI_RTOL) < PSI_RTOL_SEEN
    monkeypatch.delenv("MADAKV_SCORE_PATH")  # the cluster kernel (8 units of 4096 keys: clusters of 2)
    monkeypatch.delenv("MADAKV_SCORE_LAG")
    buf.psi.fill_(-1.0)
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert psi_close(buf.psi.cpu().numpy(), want, PSI_RTOL) < PSI_RTOL_SEEN


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("mpa,hcc", [(1, mk.HCC_PAPER), (1, mk.HCC_LITERAL), (1, mk.HCC_DEMAND), (0, mk.HCC_OFF),
                                     (0, mk.HCC_PAPER), (0, mk.HCC_DEMAND)])
def test_staged_allocate_select_compact_are_bit_exact(name, mpa, hcc):
    wl = SHAPES[name]
    inp = make_case(wl)
    cfg = config_of(wl, mpa=mpa, hcc_mode=hcc)
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    psi32 = oracle.score(dcode(wl), to_np(inp["q_win"]), to_np(inp["k"]), sl).astype(np.float32)
    ref = oracle_stages_from(wl, cfg, psi32, mask, sl, bud, to_np(inp["k"]), to_np(inp["v"]))
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, ref["capacity"])
    buf.psi.copy_(torch.from_numpy(psi32))
    mk.madakv_allocate(cfg, buf.psi, g["mask"], g["seq_len"], g["budget"], buf.mass, buf.pref, buf.demand, buf.phi,
                       buf.budgets, buf.ws)
    for key in ("mass", "pref", "demand", "phi", "budgets"):
        assert np.array_equal(getattr(buf, key).cpu().numpy(), ref[key]), key
    # stage 4a on the oracle's budgets
    buf.budgets.copy_(torch.from_numpy(ref["budgets"]))
    mk.madakv_select(cfg, buf.psi, g["mask"], g["seq_len"], buf.budgets, buf.kept_len, buf.seg_off, buf.kept_idx,
                     buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert np.array_equal(buf.kept_len.cpu().numpy(), ref["kept_len"])
    assert np.array_equal(buf.seg_off.cpu().numpy(), ref["seg_off"])
    assert_segments_equal(ref["kept_len"], ref["seg_off"], buf.kept_idx.cpu().numpy(), ref["kept_idx"], "kept_idx")
    # stage 4b on the oracle's indices
    buf.kept_idx.copy_(torch.from_numpy(ref["kept_idx"]))
    mk.madakv_compact(cfg, g["k"], g["v"], buf.kept_idx, buf.seg_off, buf.kept_len, buf.k_c, buf.v_c, buf.ws)
    assert_segments_equal(ref["kept_len"], ref["seg_off"], to_np(buf.k_c), ref["k_c"], "k_c")
    assert_segments_equal(ref["kept_len"], ref["seg_off"], to_np(buf.v_c), ref["v_c"], "v_c")


@pytest.mark.parametrize("name", ["tiny", "tiny_gqa_ragged", "bf16_gqa7", "tc_short_seqs", "tc_cluster4"])
@pytest.mark.parametrize("pool,keep", [(3, 0), (1, 1), (7, 1), (15, 1)])
@pytest.mark.parametrize("mpa,hcc", [(1, mk.HCC_PAPER), (0, mk.HCC_PAPER), (1, mk.HCC_DEMAND)])
def test_pooling_and_window_retention_are_bit_exact(name, pool, keep, mpa, hcc):
    """The two selection options outside the paper (score pooling, forced retention of the proxy tokens), staged on
    the oracle's scores: budgets with the window floors, kept positions under the pooled ranking and compacted rows are
    bit-exact against the oracle; so is the layer-by-layer allocation call."""
    wl = SHAPES[name]
    inp = make_case(wl)
    cfg = config_of(wl, mpa=mpa, hcc_mode=hcc, keep_window=keep, pool_kernel=pool)
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    if name == "tiny_gqa_ragged":
        bud = np.array([2, 60, 3], np.int32)  # budgets below the window size: the floors bind
    psi32 = oracle.score(dcode(wl), to_np(inp["q_win"]), to_np(inp["k"]), sl).astype(np.float32)
    ref = oracle_stages_from(wl, cfg, psi32, mask, sl, bud, to_np(inp["k"]), to_np(inp["v"]))
    g = dev(inp)
    d_bud = torch.from_numpy(bud).cuda()
    buf = mk.EvictionBuffers(cfg, ref["capacity"])
    buf.psi.copy_(torch.from_numpy(psi32))
    mk.madakv_allocate(cfg, buf.psi, g["mask"], g["seq_len"], d_bud, buf.mass, buf.pref, buf.demand, buf.phi,
                       buf.budgets, buf.ws)
    for key in ("mass", "pref", "demand", "phi", "budgets"):
        assert np.array_equal(getattr(buf, key).cpu().numpy(), ref[key]), key
    if keep:
        for b in range(wl.B):
            win = mask[b, max(int(sl[b]) - wl.w, 0): int(sl[b])]
            lo = [int(win.sum()), int(win.size - win.sum())] if mpa else [0, int(win.size)]
            assert (ref["budgets"][b] >= np.array(lo)).all()
    mk.madakv_select(cfg, buf.psi, g["mask"], g["seq_len"], buf.budgets, buf.kept_len, buf.seg_off, buf.kept_idx,
                     buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert np.array_equal(buf.kept_len.cpu().numpy(), ref["kept_len"])
    assert np.array_equal(buf.seg_off.cpu().numpy(), ref["seg_off"])
    got_idx = buf.kept_idx.cpu().numpy()
    assert_segments_equal(ref["kept_len"], ref["seg_off"], got_idx, ref["kept_idx"], "kept_idx")
    if keep:  # every proxy token of every unit is kept
        for u in range(wl.units):
            b = u // (wl.L * wl.Hkv)
            a0 = int(ref["seg_off"][u])
            seg = set(got_idx[a0: a0 + int(ref["kept_len"][u])].tolist())
            assert set(range(max(int(sl[b]) - wl.w, 0), int(sl[b]))) <= seg
    mk.madakv_compact(cfg, g["k"], g["v"], buf.kept_idx, buf.seg_off, buf.kept_len, buf.k_c, buf.v_c, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert_segments_equal(ref["kept_len"], ref["seg_off"], to_np(buf.k_c), ref["k_c"], "k_c")
    # the same budgets from the layer-by-layer call
    if wl.L > 1 and hcc != mk.HCC_DEMAND:
        cfg1 = config_of(synth.scaled(wl, L=1), mpa=mpa, hcc_mode=hcc, keep_window=keep, pool_kernel=pool)
        one = mk.EvictionBuffers(cfg1, capacity_of(synth.scaled(wl, L=1)))
        phi = torch.zeros((wl.B, wl.L), dtype=torch.float64, device="cuda")
        for l in range(wl.L):
            mk.madakv_allocate_layer(cfg, l, buf.psi[:, l:l + 1].contiguous(), g["mask"], g["seq_len"], d_bud, one.mass,
                                     one.pref, one.demand, phi, one.budgets, buf.ws)
            assert np.array_equal(one.budgets.cpu().numpy()[:, 0], ref["budgets"][:, l]), l


@pytest.mark.parametrize("name", list(SHAPES))
def test_end_to_end_pass_and_decode(name, record_property):
    wl = SHAPES[name]
    inp = make_case(wl)
    cfg = config_of(wl)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    assert mk.madakv_poll_status(buf.ws) == 0
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    # scores against the oracle within tolerance
    want_psi = oracle.score(dcode(wl), to_np(inp["q_win"]), to_np(inp["k"]), sl)
    psi_gpu = buf.psi.cpu().numpy()
    psi_close(psi_gpu, want_psi, PSI_RTOL)
    # every later stage: the oracle re-run on the CUDA path's own scores must agree exactly
    ref = oracle_stages_from(wl, cfg, psi_gpu, mask, sl, bud, to_np(inp["k"]), to_np(inp["v"]))
    for key in ("mass", "pref", "demand", "phi", "budgets", "kept_len", "seg_off"):
        assert np.array_equal(getattr(buf, key).cpu().numpy(), ref[key]), key
    np.testing.assert_allclose(buf.pref.cpu().numpy().sum(-1), 1.0, rtol=1e-12)
    assert_segments_equal(ref["kept_len"], ref["seg_off"], buf.kept_idx.cpu().numpy(), ref["kept_idx"], "kept_idx")
    assert_segments_equal(ref["kept_len"], ref["seg_off"], to_np(buf.k_c), ref["k_c"], "k_c")
    assert_segments_equal(ref["kept_len"], ref["seg_off"], to_np(buf.v_c), ref["v_c"], "v_c")
    # pure-oracle pipeline (the oracle's own scores all the way): identical integers except at ties within 1e-5
    # relative; every use of a tie rule is counted and reported, nothing is skipped
    got = {key: getattr(buf, key).cpu().numpy() for key in ("demand", "phi", "budgets", "kept_len", "seg_off", "kept_idx")}
    stats, agreed, pure = compare_with_pure_oracle(wl, cfg, want_psi, got, mask, sl, bud)
    record_property("tie_rule_uses", stats)
    if stats["demand_ties"] == 0 and stats["budget_rounding_ties"] == 0:
        assert np.array_equal(pure["budgets"], ref["budgets"])
    # decode: three steps with append, against the oracle on the same ragged cache
    k_c, v_c, kept_len = ref["k_c"].copy(), ref["v_c"].copy(), ref["kept_len"].copy()
    for step in range(3):
        q, kn, vn = synth.make_decode_step(wl, step)
        rc, want, want_lse = oracle.decode(dcode(wl), to_np(q), to_np(kn), to_np(vn), k_c, v_c, ref["seg_off"],
                                           kept_len, Hkv=wl.Hkv)
        assert rc == 0
        buf.run_decode(q.cuda(), kn.cuda(), vn.cuda())
        assert mk.madakv_poll_status(buf.ws) == 0
        assert np.array_equal(buf.kept_len.cpu().numpy(), kept_len)
        got = buf.out.float().cpu().numpy()
        assert np.abs(got - want).max() <= DEC_ATOL[wl.dtype], np.abs(got - want).max()
        np.testing.assert_allclose(buf.lse_dec.cpu().numpy(), want_lse, rtol=0, atol=1e-4)
    assert_segments_equal(kept_len, ref["seg_off"], to_np(buf.k_c), k_c, "k_c after append")
    # one layer only: other layers' outputs stay untouched
    if wl.L > 1:
        q, _, _ = synth.make_decode_step(wl, 9)
        before = buf.out.clone()
        buf.run_decode(q.cuda(), layer=1)
        rc, want, _ = oracle.decode(dcode(wl), to_np(q), None, None, k_c, v_c, ref["seg_off"], kept_len, Hkv=wl.Hkv,
                                    layer=1)
        got = buf.out.float().cpu().numpy()
        assert np.abs(got[:, 1] - want[:, 1]).max() <= DEC_ATOL[wl.dtype]
        assert torch.equal(buf.out[:, 0], before[:, 0])


def test_edge_cases_budget_extremes_and_single_modality():
    wl = synth.scaled(TINY, L=2, n=330, w=8)
    inp = make_case(wl)
    g = dev(inp)
    mask, sl = to_np(inp["mask"]), to_np(inp["seq_len"])
    for budget, theta, flip in ((1, 0.5, None), (10_000, 1.0, None), (40, 0.0, None), (40, 0.5, 0), (40, 0.5, 1)):
        cfg = config_of(wl, theta=theta)
        m = mask if flip is None else np.full_like(mask, flip)
        bud = np.array([budget], np.int32)
        buf = mk.EvictionBuffers(cfg, capacity_of(wl))
        buf.run_eviction(g["q_win"], g["k"], g["v"], torch.from_numpy(m).cuda(), g["seq_len"],
                         torch.from_numpy(bud).cuda())
        assert mk.madakv_poll_status(buf.ws) == 0
        ref = oracle_stages_from(wl, cfg, buf.psi.cpu().numpy(), m, sl, bud, to_np(inp["k"]), to_np(inp["v"]))
        for key in ("demand", "phi", "budgets", "kept_len", "seg_off"):
            assert np.array_equal(getattr(buf, key).cpu().numpy(), ref[key]), (key, budget, theta, flip)
        assert_segments_equal(ref["kept_len"], ref["seg_off"], buf.kept_idx.cpu().numpy(), ref["kept_idx"], "kept_idx")
        if budget >= wl.n:
            assert (ref["kept_len"] == wl.n).all()


@pytest.mark.parametrize("n", [8192, 20000])
@pytest.mark.parametrize("kind", ["few_values", "all_equal", "flat_with_peaks", "distinct"])
def test_allocate_and_select_on_crafted_scores(kind, n):
    """Stages 2-4a on hand-made importance scores, bit-exact against the oracle: thousands of tied values (one
    radix bucket then holds most keys down to the last pass), a single value, a flat floor with a few peaks, and all-distinct values; one sequence
    length that fits the registers of a block and one that takes several rounds."""
    wl = synth.scaled(TINY, B=2, L=2, Hq=2, Hkv=2, n=n, w=8, budget=n // 5, theta=0.4)
    inp = synth.make_inputs(wl, device="cpu", want_v=False)
    rng = np.random.RandomState(11)
    shape = (wl.B, wl.L, wl.Hkv, wl.n)
    if kind == "few_values":
        psi = rng.choice(np.array([1e-3, 2e-3, 2.0000002e-3, 0.25, 3e-5], np.float32), size=shape)
    elif kind == "all_equal":
        psi = np.full(shape, 1.0 / wl.n, np.float32)
    elif kind == "flat_with_peaks":
        psi = np.full(shape, 3e-4, np.float32)
        psi[..., rng.choice(wl.n, 40, replace=False)] = rng.uniform(0.1, 2.0, size=40).astype(np.float32)
    else:
        psi = rng.uniform(1e-6, 1e-2, size=shape).astype(np.float32)
    psi = np.ascontiguousarray(psi, np.float32)
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    sl = sl.copy()
    sl[1] = wl.n - 301  # ragged
    psi[1, :, :, sl[1]:] = 0.0
    for theta in (0.05, 0.4, 0.97):
        cfg = config_of(wl, theta=theta)
        buf = mk.EvictionBuffers(cfg, capacity_of(wl))
        d_psi, d_mask = torch.from_numpy(psi).cuda(), inp["mask"].cuda()
        d_sl, d_bud = torch.from_numpy(sl).cuda(), inp["budget"].cuda()
        mk.madakv_allocate(cfg, d_psi, d_mask, d_sl, d_bud, buf.mass, buf.pref, buf.demand, buf.phi, buf.budgets,
                           buf.ws)
        mk.madakv_select(cfg, d_psi, d_mask, d_sl, buf.budgets, buf.kept_len, buf.seg_off, buf.kept_idx, buf.ws)
        assert mk.madakv_poll_status(buf.ws) == 0
        al = oracle.allocate(psi, mask, sl, bud, float(np.float32(theta)))
        for key in ("mass", "pref", "demand", "phi", "budgets"):
            assert np.array_equal(getattr(buf, key).cpu().numpy(), al[key]), (key, kind, theta)
        rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"], headroom=wl.max_new_tokens,
                                                        capacity=capacity_of(wl))
        assert rc == 0
        assert np.array_equal(buf.kept_len.cpu().numpy(), kept_len)
        assert_segments_equal(kept_len, seg_off, buf.kept_idx.cpu().numpy(), kept_idx, "kept_idx")


@pytest.mark.parametrize("name", ["tiny_gqa_ragged", "bf16_d128", "bf16_gqa7", "tc_short_seqs"])
@pytest.mark.parametrize("hcc", [mk.HCC_PAPER, mk.HCC_LITERAL, mk.HCC_DEMAND])
@pytest.mark.parametrize("split", [False, True])
def test_layer_by_layer_pass_equals_the_all_layer_pass(name, hcc, split):
    """The streaming use of the library: layer after layer, single-pass scoring with given log-sum-exps, then
    madakv_allocate_layer carrying phi, then selection and compaction with one-layer configs on slices of K/V. Given
    the same fp32 scores everything downstream is bit-identical to the all-layer calls; the single-pass scores
    themselves agree with the two-pass ones to rounding. split: masses, preferences and demands of ALL layers come
    from madakv_demand_layer first (they do not depend on the budget state), then madakv_allocate_layer without
    scores walks the layers."""
    wl = SHAPES[name]
    inp = make_case(wl)
    g = dev(inp)
    cfg = config_of(wl, hcc_mode=hcc)
    cfg1 = config_of(synth.scaled(wl, L=1), hcc_mode=hcc)
    ref = mk.EvictionBuffers(cfg, capacity_of(wl), want_lse=True)
    ref.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    assert mk.madakv_poll_status(ref.ws) == 0
    per = wl.Hkv
    r_len = ref.kept_len.cpu().numpy().reshape(wl.B, wl.L, per)
    r_off = ref.seg_off.cpu().numpy()
    r_idx, r_kc, r_vc = ref.kept_idx.cpu().numpy(), ref.k_c, ref.v_c
    phi = torch.zeros((wl.B, wl.L), dtype=torch.float64, device="cuda")
    cap1 = capacity_of(synth.scaled(wl, L=1))
    ones = [mk.EvictionBuffers(cfg1, cap1) for _ in range(wl.L)]
    if split:
        for l in range(wl.L):
            mk.madakv_demand_layer(cfg, ref.psi[:, l:l + 1].contiguous(), g["mask"], g["seq_len"], ones[l].mass,
                                   ones[l].pref, ones[l].demand, ref.ws)
    for l in range(wl.L):
        one = ones[l]
        q_l, k_l, v_l = g["q_win"][:, l:l + 1], g["k"][:, l:l + 1], g["v"][:, l:l + 1]  # views: strides go through
        mk.madakv_score_lse(cfg1, q_l, k_l, g["seq_len"], ref.lse[:, l:l + 1].contiguous(), one.psi, one.ws)
        assert psi_close(one.psi.cpu().numpy(), ref.psi[:, l:l + 1].cpu().numpy().astype(np.float64), 1e-4) < 1e-4
        psi_l = ref.psi[:, l:l + 1].contiguous()  # from here on the same scores as the all-layer pass
        mk.madakv_allocate_layer(cfg, l, None if split else psi_l, g["mask"], g["seq_len"], g["budget"], one.mass,
                                 one.pref, one.demand, phi, one.budgets, ref.ws)
        for key in ("mass", "pref", "demand", "budgets"):
            assert torch.equal(getattr(one, key)[:, 0], getattr(ref, key)[:, l]), (key, l)
        mk.madakv_select(cfg1, psi_l, g["mask"], g["seq_len"], one.budgets, one.kept_len, one.seg_off, one.kept_idx,
                         one.ws)
        mk.madakv_compact(cfg1, k_l, v_l, one.kept_idx, one.seg_off, one.kept_len, one.k_c, one.v_c, one.ws)
        assert mk.madakv_poll_status(one.ws) == 0
        o_len = one.kept_len.cpu().numpy().reshape(wl.B, per)
        o_off, o_idx = one.seg_off.cpu().numpy(), one.kept_idx.cpu().numpy()
        assert np.array_equal(o_len, r_len[:, l])
        for b in range(wl.B):
            for h in range(per):
                u_all, u_one = (b * wl.L + l) * per + h, b * per + h
                a0, a1 = int(r_off[u_all]), int(r_off[u_all]) + int(o_len[b, h])
                c0, c1 = int(o_off[u_one]), int(o_off[u_one]) + int(o_len[b, h])
                assert np.array_equal(o_idx[c0:c1], r_idx[a0:a1]), (l, b, h)
                assert torch.equal(one.k_c[c0:c1], r_kc[a0:a1]) and torch.equal(one.v_c[c0:c1], r_vc[a0:a1])
    assert torch.equal(phi, ref.phi)


def test_short_sequences_and_empty_sequence():
    wl = synth.scaled(TINY, B=4, L=1, n=320 + 8, w=8, budget=16)
    inp = synth.make_inputs(wl)
    inp["seq_len"] = torch.tensor([wl.n, 3, 0, 8], dtype=torch.int32)  # shorter than the window, empty, == window
    cfg = config_of(wl)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    assert mk.madakv_poll_status(buf.ws) == 0
    sl = to_np(inp["seq_len"])
    want_psi = oracle.score(0, to_np(inp["q_win"]), to_np(inp["k"]), sl)
    psi_close(buf.psi.cpu().numpy(), want_psi, PSI_RTOL)
    ref = oracle_stages_from(wl, cfg, buf.psi.cpu().numpy(), to_np(inp["mask"]), sl, to_np(inp["budget"]),
                             to_np(inp["k"]), to_np(inp["v"]))
    for key in ("demand", "phi", "budgets", "kept_len", "seg_off"):
        assert np.array_equal(getattr(buf, key).cpu().numpy(), ref[key]), key
    q, _, _ = synth.make_decode_step(wl, 0)
    buf.run_decode(q.cuda())
    kept_len = ref["kept_len"].copy()
    rc, want, want_lse = oracle.decode(0, to_np(q), None, None, ref["k_c"], ref["v_c"], ref["seg_off"], kept_len,
                                       Hkv=wl.Hkv)
    assert np.abs(buf.out.cpu().numpy() - want).max() <= 2e-5
    got_lse = buf.lse_dec.cpu().numpy()
    assert (np.isneginf(got_lse) == np.isneginf(want_lse)).all()
    assert (buf.out[2] == 0).all()  # empty sequence: zeros


@pytest.mark.parametrize("name", ["tiny_gqa_ragged", "tc_short_seqs", "bf16_gqa7"])
def test_sequence_lengths_outside_the_range_are_clamped(name):
    # seq_len[b] is device data the host cannot check: a value above n_max acts as n_max, a negative one as 0
    wl = SHAPES[name]
    inp = synth.make_inputs(wl, device="cpu")
    g = dev(inp)
    cfg = config_of(wl)
    good = torch.full((wl.B,), wl.n, dtype=torch.int32)
    odd = good.clone()
    odd[0] = wl.n + 9
    if wl.B > 1:
        good[1], odd[1] = 0, -3
    res = []
    for sl in (good, odd):
        buf = mk.EvictionBuffers(cfg, capacity_of(wl))
        buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], sl.cuda(), g["budget"])
        q, kn, vn = [t.cuda() for t in synth.make_decode_step(wl, 0)]
        buf.run_decode(q, kn, vn)
        assert mk.madakv_poll_status(buf.ws) == 0
        res.append(buf)
    for key in ("psi", "budgets", "kept_len", "seg_off", "kept_idx", "k_c", "v_c", "out"):
        assert torch.equal(getattr(res[0], key), getattr(res[1], key)), key


def test_capacity_overflow_is_reported_not_written():
    wl = synth.scaled(TINY, L=1, max_new_tokens=1)
    inp = make_case(wl)
    cfg = config_of(wl)
    g = dev(inp)
    small = 300  # rows: two of the 4 units x 129 rows fit
    buf = mk.EvictionBuffers(cfg, small)
    guard = torch.full((small + 64,), -7, dtype=torch.int32, device="cuda")
    buf.kept_idx = guard[:small]
    buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    assert mk.madakv_poll_status(buf.ws) == mk.ECAPACITY
    assert mk.madakv_poll_status(buf.ws) == 0  # cleared by the poll
    assert (guard[small:] == -7).all()
    # decode over a cache some of whose segments did not fit: those count as empty (zeros out), nothing beyond the
    # cache is read, the segments that fit are attended to as usual
    q, _, _ = [t.cuda() for t in synth.make_decode_step(wl, 0)]
    buf.run_decode(q)
    torch.cuda.synchronize()
    assert mk.madakv_poll_status(buf.ws) == 0
    lens, offs = buf.kept_len.cpu().numpy(), buf.seg_off.cpu().numpy()
    out = buf.out.float().cpu().numpy().reshape(wl.units, wl.g, wl.d)
    fits = offs[:-1] + lens + wl.max_new_tokens <= small
    assert fits.any() and not fits.all()
    assert np.isfinite(out).all() and (out[~fits] == 0).all() and (np.abs(out[fits]).sum(axis=(1, 2)) > 0).all()
    # a segment whose rows would fit but whose headroom ends beyond the cache (4 units x (128 + 1) rows, capacity 386:
    # unit 2 ends at row 386, its headroom at 387) is refused by selection like any other and must count as empty in
    # decode too; an append to it is refused
    buf = mk.EvictionBuffers(cfg, 386)
    buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    assert mk.madakv_poll_status(buf.ws) == mk.ECAPACITY
    lens, offs = buf.kept_len.cpu().numpy(), buf.seg_off.cpu().numpy()
    assert offs[2] + lens[2] == 386 and offs[3] == 387
    q, kn, vn = [t.cuda() for t in synth.make_decode_step(wl, 0)]
    buf.run_decode(q)
    assert mk.madakv_poll_status(buf.ws) == 0
    out = buf.out.float().cpu().numpy().reshape(wl.units, wl.g, wl.d)
    assert (out[2:] == 0).all() and (np.abs(out[:2]).sum(axis=(1, 2)) > 0).all()
    buf.run_decode(q, kn, vn)
    assert mk.madakv_poll_status(buf.ws) == mk.ECAPACITY
    assert np.array_equal(buf.kept_len.cpu().numpy()[2:], lens[2:])
    assert np.array_equal(buf.kept_len.cpu().numpy()[:2], lens[:2] + 1)
    # appending beyond the headroom: first append fits, second is refused and leaves the cache unchanged
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    q, kn, vn = [t.cuda() for t in synth.make_decode_step(wl, 0)]
    buf.run_decode(q, kn, vn)
    assert mk.madakv_poll_status(buf.ws) == 0
    lens, kc = buf.kept_len.clone(), buf.k_c.clone()
    buf.run_decode(q, kn, vn)
    assert mk.madakv_poll_status(buf.ws) == mk.ECAPACITY
    assert torch.equal(buf.kept_len, lens) and torch.equal(buf.k_c, kc)


def test_decode_refusals_come_before_the_append():
    # 17 query heads per KV head is outside the supported range: the call is refused on the host BEFORE the append
    # kernel could change the cache, so a caller may retry with another configuration without appending twice
    wl = synth.scaled(TINY, dtype="bf16", L=1, Hq=17, Hkv=1, d=128, n=64, w=8, budget=16, max_new_tokens=4)
    cfg = config_of(wl)
    ws = mk.new_workspace(cfg)
    k_c = torch.zeros((14, wl.d), dtype=torch.bfloat16, device="cuda")
    v_c = torch.zeros_like(k_c)
    seg_off = torch.tensor([0, 14], dtype=torch.int64, device="cuda")
    kept_len = torch.tensor([10], dtype=torch.int32, device="cuda")
    q, kn, vn = [t.cuda() for t in synth.make_decode_step(wl, 0)]
    out = torch.zeros((1, 1, 17, wl.d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mk.MadakvError) as e:
        mk.madakv_decode_attn(cfg, -1, q, kn, vn, k_c, v_c, seg_off, kept_len, out, None, ws)
    assert e.value.code == mk.EUNSUPPORTED
    torch.cuda.synchronize()
    assert int(kept_len[0]) == 10 and not k_c.any() and not v_c.any()


@pytest.mark.parametrize("name", ["bf16_d128", "bf16_gqa7"])
def test_decode_steps_replayed_from_a_cuda_graph(name):
    """Two decode steps with append, captured into a CUDA graph and replayed, give the cache and the outputs of the
    same two steps launched eagerly (the decode kernels are launched with programmatic stream serialisation outside a
    capture and in the ordinary way inside one; both orders of execution must be the same)."""
    wl = SHAPES[name]
    g = dev(make_case(wl))
    cfg = config_of(wl)
    steps = [tuple(t.cuda() for t in synth.make_decode_step(wl, s)) for s in range(2)]

    def prepared():
        buf = mk.EvictionBuffers(cfg, capacity_of(wl))
        buf.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
        return buf

    eager, outs = prepared(), []
    for q, kn, vn in steps:
        eager.run_decode(q, kn, vn)
        outs.append(eager.out.clone())
    assert mk.madakv_poll_status(eager.ws) == 0
    graphed = prepared()
    out2 = [torch.empty_like(graphed.out) for _ in steps]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for (q, kn, vn), o in zip(steps, out2):
            mk.madakv_decode_attn(cfg, -1, q, kn, vn, graphed.k_c, graphed.v_c, graphed.seg_off, graphed.kept_len, o, None,
                                  graphed.ws)
    graph.replay()
    torch.cuda.synchronize()
    assert mk.madakv_poll_status(graphed.ws) == 0
    assert torch.equal(graphed.kept_len, eager.kept_len)
    assert torch.equal(graphed.k_c, eager.k_c) and torch.equal(graphed.v_c, eager.v_c)
    for a, b in zip(outs, out2):
        assert torch.equal(a, b)


def test_decode_with_more_than_65535_segments():
    # 70 000 short segments in one call (a grid dimension of 65 535 must not be the limit); every unit against the oracle
    wl = synth.scaled(TINY, B=70, L=100, Hq=10, Hkv=10, d=64, n=16, w=4, budget=8, max_new_tokens=2)
    cfg = config_of(wl)
    rng = np.random.RandomState(5)
    lens = rng.randint(0, 15, size=wl.units).astype(np.int32)
    seg_off = np.concatenate([[0], np.cumsum(lens.astype(np.int64) + wl.max_new_tokens)])
    rows = int(seg_off[-1])
    k_c = synth.hash_normal(1, 91, 0, rows * wl.d).view(rows, wl.d).contiguous()
    v_c = synth.hash_normal(1, 92, 0, rows * wl.d).view(rows, wl.d).contiguous()
    q, kn, vn = synth.make_decode_step(wl, 0)
    ws = mk.new_workspace(cfg)
    d_kc, d_vc = k_c.cuda(), v_c.cuda()
    d_len = torch.from_numpy(lens).cuda()
    out = torch.zeros((wl.B, wl.L, wl.Hq, wl.d), dtype=torch.float32, device="cuda")
    mk.madakv_decode_attn(cfg, -1, q.cuda(), kn.cuda(), vn.cuda(), d_kc, d_vc, torch.from_numpy(seg_off).cuda(), d_len,
                          out, None, ws)
    assert mk.madakv_poll_status(ws) == 0
    kc_np, vc_np, lens_np = k_c.numpy().copy(), v_c.numpy().copy(), lens.copy()
    rc, want, _ = oracle.decode(0, to_np(q), to_np(kn), to_np(vn), kc_np, vc_np, seg_off, lens_np, Hkv=wl.Hkv)
    assert rc == 0 and np.array_equal(d_len.cpu().numpy(), lens_np)
    assert np.abs(out.cpu().numpy() - want).max() <= 2e-5


def test_bounded_wait_runs_out_and_the_library_recovers(monkeypatch):
    """Failure detection without a GPU fault: the two-phase scoring kernel's phase-2 items wait (bounded) for row flags
    that phase 1 publishes. With the flags withheld and the bound shortened to ~1 ms the wait runs out: the kernel
    records MADAKV_ETIMEOUT with the wait site, drains its copies and tensor-core work, frees its TMEM and returns;
    nothing hangs or faults, and the next ordinary call on the same workspace gives the oracle's scores."""
    wl = synth.scaled(TINY, dtype="bf16", L=1, Hq=2, Hkv=1, d=128, n=700, w=8, budget=90, theta=0.4)  # one CTA
    inp = make_case(wl)
    cfg = config_of(wl)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    monkeypatch.setenv("MADAKV_SCORE_PATH", "twophase")
    monkeypatch.setenv("MADAKV_TEST_HOLD_FLAGS", "1")
    monkeypatch.setenv("MADAKV_TEST_WAIT_CYCLES", "2000000")
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], None, buf.psi, buf.ws)
    torch.cuda.synchronize()
    site = int(buf.ws[4:8].view(torch.int32).item())
    assert mk.madakv_poll_status(buf.ws) == mk.ETIMEOUT
    assert site & 255 == 7 and site >> 8 == 0  # the wait for another item's row flags, in block 0
    assert mk.madakv_poll_status(buf.ws) == 0   # cleared by the poll
    monkeypatch.delenv("MADAKV_TEST_HOLD_FLAGS")
    monkeypatch.delenv("MADAKV_TEST_WAIT_CYCLES")
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], None, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    want = oracle.score(1, to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["seq_len"]))
    assert psi_close(buf.psi.cpu().numpy(), want, PSI_RTOL) < PSI_RTOL_SEEN


def test_strided_kv_layout():
    # K/V stored per layer as [B, H, n, d] inside a larger allocation (token stride > d)
    wl = synth.scaled(TINY, dtype="bf16", L=2, Hq=4, Hkv=2, d=128, n=340, w=8, budget=50)
    inp = make_case(wl)
    cfg = config_of(wl)
    g = dev(inp)
    big_k = torch.zeros((wl.L, wl.B, wl.Hkv, wl.n, wl.d + 64), dtype=torch.bfloat16, device="cuda")
    big_v = torch.zeros_like(big_k)
    big_k[..., : wl.d] = g["k"].permute(1, 0, 2, 3, 4)
    big_v[..., : wl.d] = g["v"].permute(1, 0, 2, 3, 4)
    kv, vv = big_k[..., : wl.d].permute(1, 0, 2, 3, 4), big_v[..., : wl.d].permute(1, 0, 2, 3, 4)
    a = mk.EvictionBuffers(cfg, capacity_of(wl))
    a.run_eviction(g["q_win"], g["k"], g["v"], g["mask"], g["seq_len"], g["budget"])
    b = mk.EvictionBuffers(cfg, capacity_of(wl))
    b.run_eviction(g["q_win"], kv, vv, g["mask"], g["seq_len"], g["budget"])
    assert torch.equal(a.psi, b.psi) and torch.equal(a.kept_idx, b.kept_idx)
    assert torch.equal(a.k_c, b.k_c) and torch.equal(a.v_c, b.v_c)


# Full-size checks. "all": the oracle scores every unit and the pure-oracle pipeline is compared on every unit; a
# tuple of layers: the oracle scores all units of those layers (the layer recurrence of Eq. 10-11 needs every
# layer, so downstream of the scores the oracle is re-run on the CUDA path's scores there).
FULL_SIZE = {"llava": "all", "qwen1024": "all", "qwen": "all", "qwen4096": "all", "llava13b": (7, 39),
             "batched": (0, 5, 17, 27), "long": (0, 9, 20, 31)}
_oracle_scores = {}  # the three Qwen-shaped budgets share their prompt, K and scores


def _oracle_psi(wl, inp, layers):
    key = (wl.seed, wl.layout, wl.B, wl.L, wl.Hq, wl.Hkv, wl.n, wl.w, layers)
    if key not in _oracle_scores:
        _oracle_scores.clear()
        sl = to_np(inp["seq_len"])
        if layers == "all":
            _oracle_scores[key] = oracle.score(1, to_np(inp["q_win"]), to_np(inp["k"]), sl, want_lse=True)
        else:
            ls = list(layers)
            _oracle_scores[key] = oracle.score(1, to_np(inp["q_win"][:, ls]), to_np(inp["k"][:, ls]), sl, want_lse=True)
    return _oracle_scores[key]


@pytest.mark.parametrize("name", list(FULL_SIZE))
def test_full_size_workload(name, record_property):
    """The benchmark workloads at full size, in the launch configuration bench.py times. Scores and log-sum-exps
    against the oracle element by element (every unit, or every unit of four layers for the two largest); stages 2-4a
    against the oracle on every unit; the compacted rows of every unit against a gather of the kept positions; one
    decode step on sampled units. Where the oracle scores every unit the whole pure-oracle pipeline is compared:
    kept sets identical except at ties within 1e-5 relative, each use of the tie rule counted."""
    wl = synth.CONFIGS[name]
    layers = FULL_SIZE[name]
    inp = synth.make_inputs(wl, device="cuda")
    cfg = config_of(wl)
    cap = wl.units * (min(wl.n, 2 * wl.budget) + wl.max_new_tokens)
    buf = mk.EvictionBuffers(cfg, cap, want_lse=True)
    mk.madakv_score(cfg, inp["q_win"], inp["k"], inp["seq_len"], buf.lse, buf.psi, buf.ws)
    mk.madakv_allocate(cfg, buf.psi, inp["mask"], inp["seq_len"], inp["budget"], buf.mass, buf.pref, buf.demand, buf.phi,
                       buf.budgets, buf.ws)
    mk.madakv_select(cfg, buf.psi, inp["mask"], inp["seq_len"], buf.budgets, buf.kept_len, buf.seg_off, buf.kept_idx,
                     buf.ws)
    mk.madakv_compact(cfg, inp["k"], inp["v"], buf.kept_idx, buf.seg_off, buf.kept_len, buf.k_c, buf.v_c, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    psi = buf.psi.cpu().numpy()
    lse = buf.lse.cpu().numpy()
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    # ---- scores and log-sum-exps, element by element
    want, want_lse = _oracle_psi(wl, inp, layers)
    ls = list(range(wl.L)) if layers == "all" else list(layers)
    worst = psi_close(psi[:, ls], want, PSI_RTOL)
    record_property("worst_relative_score_error", worst)
    assert worst < PSI_RTOL_SEEN, worst
    np.testing.assert_allclose(lse[:, ls], want_lse, rtol=0, atol=2e-5)
    np.testing.assert_allclose(psi.sum(-1), wl.g * wl.w, rtol=1e-5)  # every softmax row sums to 1, all units
    # the single-pass call, fed the normalisers just computed, gives the same scores
    once = torch.empty_like(buf.psi)
    mk.madakv_score_lse(cfg, inp["q_win"], inp["k"], inp["seq_len"], buf.lse, once, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    assert psi_close(once.cpu().numpy(), psi.astype(np.float64), 1e-4) < 1e-4
    del once
    # ---- stages 2-4a on all units: bit-exact functions of the fp32 scores
    al = oracle.allocate(psi, mask, sl, bud, float(np.float32(cfg.theta)))
    for key in ("mass", "pref", "demand", "phi", "budgets"):
        assert np.array_equal(getattr(buf, key).cpu().numpy(), al[key]), key
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"], headroom=wl.max_new_tokens,
                                                    capacity=cap)
    assert rc == 0
    assert np.array_equal(buf.kept_len.cpu().numpy(), kept_len)
    assert np.array_equal(buf.seg_off.cpu().numpy(), seg_off)
    got_idx = buf.kept_idx.cpu().numpy()
    assert_segments_equal(kept_len, seg_off, got_idx, kept_idx, "kept_idx")
    # ---- the pure-oracle pipeline on every unit (kept sets up to ties within 1e-5 relative)
    if layers == "all":
        got = dict(demand=al["demand"], phi=al["phi"], budgets=al["budgets"], kept_len=kept_len, seg_off=seg_off,
                   kept_idx=got_idx)
        stats, agreed, _ = compare_with_pure_oracle(wl, cfg, want, got, mask, sl, bud)
        record_property("tie_rule_uses", stats)
        print(name, "tie rule uses:", stats)
    # ---- stage 4b on every unit: the compacted rows are the kept rows (bit copies)
    k5 = inp["k"].view(wl.units, wl.n, wl.d)
    v5 = inp["v"].view(wl.units, wl.n, wl.d)
    d_idx = buf.kept_idx.long()
    for u in range(wl.units):
        a, b = int(seg_off[u]), int(seg_off[u] + kept_len[u])
        assert torch.equal(buf.k_c[a:b], k5[u][d_idx[a:b]]) and torch.equal(buf.v_c[a:b], v5[u][d_idx[a:b]]), u
    # ---- one decode step on sampled units against the oracle
    rng = np.random.RandomState(7)
    q, kn, vn = synth.make_decode_step(wl, 0, device="cuda")
    buf.run_decode(q, None, None)
    assert mk.madakv_poll_status(buf.ws) == 0
    out = buf.out.float().cpu().numpy().reshape(wl.B * wl.L, wl.Hq, wl.d)
    q3 = q.view(wl.B * wl.L, wl.Hq, wl.d)
    worst_dec = 0.0
    for u in rng.choice(wl.units, size=6, replace=False).tolist() + [0, wl.units - 1]:
        a, b = int(seg_off[u]), int(seg_off[u] + kept_len[u])
        kc, vc = to_np(buf.k_c[a:b]), to_np(buf.v_c[a:b])
        bl, h = divmod(u, wl.Hkv)
        heads = slice(h * wl.g, (h + 1) * wl.g)
        rc, want_o, _ = oracle.decode(1, to_np(q3[bl, heads]).reshape(1, 1, wl.g, wl.d), None, None, kc, vc,
                                      np.array([0, b - a], np.int64), np.array([b - a], np.int32), Hkv=1)
        worst_dec = max(worst_dec, float(np.abs(out[bl, heads] - want_o.reshape(wl.g, wl.d)).max()))
        assert worst_dec <= DEC_ATOL["bf16"], u
    record_property("worst_decode_abs_error", worst_dec)


@pytest.mark.parametrize("name", ["batched", "long"])
def test_full_size_decode_run_with_append(name):
    """The decode protocol of the two serving workloads at full size: max_new_tokens steps (128 / 256), each appending
    one row to every segment (Eq. 4) and attending over the grown cache (Eq. 5). Lengths grow by one per step, the
    appended rows are the steps' k_new / v_new bit for bit on every unit, the attention output matches the oracle at
    the first, a middle and the last step on sampled units, and one step more is refused with MADAKV_ECAPACITY."""
    wl = synth.CONFIGS[name]
    inp = synth.make_inputs(wl, device="cuda")
    cfg = config_of(wl)
    cap = wl.units * (min(wl.n, 2 * wl.budget) + wl.max_new_tokens)
    buf = mk.EvictionBuffers(cfg, cap)
    buf.run_eviction(inp["q_win"], inp["k"], inp["v"], inp["mask"], inp["seq_len"], inp["budget"])
    assert mk.madakv_poll_status(buf.ws) == 0
    len0 = buf.kept_len.clone()
    seg_off = buf.seg_off.cpu().numpy()
    T = wl.max_new_tokens
    rng = np.random.RandomState(3)
    sample = sorted(set(rng.choice(wl.units, size=5, replace=False).tolist() + [0, wl.units - 1]))
    new_k = torch.empty((T, wl.units, wl.d), dtype=torch.bfloat16, device="cuda")
    new_v = torch.empty_like(new_k)
    for t in range(T):
        q, kn, vn = synth.make_decode_step(wl, t, device="cuda")
        new_k[t], new_v[t] = kn.view(wl.units, wl.d), vn.view(wl.units, wl.d)
        buf.run_decode(q, kn, vn)
        if t in (0, T // 2, T - 1):
            assert mk.madakv_poll_status(buf.ws) == 0
            assert torch.equal(buf.kept_len, len0 + (t + 1))
            out = buf.out.float().cpu().numpy().reshape(wl.B * wl.L, wl.Hq, wl.d)
            lens = buf.kept_len.cpu().numpy()
            q3 = q.view(wl.B * wl.L, wl.Hq, wl.d)
            for u in sample:
                a, b = int(seg_off[u]), int(seg_off[u]) + int(lens[u])
                bl, h = divmod(u, wl.Hkv)
                heads = slice(h * wl.g, (h + 1) * wl.g)
                rc, want_o, _ = oracle.decode(1, to_np(q3[bl, heads]).reshape(1, 1, wl.g, wl.d), None, None,
                                              to_np(buf.k_c[a:b]), to_np(buf.v_c[a:b]), np.array([0, b - a], np.int64),
                                              np.array([b - a], np.int32), Hkv=1)
                assert np.abs(out[bl, heads] - want_o.reshape(wl.g, wl.d)).max() <= DEC_ATOL["bf16"], (t, u)
    assert mk.madakv_poll_status(buf.ws) == 0
    # the appended rows of every unit: row len0[u] + t of the segment is step t's k_new / v_new
    rows = (buf.seg_off[:-1] + len0).view(1, wl.units) + torch.arange(T, device="cuda").view(T, 1)
    assert torch.equal(buf.k_c[rows.reshape(-1)].view(T, wl.units, wl.d), new_k)
    assert torch.equal(buf.v_c[rows.reshape(-1)].view(T, wl.units, wl.d), new_v)
    # the headroom is used up: one more append is refused and changes nothing
    lens, kc = buf.kept_len.clone(), buf.k_c.clone()
    q, kn, vn = synth.make_decode_step(wl, T, device="cuda")
    buf.run_decode(q, kn, vn)
    assert mk.madakv_poll_status(buf.ws) == mk.ECAPACITY
    assert torch.equal(buf.kept_len, lens) and torch.equal(buf.k_c, kc)


@pytest.mark.parametrize("path", ["auto", "twophase"])
def test_score_with_logits_far_apart(path, monkeypatch):
    # a softmax scale of 6 instead of 1/sqrt(d) spreads the logits over several hundred binades: sums of exp2 taken
    # against anything but the true row maximum overflow, so the cluster kernel has to fall back to its exact
    # two-sweep statistics; psi is then close to one-hot per window row
    if path == "twophase":
        monkeypatch.setenv("MADAKV_SCORE_PATH", "twophase")
    wl = synth.scaled(TINY, dtype="bf16", B=2, L=2, Hq=4, Hkv=4, d=128, n=3000, w=32, budget=300, theta=0.3)
    inp = make_case(wl)
    cfg = config_of(wl, softmax_scale=6.0)
    g = dev(inp)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl), want_lse=True)
    mk.madakv_score(cfg, g["q_win"], g["k"], g["seq_len"], buf.lse, buf.psi, buf.ws)
    assert mk.madakv_poll_status(buf.ws) == 0
    want, want_lse = oracle.score(1, to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["seq_len"]), scale=6.0,
                                  want_lse=True)
    got = buf.psi.cpu().numpy()
    assert np.isfinite(got).all()
    # logits of several hundred: fp32 accumulation gives ~1e-4 relative on the big entries
    psi_close(got, want, PSI_RTOL, atol=1e-6)
    np.testing.assert_allclose(got.sum(-1), wl.g * wl.w, rtol=1e-4)
    np.testing.assert_allclose(buf.lse.cpu().numpy(), want_lse, rtol=1e-5, atol=1e-3)
