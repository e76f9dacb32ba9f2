"""The no-allocation decode entry point against the regular one, through the C ABI.

madakv_decode_attn_static exists for callers that cannot hand the library a workspace because they cannot allocate
device memory where they run (a plug-in inside another engine's step, a latency-critical loop). It must give the same
output as madakv_decode_attn on the same ragged cache. The scratch it uses is one array shared by all calls, so the
check is made on calls in a row with different queries: stale contents of one call must not leak into the next.
This file is collected last on purpose, and also passes when run alone in a fresh process.
"""
import pytest
import torch

from paper_2506_15724_b200 import binding as mk
from paper_2506_15724_b200 import synth
from helpers import capacity_of, config_of

pytestmark = pytest.mark.gpu

DEC_ATOL = {"bf16": 2e-2, "f32": 2e-5}
TINY = synth.CONFIGS["tiny"]
CASES = {
    "f32_d64": synth.scaled(TINY, L=2, n=1500, budget=700),
    "bf16_gqa_ragged": synth.scaled(TINY, dtype="bf16", B=2, L=3, Hq=8, Hkv=2, d=128, n=1700, w=16, budget=700,
                                    theta=0.3, n_needles=8),
}


@pytest.mark.parametrize("name", list(CASES))
def test_static_scratch_decode_matches_workspace_decode(name):
    wl = CASES[name]
    inp = {k: v.cuda() for k, v in synth.make_inputs(wl).items()}
    cfg = config_of(wl)
    buf = mk.EvictionBuffers(cfg, capacity_of(wl))
    buf.run_eviction(inp["q_win"], inp["k"], inp["v"], inp["mask"], inp["seq_len"], inp["budget"])
    assert mk.madakv_poll_status(buf.ws) == 0
    assert int(buf.kept_len.max()) > 256, "the case must span several splits"
    for step, layer in ((0, -1), (1, -1), (2, wl.L - 1)):  # calls in a row on the shared scratch
        q = synth.make_decode_step(wl, step)[0].cuda()
        want, want_lse = torch.zeros_like(buf.out), torch.zeros_like(buf.lse_dec)
        mk.madakv_decode_attn(cfg, layer, q, None, None, buf.k_c, buf.v_c, buf.seg_off, buf.kept_len, want, want_lse,
                              buf.ws)
        got, got_lse = torch.zeros_like(buf.out), torch.zeros_like(buf.lse_dec)
        mk.madakv_decode_attn_static(cfg, layer, q, buf.k_c, buf.v_c, buf.seg_off, buf.kept_len, got, got_lse)
        torch.cuda.synchronize()
        assert float((got.float() - want.float()).abs().max()) <= DEC_ATOL[wl.dtype]
        assert torch.equal(got, want) and torch.equal(got_lse, want_lse)  # same kernels: the bits agree too
        assert float(want.float().abs().max()) > 0


def test_static_scratch_limit_is_reported():
    # 64 layers * 64 query heads * 33 splits * 130 floats * 4 B > 16 MiB: refused on the host, nothing is launched
    wl = synth.scaled(TINY, dtype="bf16", L=64, Hq=64, Hkv=64, d=128, n=8192)
    cfg = config_of(wl)
    dummy = torch.zeros(4096, dtype=torch.bfloat16, device="cuda").view(-1, 128)
    off = torch.zeros(wl.units + 1, dtype=torch.int64, device="cuda")
    ln = torch.zeros(wl.units, dtype=torch.int32, device="cuda")
    with pytest.raises(mk.MadakvError) as e:
        mk.madakv_decode_attn_static(cfg, -1, dummy, dummy, dummy, off, ln, dummy, None)
    assert e.value.code == mk.ESTATIC
