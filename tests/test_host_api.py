"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol, and rejects bad
arguments before any kernel launch."""
import ctypes
import os
import re

import pytest

from paper_2506_15724_b200 import binding as mk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = ctypes.c_void_p(0x10000)  # aligned, never dereferenced: every case below fails validation first


@pytest.fixture(scope="module")
def lib():
    from paper_2506_15724_b200 import build

    build.build()
    return mk.lib()


def _cfg(**kw):
    base = dict(dtype=mk.MADAKV_BF16, batch=1, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=128, max_seq_len=256,
                window=8)
    base.update(kw)
    return mk.make_config(**base)


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "madakv.h")).read()
    declared = set(re.findall(r"\b(madakv_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(mk.EXPORTS)
    assert lib.madakv_abi_version() == 4
    assert mk.madakv_status_string(mk.ECAPACITY) == "ragged cache capacity exceeded"


def test_workspace_bytes_and_config_validation(lib):
    assert mk.madakv_workspace_bytes(_cfg()) > 256
    bad = [
        (dict(head_dim=96), mk.EUNSUPPORTED),
        (dict(dtype=7), mk.EUNSUPPORTED),
        (dict(n_q_heads=5), mk.ESHAPE),
        (dict(batch=0), mk.ESHAPE),
        (dict(window=0), mk.ESHAPE),
        (dict(theta=1.5), mk.EINVAL),
        (dict(causal=2), mk.EINVAL),
        (dict(hcc_mode=9), mk.EINVAL),
        (dict(max_new_tokens=-1), mk.ESHAPE),
        (dict(pool_kernel=4), mk.EINVAL),       # the pooling width is odd
        (dict(pool_kernel=0), mk.EINVAL),
        (dict(pool_kernel=17), mk.EUNSUPPORTED),
        (dict(keep_window=2), mk.EINVAL),
    ]
    assert mk.madakv_workspace_bytes(_cfg(pool_kernel=7, keep_window=1)) > 256
    for kw, code in bad:
        with pytest.raises(mk.MadakvError) as e:
            mk.madakv_workspace_bytes(_cfg(**kw))
        assert e.value.code == code, kw
    c = _cfg()
    c.struct_size = 12
    with pytest.raises(mk.MadakvError) as e:
        mk.madakv_workspace_bytes(c)
    assert e.value.code == mk.EINVAL


def test_entry_points_reject_bad_arguments_before_launch(lib):
    c = _cfg()
    st = mk.MadakvStrides(1, 1, 1, 128)
    good = mk.MadakvStrides(2 * 4 * 8 * 128, 4 * 8 * 128, 8 * 128, 128)
    cref = ctypes.byref(c)
    need = mk.madakv_workspace_bytes(c)
    odd = ctypes.c_void_p(0x10004)
    # null pointers
    assert lib.madakv_score(cref, None, good, FAKE, good, FAKE, None, FAKE, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_allocate(cref, FAKE, None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_select(cref, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, 10, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_compact(cref, FAKE, FAKE, good, FAKE, FAKE, FAKE, FAKE, None, 10, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_decode_attn(cref, -1, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE, 10, FAKE, None, FAKE, need,
                                  None) == mk.EINVAL
    # the single-pass scoring needs its normalisers; the per-layer allocation a layer inside the depth
    assert lib.madakv_score_lse(cref, FAKE, good, FAKE, good, FAKE, None, FAKE, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_score_lse(cref, FAKE, good, FAKE, good, FAKE, FAKE, FAKE, FAKE, need - 1, None) == mk.EWORKSPACE
    assert lib.madakv_allocate_layer(cref, 2, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need,
                                     None) == mk.ESHAPE
    assert lib.madakv_allocate_layer(cref, -1, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need,
                                     None) == mk.ESHAPE
    assert lib.madakv_allocate_layer(cref, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, FAKE, need,
                                     None) == mk.EINVAL
    # the budget-free half of the per-layer allocation needs its score array; the other half may go without
    assert lib.madakv_demand_layer(cref, None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need, None) == mk.EINVAL
    assert lib.madakv_demand_layer(cref, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need - 1, None) == mk.EWORKSPACE
    assert lib.madakv_allocate_layer(cref, 0, None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, need - 1,
                                     None) == mk.EWORKSPACE
    # misaligned pointer / stride
    assert lib.madakv_score(cref, odd, good, FAKE, good, FAKE, None, FAKE, FAKE, need, None) == mk.EALIGN
    assert lib.madakv_score(cref, FAKE, st, FAKE, good, FAKE, None, FAKE, FAKE, need, None) == mk.EALIGN
    assert lib.madakv_compact(cref, FAKE, FAKE, good, FAKE, FAKE, FAKE, odd, FAKE, 10, FAKE, need, None) == mk.EALIGN
    # workspace too small / missing / misaligned
    assert lib.madakv_score(cref, FAKE, good, FAKE, good, FAKE, None, FAKE, FAKE, need - 1, None) == mk.EWORKSPACE
    assert lib.madakv_score(cref, FAKE, good, FAKE, good, FAKE, None, FAKE, None, need, None) == mk.EINVAL
    assert lib.madakv_select(cref, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 10, ctypes.c_void_p(0x10010), need,
                             None) == mk.EALIGN
    # capacity and layer range
    assert lib.madakv_select(cref, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 0, FAKE, need, None) == mk.ECAPACITY
    assert lib.madakv_decode_attn(cref, 2, FAKE, None, None, FAKE, FAKE, FAKE, FAKE, 10, FAKE, None, FAKE, need,
                                  None) == mk.ESHAPE
    # bad config reaches every entry point
    b = _cfg(head_dim=80)
    assert lib.madakv_compact(ctypes.byref(b), FAKE, FAKE, good, FAKE, FAKE, FAKE, FAKE, FAKE, 10, FAKE, need,
                              None) == mk.EUNSUPPORTED
    assert lib.madakv_poll_status(None, None, None) == mk.EINVAL
