"""The multi-GPU launch of bench.py on CPU: two gloo ranks. The path shards over independent sequences (one batch
per rank, no data-path collective), so what N > 1 adds is host logic: every rank's own seeded batch, the MAX / SUM
reductions behind the whole-job figures, and the claim that a sequence's result does not depend on which other
sequences share its batch (checked with the oracle: each rank evicts one half of a batch, the halves equal the
oracle's result on the whole batch)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

WORLD = 2


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _evict(oracle, wl, inp, rows):
    """Oracle stages 1-4a on the sequences `rows` of a batch; returns (budgets, kept_len, kept index lists)."""
    from helpers import dcode, to_np

    q, k = to_np(inp["q_win"][rows]), to_np(inp["k"][rows])
    mask, sl, bud = to_np(inp["mask"][rows]), to_np(inp["seq_len"][rows]), to_np(inp["budget"][rows])
    psi = oracle.score(dcode(wl), q, k, sl).astype(np.float32)
    al = oracle.allocate(psi, mask, sl, bud, float(np.float32(wl.theta)))
    cap = len(rows) * wl.L * wl.Hkv * (wl.n + wl.max_new_tokens)
    rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"], headroom=wl.max_new_tokens,
                                                    capacity=cap)
    assert rc == 0
    lists = [kept_idx[seg_off[u]:seg_off[u] + kept_len[u]].copy() for u in range(len(kept_len.reshape(-1)))]
    return al["budgets"], kept_len, lists


def _rank_main(rank, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(WORLD))
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        import bench
        import oracle
        from paper_2506_15724_b200 import synth

        tiny = synth.scaled(synth.CONFIGS["tiny"], B=4, L=2, n=389, budget=60, theta=0.3)
        # (1) every rank draws its own batch
        mine = synth.make_inputs(bench.rank_workload(tiny, rank))
        digest = torch.tensor([float(mine["k"].double().sum())], dtype=torch.float64)
        both = [torch.zeros_like(digest) for _ in range(WORLD)]
        dist.all_gather(both, digest)
        assert float(both[0]) != float(both[1])
        # (2) whole-job figures: slowest rank's time, all ranks' tokens
        tokens = int(mine["seq_len"].sum())
        total_ms, tokens_all = bench.reduce_over_ranks(10.0 * (rank + 1), tokens, torch.device("cpu"), WORLD)
        assert total_ms == 20.0 and tokens_all == WORLD * tokens
        assert bench.job_throughput(total_ms, 4, tokens_all) == tokens_all / 5e-3
        # (3) sequences are independent: rank r evicts sequences [2r, 2r + 2) of one shared batch
        shared = synth.make_inputs(tiny)
        rows = list(range(2 * rank, 2 * rank + 2))
        bud_r, len_r, lists_r = _evict(oracle, tiny, shared, rows)
        bud_all, len_all, lists_all = _evict(oracle, tiny, shared, list(range(tiny.B)))
        per = tiny.L * tiny.Hkv
        assert np.array_equal(bud_r, bud_all[rows])
        assert np.array_equal(len_r.reshape(-1), len_all.reshape(-1)[rows[0] * per:(rows[-1] + 1) * per])
        for a, b in zip(lists_r, lists_all[rows[0] * per:(rows[-1] + 1) * per]):
            assert np.array_equal(a, b)
        out.put((rank, "ok"))
    except BaseException as e:  # report instead of hanging the parent
        import traceback

        out.put((rank, traceback.format_exc()))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_batches_and_reduce():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, port, out)) for r in range(WORLD)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=240) for _ in range(WORLD))
    for p in procs:
        p.join(timeout=60)
    assert results == {0: "ok", 1: "ok"}, results
