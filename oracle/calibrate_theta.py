"""Finds, for every benchmark workload, the Eq. 9 threshold theta at which the layer-1 demand mean_h(k_v + k_t)
matches the nominal per-head budget (bisection on the CPU oracle; inputs from the seeded generator).

The paper gives theta no value; on synthetic Gaussian logits an arbitrary theta would make the layer compensation
of Eq. 10-11 run into its clamps. Run once; the printed values are stored in paper_2506_15724_b200/synth.py CONFIGS.

    python -m oracle.calibrate_theta [workload | workload:budget ...]

`workload:budget` calibrates for another per-head budget than the stored one (budget sweeps of bench.py).
"""
import sys

import numpy as np
import torch

import oracle
from paper_2506_15724_b200 import synth


def to_np(t):
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def calibrate(name, budget=None):
    wl = synth.scaled(synth.CONFIGS[name], L=1)
    if budget is not None:
        wl = synth.scaled(wl, budget=int(budget))
    inp = synth.make_inputs(wl, want_v=False)
    mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
    psi = oracle.score(0 if wl.dtype == "f32" else 1, to_np(inp["q_win"]), to_np(inp["k"]), sl).astype(np.float32)
    lo, hi = 0.0, 1.0
    for _ in range(30):
        mid = 0.5 * (lo + hi)
        dem = oracle.allocate(psi, mask, sl, bud, mid)["demand"].sum(-1).mean()
        if dem < wl.budget:
            lo = mid
        else:
            hi = mid
    theta = float(np.float32(0.5 * (lo + hi)))
    dem = oracle.allocate(psi, mask, sl, bud, theta)["demand"].sum(-1).mean()
    return theta, float(dem)


if __name__ == "__main__":
    for arg in sys.argv[1:] or list(synth.CONFIGS):
        name, _, bud = arg.partition(":")
        budget = int(bud) if bud else synth.CONFIGS[name].budget
        theta, dem = calibrate(name, budget)
        print(f"{name}: theta = {theta:.6f}  (layer-1 demand {dem:.1f}, budget {budget})", flush=True)
