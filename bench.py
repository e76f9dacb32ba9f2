#!/usr/bin/env python
"""Benchmark of the MadaKV eviction pass on B200: prompt tokens evicted per second, decode-step latency and the
fraction of the HBM roofline, with the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llava] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic input: stages 1-4 (score, allocate, select,
compact) for every layer and head, then one decode step (append + attention over the ragged cache, all layers).
With N > 1 (torchrun, one rank per GPU) every rank runs its own batch (different seed): the path shards over
independent sequences with no data-path collective, so scaling is weak and the value is N batches / slowest rank.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_15724_b200 import synth  # noqa: E402

METRIC = "prompt tokens evicted/sec"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while the timed region runs (read-only NVML queries
    from a thread, every ~2 ms; nvidia-smi polling as a fallback when NVML cannot be loaded)."""
    SMI_FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                  "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                  "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        import threading

        self.samples, self.reasons, self.max_mhz, self.proc, self.thread = [], set(), None, None, None
        self._stop = threading.Event()
        try:
            import pynvml

            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            bits = {
                "hw_slowdown": getattr(pynvml, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(pynvml, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(pynvml, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(pynvml, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            }

            def loop():
                while not self._stop.is_set():
                    try:
                        self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        r = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                        for name, bit in bits.items():
                            if r & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    time.sleep(0.002)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
        except Exception:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.proc = subprocess.Popen(
                    ["nvidia-smi", "-i", str(index), f"--query-gpu={self.SMI_FIELDS}", "--format=csv,noheader,nounits",
                     "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
            except Exception:
                self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "source": "nvml"}
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
        elif self.proc is not None:
            out["source"] = "nvidia-smi"
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.tmp.flush()
            self.tmp.seek(0)
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            mx = []
            for line in self.tmp.read().splitlines():
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    self.samples.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        self.reasons.add(nm)
            self.tmp.close()
            os.unlink(self.tmp.name)
            if mx:
                out["sm_max_mhz"] = max(mx)
        if self.samples:
            sm = sorted(self.samples)
            out.update(sm_mhz=sm[len(sm) // 2], reasons=sorted(self.reasons), samples=len(sm))
        return out


def rank_workload(wl, rank):
    """The batch of rank `rank`: same shape, its own seed. The path shards over independent sequences, so ranks
    exchange nothing on the data path."""
    return synth.scaled(wl, seed=wl.seed + 1000 * rank)


def reduce_over_ranks(total_ms, tokens, device, world):
    """Whole-job figures from per-rank ones: the slowest rank's time (MAX) and all ranks' prompt tokens (SUM). The
    only collectives of a multi-GPU run; any backend (NCCL on GPUs, gloo in the CPU tests)."""
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.int64, device=device)
    if world > 1:
        import torch.distributed as dist

        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def job_throughput(total_ms, steps, tokens_all_ranks):
    """Prompt tokens of all ranks per second of the slowest rank's step."""
    return tokens_all_ranks / (total_ms / steps * 1e-3)


def cpu_oracle_leg(wl, seconds_target=15.0):
    """The oracle, as it stands, on a bounded sample of the workload: the first layers of the same inputs (all of
    them when the whole workload fits the time target), repeated until about `seconds_target` of CPU work is done."""
    import numpy as np

    import oracle

    def to_np(t):
        t = t.detach().cpu().contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()

    code = 0 if wl.dtype == "f32" else 1

    def prepare(layers):
        sub = synth.scaled(wl, L=layers)
        inp = synth.make_inputs(sub)
        q, k, v = to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["v"])
        mask, sl, bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
        dq, kn, vn = [to_np(t) for t in synth.make_decode_step(sub, 0)]
        cap = sub.units * (sub.n + sub.max_new_tokens)

        def one_pass():
            psi = oracle.score(code, q, k, sl).astype(np.float32)
            al = oracle.allocate(psi, mask, sl, bud, wl.theta)
            rc, kept_len, seg_off, kept_idx = oracle.select(psi, mask, sl, al["budgets"], headroom=sub.max_new_tokens,
                                                            capacity=cap)
            k_c, v_c = oracle.compact(code, k, v, kept_idx, seg_off, kept_len, cap)
            oracle.decode(code, dq, kn, vn, k_c, v_c, seg_off, kept_len, Hkv=sub.Hkv)

        return sub, one_pass, int(sl.sum())

    sub, one_pass, tokens = prepare(1)
    t0 = time.perf_counter()
    one_pass()
    t1 = time.perf_counter() - t0
    layers = int(max(1, min(wl.L, seconds_target / 2 / max(t1, 1e-3))))
    if layers > 1:
        sub, one_pass, tokens = prepare(layers)
    reps = int(max(1, min(16, seconds_target / max(t1 * layers, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        one_pass()
    dt = (time.perf_counter() - t0) / reps
    value = tokens * (layers / wl.L) / dt  # tokens/s of the full-depth pass at the sampled layers' rate
    return {
        "value": value, "unit": UNIT, "cores": oracle.hardware_threads(), "kind": "oracle",
        "sample": f"{layers} of {wl.L} layers of workload '{wl.name}' (all {sub.Hkv} KV heads, all {wl.n} tokens, "
                  f"one decode step), {reps} repetition(s), {dt:.2f} s each; value scaled by layers/{wl.L}",
    }, dt


def workload_config(wl):
    """The `config` object of the JSON line: the same for both arms."""
    k_gb = wl.units * wl.n * wl.d * wl.elem_bytes / 1e9
    return {"workload": wl.name, "batch": wl.B, "layers": wl.L, "q_heads": wl.Hq, "kv_heads": wl.Hkv,
            "head_dim": wl.d, "context": wl.n, "window": wl.w, "budget_per_head": wl.budget, "theta": wl.theta,
            "l2": "inputs larger than L2 (K alone is %.2f GB)" % k_gb,
            "step": "stages 1-4 + one all-layer decode step with append"}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    info = None
    for i in range(args.warmup + args.steps):
        info, dt = cpu_oracle_leg(wl, seconds_target=4.0)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    line = {
        "impl": "reference", "metric": METRIC, "value": info["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": dict(workload_config(wl), note="CPU oracle on a bounded sample; each step = the sample once"),
        "cpu_baseline": info,
        "e2e": {"value": info["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llava", choices=list(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-full-cache", action="store_true", help="skip the full-cache decode comparison")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-single-pass", action="store_true", help="skip the timing of madakv_score_lse (profiling runs)")
    ap.add_argument("--layers", type=int, default=0, help="profiling only: run a reduced-depth copy of the workload")
    ap.add_argument("--budget", type=int, default=0, help="budget sweeps: another per-head budget than the workload's")
    ap.add_argument("--theta", type=float, default=0.0, help="budget sweeps: the Eq. 9 threshold calibrated for --budget "
                    "(python -m oracle.calibrate_theta workload:budget)")
    args = ap.parse_args()
    wl = synth.CONFIGS[args.workload]
    if args.layers > 0:
        wl = synth.scaled(wl, L=args.layers, name=f"{wl.name}[L={args.layers}]")
    if args.budget > 0:
        wl = synth.scaled(wl, budget=args.budget, theta=args.theta if args.theta > 0 else wl.theta,
                          name=f"{wl.name}[budget={args.budget}]")
    if args.impl == "reference":
        run_reference(args, wl)
        return
    args.warmup = max(args.warmup, 3)

    from paper_2506_15724_b200 import binding as mk
    from paper_2506_15724_b200 import build as mkbuild

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        mkbuild.build()
    if world > 1:
        dist.barrier()
    mk.lib()

    wl_r = rank_workload(wl, rank)  # every rank its own batch
    dev = torch.device("cuda", local)
    inp = synth.make_inputs(wl_r, device=dev)
    cfg = mk.make_config(wl.torch_dtype, wl.B, wl.L, wl.Hq, wl.Hkv, wl.d, wl.n, wl.w, max_new_tokens=wl.max_new_tokens,
                         theta=wl.theta)
    cap = wl.units * (min(wl.n, 2 * wl.budget) + wl.max_new_tokens)
    buf = mk.EvictionBuffers(cfg, cap, device=dev)
    n_dec = 4
    dec = [synth.make_decode_step(wl_r, s, device=dev) for s in range(n_dec)]
    tokens = int(inp["seq_len"].sum().item())

    def step(i, ev=None):
        c = buf.cfg
        q, kn, vn = dec[i % n_dec]
        if ev:
            ev[0].record()
        mk.madakv_score(c, inp["q_win"], inp["k"], inp["seq_len"], None, buf.psi, buf.ws)
        if ev:
            ev[1].record()
        mk.madakv_allocate(c, buf.psi, inp["mask"], inp["seq_len"], inp["budget"], buf.mass, buf.pref, buf.demand,
                           buf.phi, buf.budgets, buf.ws)
        if ev:
            ev[2].record()
        mk.madakv_select(c, buf.psi, inp["mask"], inp["seq_len"], buf.budgets, buf.kept_len, buf.seg_off, buf.kept_idx,
                         buf.ws)
        if ev:
            ev[3].record()
        mk.madakv_compact(c, inp["k"], inp["v"], buf.kept_idx, buf.seg_off, buf.kept_len, buf.k_c, buf.v_c, buf.ws)
        if ev:
            ev[4].record()
        mk.madakv_decode_attn(c, -1, q, kn, vn, buf.k_c, buf.v_c, buf.seg_off, buf.kept_len, buf.out, buf.lse_dec,
                              buf.ws)
        if ev:
            ev[5].record()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    sync_all()
    site = int(buf.ws[4:8].view(torch.int32).item())  # diagnostic word beside the status (which wait gave up)
    status = mk.madakv_poll_status(buf.ws)
    if status != 0:
        raise SystemExit(f"device status {mk.madakv_status_string(status)} after warm-up (wait site {site & 255}, "
                         f"block {site >> 8})")

    sampler = ClockSampler(local) if rank == 0 else None
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    sync_all()
    for i in range(args.steps):
        step(i, evs[i])
    sync_all()
    clocks = sampler.stop() if sampler else None
    total_ms = evs[0][0].elapsed_time(evs[-1][5])
    stage_ms = [sum(e[j].elapsed_time(e[j + 1]) for e in evs) / args.steps for j in range(5)]
    total_ms, tokens_all = reduce_over_ranks(total_ms, tokens, dev, world)
    ms_per_step = total_ms / args.steps
    value = job_throughput(total_ms, args.steps, tokens_all)

    # bytes the method must move (algorithmic): K read once; kept K/V rows read and written; decode reads K_c + V_c
    rows = int(buf.kept_len.sum().item()) - wl.units  # kept rows before this step's append
    e = wl.elem_bytes
    k_bytes = wl.units * wl.n * wl.d * e
    compact_bytes = 4 * rows * wl.d * e
    decode_bytes = 2 * (rows + wl.units) * wl.d * e
    peak, peak_kind = measured_peaks()
    score_gbs = k_bytes / (stage_ms[0] * 1e-3) / 1e9
    pass_ms = sum(stage_ms[:4])
    pass_gbs = (k_bytes + compact_bytes) / (pass_ms * 1e-3) / 1e9
    dec_gbs = decode_bytes / (stage_ms[4] * 1e-3) / 1e9

    # The dominant kernel is the score stage. With up to 64 window rows per KV head it is bound by reading K once
    # (HBM). With more (the grouped-query workloads) every key meets g * w exponentials in each of the two passes and
    # the special-function unit binds first: 16 exp2 per clock and SM, at the maximum SM clock.
    if wl.g * wl.w <= 64:
        roofline = {"bound": "hbm", "kernel": "score stage (stage 1)", "achieved": score_gbs, "peak": peak,
                    "unit": "GB/s", "frac": score_gbs / peak, "traffic": TRAFFIC.get(wl.name),
                    "peak_kind": peak_kind, "algorithmic_bytes": k_bytes}
    else:
        props = torch.cuda.get_device_properties(dev)
        sm_ghz = (clocks or {}).get("sm_max_mhz") or 1965.0
        exp_peak = props.multi_processor_count * 16 * sm_ghz * 1e6 / 1e12
        n_exp = 2.0 * wl.g * wl.w * float(inp["seq_len"].sum().item()) * wl.L * wl.Hkv  # two passes over every logit
        achieved = n_exp / (stage_ms[0] * 1e-3) / 1e12
        roofline = {"bound": "alu", "kernel": "score stage (stage 1)", "achieved": achieved, "peak": exp_peak,
                    "unit": "Texp2/s", "frac": achieved / exp_peak, "traffic": None,
                    "peak_kind": "derived: SMs x 16 exp2 per clock x max SM clock", "algorithmic_exp2": n_exp,
                    "hbm": {"achieved": score_gbs, "peak": peak, "unit": "GB/s", "frac": score_gbs / peak,
                            "algorithmic_bytes": k_bytes}}

    # ---- end to end through the C ABI with host buffers (pinned): H2D of the step's inputs, D2H of its result
    h2d = d2h = 0
    if not args.no_e2e:
        host = {k: v.cpu().pin_memory() for k, v in inp.items()}
        hdec = [tuple(x.cpu().pin_memory() for x in d) for d in dec]
        h_out = torch.empty_like(buf.out, device="cpu").pin_memory()
        h_len = torch.empty_like(buf.kept_len, device="cpu").pin_memory()
        h2d = sum(v.numel() * v.element_size() for v in host.values()) + sum(x.numel() * x.element_size()
                                                                             for x in hdec[0])
        d2h = h_out.numel() * h_out.element_size() + h_len.numel() * h_len.element_size()

    def e2e_step(i):
        for k_, v_ in host.items():
            inp[k_].copy_(v_, non_blocking=True)
        for dst, src in zip(dec[i % n_dec], hdec[i % n_dec]):
            dst.copy_(src, non_blocking=True)
        step(i)
        h_out.copy_(buf.out, non_blocking=True)
        h_len.copy_(buf.kept_len, non_blocking=True)

    e2e_ms = e2e_value = None
    if not args.no_e2e:
        e2e_step(0)
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.e2e_steps):
            e2e_step(i)
        e1.record()
        sync_all()
        e2e_total, _ = reduce_over_ranks(e0.elapsed_time(e1), tokens, dev, world)
        e2e_ms = e2e_total / args.e2e_steps
        e2e_value = job_throughput(e2e_total, args.e2e_steps, tokens_all)

    # ---- decode-step latency: compressed cache (per step, all layers in one call) against the full cache
    def time_decode(b, steps=20):
        for i in range(3):
            q, kn, vn = dec[i % n_dec]
            mk.madakv_decode_attn(b.cfg, -1, q, None, None, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)
        torch.cuda.synchronize()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(steps):
            q, kn, vn = dec[i % n_dec]
            mk.madakv_decode_attn(b.cfg, -1, q, None, None, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)
        z.record()
        torch.cuda.synchronize()
        return a.elapsed_time(z) / steps * 1e3

    # ---- stage 1 in a single pass, for callers that bring the prefill's log-sum-exps (here: those of madakv_score)
    def time_single_pass(steps=20):
        lse = torch.empty((wl.B, wl.L, wl.Hq, wl.w), dtype=torch.float32, device=dev)
        psi1 = torch.empty_like(buf.psi)
        mk.madakv_score(buf.cfg, inp["q_win"], inp["k"], inp["seq_len"], lse, buf.psi, buf.ws)
        for _ in range(3):
            mk.madakv_score_lse(buf.cfg, inp["q_win"], inp["k"], inp["seq_len"], lse, psi1, buf.ws)
        torch.cuda.synchronize()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            mk.madakv_score_lse(buf.cfg, inp["q_win"], inp["k"], inp["seq_len"], lse, psi1, buf.ws)
        z.record()
        torch.cuda.synchronize()
        return a.elapsed_time(z) / steps

    single_ms = None if args.no_single_pass else time_single_pass()

    # ---- the layer-by-layer order (a layer is evicted right after its prefill): per layer single-pass scoring with
    # the prefill's log-sum-exps, madakv_allocate_layer carrying phi, selection and compaction of that layer
    def time_streamed(steps=5):
        cfg1 = mk.make_config(wl.torch_dtype, wl.B, 1, wl.Hq, wl.Hkv, wl.d, wl.n, wl.w,
                              max_new_tokens=wl.max_new_tokens, theta=wl.theta)
        one = mk.EvictionBuffers(cfg1, cap // wl.L + wl.B * wl.Hkv, device=dev)
        lse = torch.empty((wl.B, wl.L, wl.Hq, wl.w), dtype=torch.float32, device=dev)
        mk.madakv_score(buf.cfg, inp["q_win"], inp["k"], inp["seq_len"], lse, buf.psi, buf.ws)
        lse_l = [lse[:, l:l + 1].contiguous() for l in range(wl.L)]
        phi = torch.zeros((wl.B, wl.L), dtype=torch.float64, device=dev)

        def one_pass():
            for l in range(wl.L):
                q_l, k_l, v_l = inp["q_win"][:, l:l + 1], inp["k"][:, l:l + 1], inp["v"][:, l:l + 1]
                mk.madakv_score_lse(cfg1, q_l, k_l, inp["seq_len"], lse_l[l], one.psi, one.ws)
                mk.madakv_allocate_layer(buf.cfg, l, one.psi, inp["mask"], inp["seq_len"], inp["budget"], one.mass,
                                         one.pref, one.demand, phi, one.budgets, buf.ws)
                mk.madakv_select(cfg1, one.psi, inp["mask"], inp["seq_len"], one.budgets, one.kept_len, one.seg_off,
                                 one.kept_idx, one.ws)
                mk.madakv_compact(cfg1, k_l, v_l, one.kept_idx, one.seg_off, one.kept_len, one.k_c, one.v_c, one.ws)

        for _ in range(2):
            one_pass()
        torch.cuda.synchronize()
        if mk.madakv_poll_status(one.ws) != 0 or mk.madakv_poll_status(buf.ws) != 0:
            return None
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            one_pass()
        z.record()
        torch.cuda.synchronize()
        return a.elapsed_time(z) / steps

    streamed_ms = None if args.no_single_pass else time_streamed()

    decode_us = {"compressed": time_decode(buf), "full": None,
                 "compressed_rows_per_head": (rows + wl.units) / wl.units}
    if not args.no_full_cache and rank == 0:
        full = mk.EvictionBuffers(cfg, wl.units * (wl.n + wl.max_new_tokens), device=dev)
        big = torch.full_like(inp["budget"], wl.n)
        full.run_eviction(inp["q_win"], inp["k"], inp["v"], inp["mask"], inp["seq_len"], big)
        torch.cuda.synchronize()
        decode_us["full"] = time_decode(full, steps=5)
        del full
    site = int(buf.ws[4:8].view(torch.int32).item())
    status = mk.madakv_poll_status(buf.ws)
    if status != 0:
        raise SystemExit(f"device status {mk.madakv_status_string(status)} after the timed region (wait site "
                         f"{site & 255}, block {site >> 8})")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu, _ = cpu_oracle_leg(wl)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": workload_config(wl),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": args.steps * launches_per_step(wl),
        "roofline": roofline,
        "stages_ms": dict(zip(["score", "allocate", "select", "compact", "decode"], stage_ms)),
        "eviction_pass": {"ms": pass_ms, "tokens_per_s": tokens / (pass_ms * 1e-3), "algorithmic_bytes":
                          k_bytes + compact_bytes, "gbs": pass_gbs, "frac_of_measured_peak": pass_gbs / peak,
                          "frac_of_8TBs": pass_gbs / 8000.0, "kept_rows": rows},
        "decode": {"us_per_step": decode_us, "algorithmic_bytes": decode_bytes, "gbs_in_step": dec_gbs,
                   "frac_of_measured_peak_in_step": dec_gbs / peak,
                   "gbs_alone": decode_bytes / (decode_us["compressed"] * 1e-6) / 1e9},
        "single_pass_score": None if single_ms is None else {
            "ms": single_ms, "gbs": k_bytes / (single_ms * 1e-3) / 1e9,
            "frac_of_measured_peak": k_bytes / (single_ms * 1e-3) / 1e9 / peak,
            "note": "madakv_score_lse: stage 1 with the rows' log-sum-exps supplied; not part of the step"},
        "streamed_pass": None if streamed_ms is None else {
            "ms": streamed_ms, "tokens_per_s": tokens / (streamed_ms * 1e-3), "launches": wl.L * 7,
            "note": "stages 1-4 layer by layer (madakv_score_lse, madakv_allocate_layer, select and compact with "
                    "one-layer configs), launch-bound at this depth; not part of the step"},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def launches_per_step(wl):
    """Kernels of this library launched by one step: score 1 (bf16 with g * w <= 64: one tensor-core kernel) or 3
    (bf16 with g * w <= 256: pass 1, merge, pass 2; otherwise the three fp32 kernels), allocate 2, select 2,
    compact 1, decode 3 (append, partial, merge)."""
    one_kernel = wl.dtype == "bf16" and wl.g * wl.w <= 64
    return (1 if one_kernel else 3) + 2 + 2 + 1 + 3


# dram bytes (read + write) per launch of the dominant kernel (score_cluster), per workload, from the ncu capture
# summarised in profiles/all_kernels_llava.md: 274.2 MB measured on the 4-layer case, times 8 for the 32 layers
# (traffic grows with the number of units); None = not captured
TRAFFIC = {"llava": 8 * 274.2e6}

if __name__ == "__main__":
    main()
