#!/usr/bin/env python
"""Benchmark of the MadaKV eviction pass on B200: prompt tokens evicted per second, decode-step latency and the
fraction of the roofline, with the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload long] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic input: stages 1-4 (score, allocate, select,
compact) for every layer and head, then one decode step (append + attention over the ragged cache, all layers).
The headline (`value`, `roofline`, `e2e`, `cpu_baseline`) is measured on the largest single-GPU workload (`long`:
131072 tokens, 32 layers, 32 query / 8 KV heads, window 64); the `workloads` object of the same JSON line carries the
stage times, roofline fractions and decode latencies of every other benchmark workload (llava, qwen at budgets
1024 / 2048 / 4096, batched), each from its own timed steps.
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
NOMINAL_HBM_GBS = 8000.0
# exp2 results per clock and SM of the special-function unit: measured in the same run by the exp2-roof probe
# (paper_2506_15724_b200/csrc/probe/exp2_roof.cu, a register-only kernel of independent ex2.approx chains); this is
# the figure an earlier run of that probe gave on this machine's B200, used only if the probe cannot be run
EXP2_PER_CLK_PER_SM_RECORDED = 15.99
HEADLINE = "long"
OTHER_WORKLOADS = ("llava", "qwen1024", "qwen", "qwen4096", "batched")


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measure_exp2_roof():
    """exp2 per clock and SM from the probe binary (built with the library), and how the figure was obtained."""
    from paper_2506_15724_b200 import build as mkbuild

    try:
        out = subprocess.run([mkbuild.PROBE], capture_output=True, text=True, timeout=60).stdout
        rec = json.loads(out.strip().splitlines()[-1])
        return float(rec["exp2_per_clk_per_sm"]), "measured in this run by the exp2-roof probe", rec
    except Exception as e:  # no binary, no device, unreadable output
        return EXP2_PER_CLK_PER_SM_RECORDED, f"recorded from an earlier run of the exp2-roof probe ({type(e).__name__} now)", None


def ncu_traffic(kernel, workload):
    """DRAM bytes (read + write) per launch of `kernel` on `workload`, from the committed ncu summary table
    (profiles/dram_traffic.txt: kernel, workload, bytes per launch); None when no capture of the present kernel exists."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 3 and not line.startswith("#") and parts[0] == kernel and parts[1] == workload:
                    return float(parts[2])
    except Exception:
        pass
    return None


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


# ----------------------------------------------------------------------------------------------- CPU oracle legs
class OracleSample:
    """The oracle, as it stands, on a bounded sample of a workload: the first layers of the same seeded inputs (all
    KV heads, all tokens, one decode step). The sample is sized by time: as many layers as give every host thread a
    unit, as long as one pass stays near `seconds_per_pass`."""

    def __init__(self, wl, seconds_per_pass):
        import numpy as np

        import oracle

        self.oracle, self.np, self.wl = oracle, np, wl
        self.cores = oracle.hardware_threads()
        self.layers = 1
        self._prepare(1)
        t0 = time.perf_counter()
        self.one_pass()
        t1 = time.perf_counter() - t0
        per_layer = wl.B * wl.Hkv
        # one pass of `layers` layers takes about t1 * ceil(layers * per_layer / cores) / ceil(per_layer / cores)
        rounds1 = -(-per_layer // self.cores)
        want = 1
        for layers in range(2, wl.L + 1):
            rounds = -(-layers * per_layer // self.cores)
            if t1 * rounds / rounds1 > seconds_per_pass:
                break
            want = layers
            if layers * per_layer >= self.cores and t1 * rounds / rounds1 > seconds_per_pass / 2:
                break
        if want > 1:
            self.layers = want
            self._prepare(want)

    def _prepare(self, layers):
        np, wl = self.np, self.wl

        def to_np(t):
            t = t.detach().cpu().contiguous()
            return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()

        sub = synth.scaled(wl, L=layers)
        inp = synth.make_inputs(sub)
        self.sub = sub
        self.q, self.k, self.v = to_np(inp["q_win"]), to_np(inp["k"]), to_np(inp["v"])
        self.mask, self.sl, self.bud = to_np(inp["mask"]), to_np(inp["seq_len"]), to_np(inp["budget"])
        self.dq, self.kn, self.vn = [to_np(t) for t in synth.make_decode_step(sub, 0)]
        self.cap = sub.units * (sub.n + sub.max_new_tokens)
        self.tokens = int(self.sl.sum())
        self.threads = min(self.cores, sub.units)

    def one_pass(self):
        o, np, sub = self.oracle, self.np, self.sub
        code = 0 if sub.dtype == "f32" else 1
        psi = o.score(code, self.q, self.k, self.sl).astype(np.float32)
        al = o.allocate(psi, self.mask, self.sl, self.bud, self.wl.theta)
        rc, kept_len, seg_off, kept_idx = o.select(psi, self.mask, self.sl, al["budgets"],
                                                   headroom=sub.max_new_tokens, capacity=self.cap)
        k_c, v_c = o.compact(code, self.k, self.v, kept_idx, seg_off, kept_len, self.cap)
        o.decode(code, self.dq, self.kn, self.vn, k_c, v_c, seg_off, kept_len, Hkv=sub.Hkv)

    def timed(self, passes):
        ts = []
        for _ in range(passes):
            t0 = time.perf_counter()
            self.one_pass()
            ts.append(time.perf_counter() - t0)
        return ts

    def value(self, dt):
        """tokens/s of the full-depth pass at the sampled layers' rate"""
        return self.tokens * (self.layers / self.wl.L) / dt

    def info(self, dt, passes):
        wl = self.wl
        return {
            "value": self.value(dt), "unit": UNIT, "cores": self.threads, "kind": "oracle",
            "sample": f"{self.layers} of {wl.L} layers of workload '{wl.name}' (all {wl.Hkv} KV heads, all {wl.n} tokens "
                      f"of every sequence, one decode step), {passes} pass(es), {dt:.2f} s each on {self.threads} of "
                      f"{self.cores} host threads (one thread per unit); value scaled by layers/{wl.L}",
        }


def cpu_oracle_leg(wl, seconds_target=15.0):
    s = OracleSample(wl, seconds_per_pass=seconds_target / 2)
    passes = 2
    ts = s.timed(passes)
    dt = sum(ts) / len(ts)
    return s.info(dt, passes), dt


def workload_config(wl):
    """The `config` object of the JSON line: the same for both arms."""
    k_gb = wl.units * wl.n * wl.d * wl.elem_bytes / 1e9
    return {"workload": wl.name, "batch": wl.B, "layers": wl.L, "q_heads": wl.Hq, "kv_heads": wl.Hkv,
            "head_dim": wl.d, "context": wl.n, "window": wl.w, "budget_per_head": wl.budget, "theta": wl.theta,
            "l2": "inputs larger than L2 (K alone is %.2f GB)" % k_gb,
            "step": "stages 1-4 + one all-layer decode step with append"}


def run_reference(args, wl):
    """The reference arm: there is no reference implementation (the reference is a paper), so this arm times the
    CPU oracle, as it stands, on the host cores: each step is one pass over a bounded sample of the workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    n_pass = args.warmup + args.steps
    per_pass = max(1.0, min(6.0, 150.0 / max(n_pass, 1)))  # the whole run stays within a few minutes
    s = OracleSample(wl, seconds_per_pass=per_pass)
    s.timed(args.warmup)
    ts = s.timed(args.steps)
    dt = sum(ts) / len(ts)
    info = s.info(dt, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": info["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": workload_config(wl),
        "note": "CPU oracle on a bounded sample of the workload; each step = the sample once",
        "cpu_baseline": info,
        "e2e": {"value": info["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- the CUDA arm
def launches_per_step(wl):
    """Kernels of this library launched by one step: score 1 (bf16 with g * w <= 64: one tensor-core kernel) or 3
    (bf16 with g * w <= 256: pass 1, merge, pass 2; otherwise the three fp32 kernels), allocate 2, select 2,
    compact 1, decode 2 (partial with the append of Eq. 4 inside, merge)."""
    one_kernel = wl.dtype == "bf16" and wl.g * wl.w <= 64
    return (1 if one_kernel else 3) + 2 + 2 + 1 + 2


class Bench:
    """One workload resident on the device: inputs, buffers, and the timed legs."""

    def __init__(self, mk, wl, dev, rank, inputs=None):
        self.mk, self.wl, self.dev = mk, wl, dev
        wl_r = rank_workload(wl, rank)  # every rank its own batch
        self.inp = inputs if inputs is not None else synth.make_inputs(wl_r, device=dev)
        self.inp["budget"] = torch.full((wl.B,), wl.budget, dtype=torch.int32, device=dev)
        self.cfg = mk.make_config(wl.torch_dtype, wl.B, wl.L, wl.Hq, wl.Hkv, wl.d, wl.n, wl.w,
                                  max_new_tokens=wl.max_new_tokens, theta=wl.theta)
        self.cap = wl.units * (min(wl.n, 2 * wl.budget) + wl.max_new_tokens)
        self.buf = mk.EvictionBuffers(self.cfg, self.cap, device=dev)
        self.n_dec = 4
        self.dec = [synth.make_decode_step(wl_r, s, device=dev) for s in range(self.n_dec)]
        self.tokens = int(self.inp["seq_len"].sum().item())
        self.peak, self.peak_kind = measured_peaks()
        self.exp2_roof = None  # (exp2 per clock and SM, how obtained, probe record): set by main() once per run

    def step(self, i, ev=None):
        mk, c, buf, inp = self.mk, self.cfg, self.buf, self.inp
        q, kn, vn = self.dec[i % self.n_dec]
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

    def check_status(self, where, buf=None):
        buf = buf or self.buf
        site = int(buf.ws[4:8].view(torch.int32).item())  # diagnostic word beside the status (which wait gave up)
        status = self.mk.madakv_poll_status(buf.ws)
        if status != 0:
            raise SystemExit(f"device status {self.mk.madakv_status_string(status)} {where} on '{self.wl.name}' "
                             f"(wait site {site & 255}, block {site >> 8})")

    def timed_steps(self, steps, warmup, sync_all, sampler_index=None):
        for i in range(warmup):
            self.step(i)
        sync_all()
        self.check_status("after warm-up")
        sampler = ClockSampler(sampler_index) if sampler_index is not None else None
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(steps)]
        sync_all()
        for i in range(steps):
            self.step(i, evs[i])
        sync_all()
        clocks = sampler.stop() if sampler else None
        total_ms = evs[0][0].elapsed_time(evs[-1][5])
        stage_ms = [sum(e[j].elapsed_time(e[j + 1]) for e in evs) / steps for j in range(5)]
        self.check_status("after the timed region")
        return total_ms, stage_ms, clocks

    # ---- decode-step latency on a fixed cache, all layers in one call (the roofline form)
    def time_decode(self, b, steps=20):
        mk = self.mk
        for i in range(3):
            q, kn, vn = self.dec[i % self.n_dec]
            mk.madakv_decode_attn(b.cfg, -1, q, None, None, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)
        torch.cuda.synchronize()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(steps):
            q, kn, vn = self.dec[i % self.n_dec]
            mk.madakv_decode_attn(b.cfg, -1, q, None, None, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)
        z.record()
        torch.cuda.synchronize()
        return a.elapsed_time(z) / steps * 1e3

    # ---- the decode run of the workload: max_new_tokens steps, each appending one row per KV head (Eq. 4) and
    # attending over the grown cache (Eq. 5); per-step device times. `layerwise` issues the L dependent per-layer
    # calls a model makes (layer l + 1's query depends on layer l's output) instead of one all-layer call.
    def time_decode_run(self, b, layerwise=False, max_steps=None, graph=False):
        """Decode steps with append, one event per step. graph: one step (its L per-layer calls) is captured into a
        CUDA graph once and replayed, as a serving loop would do; the step's inputs are then the same every time."""
        mk, wl = self.mk, self.wl
        n_steps = wl.max_new_tokens if max_steps is None else min(max_steps, wl.max_new_tokens)
        keep = b.kept_len.clone()

        def one_step(q, kn, vn):
            if layerwise:
                for l in range(wl.L):
                    mk.madakv_decode_attn(b.cfg, l, q, kn, vn, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)
            else:
                mk.madakv_decode_attn(b.cfg, -1, q, kn, vn, b.k_c, b.v_c, b.seg_off, b.kept_len, b.out, None, b.ws)

        g = None
        if graph:
            one_step(*self.dec[0])  # everything the calls set up on the host has happened before the capture
            torch.cuda.synchronize()
            b.kept_len.copy_(keep)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                one_step(*self.dec[0])
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for s in range(n_steps):
            if g is not None:
                g.replay()
            else:
                one_step(*self.dec[s % self.n_dec])
            evs[s + 1].record()
        torch.cuda.synchronize()
        grown = int((b.kept_len - keep).min().item()), int((b.kept_len - keep).max().item())
        self.check_status("after the decode run", b)
        b.kept_len.copy_(keep)  # the appended rows lie in the headroom: dropping them restores the cache
        us = sorted(evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(n_steps))
        return {"steps": n_steps, "us_median": us[len(us) // 2], "us_min": us[0], "us_max": us[-1],
                "us_mean": sum(us) / len(us), "rows_appended_per_segment": grown[0] if grown[0] == grown[1] else grown}

    # ---- stage 1 in a single pass, for callers that bring the prefill's log-sum-exps (here: those of madakv_score)
    def time_single_pass(self, steps=10):
        mk, wl, buf, inp = self.mk, self.wl, self.buf, self.inp
        lse = torch.empty((wl.B, wl.L, wl.Hq, wl.w), dtype=torch.float32, device=self.dev)
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

    # ---- the layer-by-layer order (a layer is evicted right after its prefill): per layer single-pass scoring with
    # the prefill's log-sum-exps, madakv_allocate_layer carrying phi, selection and compaction of that layer.
    # Eager on one stream it is launch- and latency-bound (a layer's allocation and selection have only B * H_kv
    # blocks). The overlapped form keeps several layers in flight: scoring on one stream, allocation + selection of
    # layer l on stream l % NS, compaction on another; the dependencies score(l) -> allocate(l) -> select(l) ->
    # compact(l), phi(l) -> allocate(l + 1) and the reuse of a layer's scratch are events. The whole pass is captured
    # once into a CUDA graph and replayed, so the host's launch cost is out of the picture.
    def time_streamed(self, steps=3, overlapped=True, NS=8):
        mk, wl, buf, inp = self.mk, self.wl, self.buf, self.inp
        cfg1 = mk.make_config(wl.torch_dtype, wl.B, 1, wl.Hq, wl.Hkv, wl.d, wl.n, wl.w,
                              max_new_tokens=wl.max_new_tokens, theta=wl.theta)
        slots = NS if overlapped else 1  # layers in flight, each with its own scratch
        # a single layer may be given far more than the nominal budget by the compensation of Eq. 10-11
        per_layer = wl.B * wl.Hkv * (wl.n + wl.max_new_tokens)
        one = [mk.EvictionBuffers(cfg1, per_layer, device=self.dev) for _ in range(slots)]
        ws_side = [mk.new_workspace(buf.cfg, self.dev) for _ in range(slots)]  # allocate_layer's and select's workspace
        lse = torch.empty((wl.B, wl.L, wl.Hq, wl.w), dtype=torch.float32, device=self.dev)
        mk.madakv_score(buf.cfg, inp["q_win"], inp["k"], inp["seq_len"], lse, buf.psi, buf.ws)
        lse_l = [lse[:, l:l + 1].contiguous() for l in range(wl.L)]
        phi = torch.zeros((wl.B, wl.L), dtype=torch.float64, device=self.dev)
        torch.cuda.synchronize()

        def one_pass(main):
            if not overlapped:
                for l in range(wl.L):
                    o = one[0]
                    q_l, k_l, v_l = inp["q_win"][:, l:l + 1], inp["k"][:, l:l + 1], inp["v"][:, l:l + 1]
                    mk.madakv_score_lse(cfg1, q_l, k_l, inp["seq_len"], lse_l[l], o.psi, o.ws)
                    mk.madakv_allocate_layer(buf.cfg, l, o.psi, inp["mask"], inp["seq_len"], inp["budget"], o.mass,
                                             o.pref, o.demand, phi, o.budgets, ws_side[0])
                    mk.madakv_select(cfg1, o.psi, inp["mask"], inp["seq_len"], o.budgets, o.kept_len, o.seg_off,
                                     o.kept_idx, ws_side[0])
                    mk.madakv_compact(cfg1, k_l, v_l, o.kept_idx, o.seg_off, o.kept_len, o.k_c, o.v_c, o.ws)
                return
            side = [torch.cuda.Stream() for _ in range(slots)]
            cmp_s = torch.cuda.Stream()
            start = torch.cuda.Event()
            start.record(main)
            for st in side + [cmp_s]:
                st.wait_event(start)
            sel_done, cmp_done, alloc_done = {}, {}, {}
            for l in range(wl.L):
                o, sd = one[l % slots], side[l % slots]
                q_l, k_l, v_l = inp["q_win"][:, l:l + 1], inp["k"][:, l:l + 1], inp["v"][:, l:l + 1]
                if l - slots in sel_done:
                    main.wait_event(sel_done[l - slots])  # psi of this scratch is free once its selection has run
                mk.madakv_score_lse(cfg1, q_l, k_l, inp["seq_len"], lse_l[l], o.psi, o.ws)
                scored = torch.cuda.Event()
                scored.record(main)
                with torch.cuda.stream(sd):
                    sd.wait_event(scored)
                    # masses, preferences and demands (Eq. 6, 9) do not depend on the layer before ...
                    mk.madakv_demand_layer(buf.cfg, o.psi, inp["mask"], inp["seq_len"], o.mass, o.pref, o.demand,
                                           ws_side[l % slots])
                    if l - 1 in alloc_done:
                        sd.wait_event(alloc_done[l - 1])  # ... phi^l does (Eq. 11)
                    if l - slots in cmp_done:
                        sd.wait_event(cmp_done[l - slots])  # the scratch's kept positions were read by its compaction
                    mk.madakv_allocate_layer(buf.cfg, l, None, inp["mask"], inp["seq_len"], inp["budget"], o.mass,
                                             o.pref, o.demand, phi, o.budgets, ws_side[l % slots])
                    alloc_done[l] = torch.cuda.Event()
                    alloc_done[l].record(sd)
                    mk.madakv_select(cfg1, o.psi, inp["mask"], inp["seq_len"], o.budgets, o.kept_len, o.seg_off,
                                     o.kept_idx, ws_side[l % slots])
                    sel_done[l] = torch.cuda.Event()
                    sel_done[l].record(sd)
                with torch.cuda.stream(cmp_s):
                    cmp_s.wait_event(sel_done[l])
                    mk.madakv_compact(cfg1, k_l, v_l, o.kept_idx, o.seg_off, o.kept_len, o.k_c, o.v_c, o.ws)
                    cmp_done[l] = torch.cuda.Event()
                    cmp_done[l].record(cmp_s)
            for st in side + [cmp_s]:  # join
                e = torch.cuda.Event()
                e.record(st)
                main.wait_event(e)

        def statuses():
            return [mk.madakv_poll_status(o.ws) for o in one] + [mk.madakv_poll_status(w) for w in ws_side] + \
                   [mk.madakv_poll_status(buf.ws)]

        cap_stream = torch.cuda.Stream()
        with torch.cuda.stream(cap_stream):
            one_pass(cap_stream)  # eager once: every kernel's attributes are set before the capture
        torch.cuda.synchronize()
        if any(statuses()):
            return None
        graph = None
        if overlapped:
            try:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=cap_stream):
                    one_pass(cap_stream)
            except Exception:
                graph = None
                torch.cuda.synchronize()

        def run():
            if graph is not None:
                graph.replay()
            else:
                with torch.cuda.stream(cap_stream):
                    one_pass(cap_stream)

        run()
        torch.cuda.synchronize()
        if any(statuses()):
            return None
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        with torch.cuda.stream(cap_stream):
            a.record()
            for _ in range(steps):
                run()
            z.record()
        torch.cuda.synchronize()
        return {"ms": a.elapsed_time(z) / steps, "cuda_graph": graph is not None}

    def full_cache(self):
        """The same cache without eviction (budget = context length): what decode costs uncompressed."""
        wl = self.wl
        full = self.mk.EvictionBuffers(self.cfg, wl.units * (wl.n + wl.max_new_tokens), device=self.dev)
        big = torch.full_like(self.inp["budget"], wl.n)
        full.run_eviction(self.inp["q_win"], self.inp["k"], self.inp["v"], self.inp["mask"], self.inp["seq_len"], big)
        torch.cuda.synchronize()
        return full

    def record(self, stage_ms, clocks, args, with_streamed=True):
        """Per-workload figures of the JSON line from the timed steps and the decode legs."""
        wl, buf = self.wl, self.buf
        buf.kept_len.sub_(1)  # the last step's append lies in the headroom: dropping it restores the compacted cache
        rows = int(buf.kept_len.sum().item())  # kept rows of the pass
        e = wl.elem_bytes
        # bytes the method must move (algorithmic): K read once; kept K/V rows read and written; decode reads K_c + V_c
        k_bytes = wl.units * wl.n * wl.d * e
        compact_bytes = 4 * rows * wl.d * e
        decode_bytes = 2 * (rows + wl.units) * wl.d * e  # the step's decode reads the appended row too
        peak = self.peak
        score_gbs = k_bytes / (stage_ms[0] * 1e-3) / 1e9
        pass_ms = sum(stage_ms[:4])
        pass_gbs = (k_bytes + compact_bytes) / (pass_ms * 1e-3) / 1e9
        dec_gbs = decode_bytes / (stage_ms[4] * 1e-3) / 1e9
        # The dominant kernel is the score stage. With up to 64 window rows per KV head it is bound by reading K
        # once (HBM). With more (the grouped-query workloads) every key meets g * w exponentials in each of the two
        # passes and the special-function unit binds first: a measured 15.99 exp2 per clock and SM, at the median
        # SM clock sampled during the timed region.
        if wl.g * wl.w <= 64:
            roofline = {"bound": "hbm", "kernel": "score_cluster_kernel (stage 1)", "achieved": score_gbs, "peak": peak,
                        "unit": "GB/s", "frac": score_gbs / peak,
                        "traffic": ncu_traffic("score_cluster_kernel", wl.name),
                        "peak_kind": self.peak_kind, "algorithmic_bytes": k_bytes}
        else:
            props = torch.cuda.get_device_properties(self.dev)
            sm_mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
            per_clk, roof_how, _ = self.exp2_roof or (EXP2_PER_CLK_PER_SM_RECORDED, "recorded", None)
            exp_peak = props.multi_processor_count * per_clk * sm_mhz * 1e6 / 1e12
            n_exp = 2.0 * wl.g * wl.w * float(self.tokens) * wl.L * wl.Hkv  # two passes over every logit
            achieved = n_exp / (stage_ms[0] * 1e-3) / 1e12
            roofline = {"bound": "alu", "kernel": "score_rows_kernel pass 1 + pass 2 (stage 1)", "achieved": achieved,
                        "peak": exp_peak, "unit": "Texp2/s", "frac": achieved / exp_peak,
                        "traffic": ncu_traffic("score_rows_kernel", wl.name),
                        "peak_kind": f"{per_clk:.2f} exp2 per clock and SM ({roof_how}) x "
                                     f"{props.multi_processor_count} SMs x the median SM clock sampled in the timed "
                                     f"region ({sm_mhz:.0f} MHz)",
                        "algorithmic_exp2": n_exp,
                        "hbm": {"achieved": score_gbs, "peak": peak, "unit": "GB/s", "frac": score_gbs / peak,
                                "algorithmic_bytes": k_bytes, "peak_kind": self.peak_kind,
                                "exp2_bound_allows_frac": min(1.0, (k_bytes / (peak * 1e9)) / (n_exp / (exp_peak * 1e12)))}}
        rec = {
            "config": workload_config(wl),
            "stages_ms": dict(zip(["score", "allocate", "select", "compact", "decode"], stage_ms)),
            "roofline": roofline,
            "eviction_pass": {"ms": pass_ms, "tokens_per_s": self.tokens / (pass_ms * 1e-3),
                              "algorithmic_bytes": k_bytes + compact_bytes, "gbs": pass_gbs,
                              "frac_of_measured_peak": pass_gbs / peak, "frac_of_8TBs": pass_gbs / NOMINAL_HBM_GBS,
                              "kept_rows": rows},
            "clocks": clocks,
        }
        dec = {"algorithmic_bytes": decode_bytes, "gbs_in_step": dec_gbs,
               "frac_of_measured_peak_in_step": dec_gbs / peak,
               "compressed_rows_per_head": (rows + wl.units) / wl.units}
        us = self.time_decode(buf)
        dec["us_per_step"] = {"compressed": us, "full": None}
        dec["gbs_alone"] = decode_bytes / (us * 1e-6) / 1e9
        dec["frac_of_measured_peak_alone"] = dec["gbs_alone"] / peak
        dec["frac_of_8TBs_alone"] = dec["gbs_alone"] / NOMINAL_HBM_GBS
        dec["run_with_append"] = {"compressed": self.time_decode_run(buf), "full": None}
        dec["us_per_step_layer_sequential"] = {"compressed": self.time_decode_run(buf, layerwise=True, max_steps=16),
                                               "full": None}
        dec["us_per_step_layer_sequential_cuda_graph"] = {
            "compressed": self.time_decode_run(buf, layerwise=True, max_steps=16, graph=True), "full": None}
        if not args.no_full_cache:
            full = self.full_cache()
            dec["us_per_step"]["full"] = self.time_decode(full, steps=5)
            dec["run_with_append"]["full"] = self.time_decode_run(full, max_steps=32)
            dec["us_per_step_layer_sequential"]["full"] = self.time_decode_run(full, layerwise=True, max_steps=4)
            dec["us_per_step_layer_sequential_cuda_graph"]["full"] = self.time_decode_run(full, layerwise=True, max_steps=4,
                                                                                         graph=True)
            full_bytes = 2 * int(full.kept_len.sum().item()) * wl.d * e
            dec["full_cache_gbs"] = full_bytes / (dec["us_per_step"]["full"] * 1e-6) / 1e9
            dec["speedup_compressed_vs_full"] = dec["us_per_step"]["full"] / us
            del full
        rec["decode"] = dec
        if not args.no_single_pass:
            single_ms = self.time_single_pass()
            rec["single_pass_score"] = {
                "ms": single_ms, "gbs": k_bytes / (single_ms * 1e-3) / 1e9,
                "frac_of_measured_peak": k_bytes / (single_ms * 1e-3) / 1e9 / peak,
                "note": "madakv_score_lse: stage 1 with the rows' log-sum-exps supplied; not part of the step"}
            if with_streamed:
                s2, s1 = self.time_streamed(overlapped=True), self.time_streamed(overlapped=False)
                rec["streamed_pass"] = {
                    "ms_overlapped": None if s2 is None else s2["ms"],
                    "overlapped_is_a_cuda_graph": None if s2 is None else s2["cuda_graph"],
                    "ms_eager_one_stream": None if s1 is None else s1["ms"],
                    "ratio_to_all_layer_pass": None if s2 is None else s2["ms"] / pass_ms, "launches": wl.L * 7,
                    "note": "stages 1-4 layer by layer (madakv_score_lse, madakv_allocate_layer, select and compact "
                            "with one-layer configs). overlapped: eight layers in flight on their own streams (scoring; "
                            "madakv_demand_layer, then madakv_allocate_layer without scores once the layer before "
                            "has passed phi on, selection; compaction), replayed from one CUDA graph; not part of "
                            "the step"}
        return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=HEADLINE, choices=list(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--only", action="store_true", help="time the headline workload only (no `workloads` records)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-full-cache", action="store_true", help="skip the full-cache decode comparison")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-single-pass", action="store_true", help="skip madakv_score_lse and the streamed order")
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
    dev = torch.device("cuda", local)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    exp2_roof = measure_exp2_roof() if rank == 0 else None

    # ---- headline workload
    b = Bench(mk, wl, dev, rank)
    b.exp2_roof = exp2_roof
    total_ms, stage_ms, clocks = b.timed_steps(args.steps, args.warmup, sync_all, local if rank == 0 else None)
    total_ms, tokens_all = reduce_over_ranks(total_ms, b.tokens, dev, world)
    ms_per_step = total_ms / args.steps
    value = job_throughput(total_ms, args.steps, tokens_all)

    # ---- end to end through the C ABI with host buffers (pinned): H2D of the step's inputs, D2H of its result
    h2d = d2h = 0
    e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    if not args.no_e2e:
        inp, buf = b.inp, b.buf

        def pinned(t):
            h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            h.copy_(t)
            return h

        host = {k: pinned(v) for k, v in inp.items()}
        hdec = [tuple(pinned(x) for x in d) for d in b.dec]
        h_out = torch.empty(buf.out.shape, dtype=buf.out.dtype, pin_memory=True)
        h_len = torch.empty(buf.kept_len.shape, dtype=buf.kept_len.dtype, pin_memory=True)
        h2d = sum(v.numel() * v.element_size() for v in host.values()) + sum(x.numel() * x.element_size()
                                                                             for x in hdec[0])
        d2h = h_out.numel() * h_out.element_size() + h_len.numel() * h_len.element_size()

        def e2e_step(i):
            for k_, v_ in host.items():
                inp[k_].copy_(v_, non_blocking=True)
            for dst, src in zip(b.dec[i % b.n_dec], hdec[i % b.n_dec]):
                dst.copy_(src, non_blocking=True)
            b.step(i)
            h_out.copy_(buf.out, non_blocking=True)
            h_len.copy_(buf.kept_len, non_blocking=True)

        e2e_step(0)
        sync_all()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.e2e_steps + 1)]
        evs[0].record()
        for i in range(args.e2e_steps):
            e2e_step(i)
            evs[i + 1].record()
        sync_all()
        per = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(args.e2e_steps))
        e2e_total, _ = reduce_over_ranks(evs[0].elapsed_time(evs[-1]), b.tokens, dev, world)
        e2e = {"value": job_throughput(e2e_total, args.e2e_steps, tokens_all), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_total / args.e2e_steps,
               "ms_per_step_min": per[0], "ms_per_step_median": per[len(per) // 2], "steps": args.e2e_steps}
        del host, hdec

    if rank != 0:
        # the other ranks only take part in the headline's timed region
        if world > 1:
            dist.destroy_process_group()
        return

    head = b.record(stage_ms, clocks, args)
    launches = args.steps * launches_per_step(wl)
    del b
    torch.cuda.empty_cache()

    # ---- the other benchmark workloads, each from its own timed steps (rank 0; their decode and streamed legs too)
    workloads = {wl.name: head}
    if not args.only and world == 1 and args.layers == 0 and args.budget == 0:
        shared = {}
        for name in OTHER_WORKLOADS:
            if name == wl.name:
                continue
            w2 = synth.CONFIGS[name]
            key = (w2.seed, w2.layout, w2.B, w2.L, w2.Hq, w2.Hkv, w2.n, w2.w)  # the qwen budgets share their inputs
            if key not in shared:
                shared.clear()
                torch.cuda.empty_cache()
                shared[key] = synth.make_inputs(rank_workload(w2, rank), device=dev)
            bb = Bench(mk, w2, dev, rank, inputs=shared[key])
            bb.exp2_roof = exp2_roof
            t_ms, st_ms, clk = bb.timed_steps(max(args.steps, 20), args.warmup, sync_all, local)
            rec = bb.record(st_ms, clk, args)
            rec["ms_per_step"] = t_ms / max(args.steps, 20)
            rec["steps"] = max(args.steps, 20)
            workloads[name] = rec
            del bb
        shared.clear()
        torch.cuda.empty_cache()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu, _ = cpu_oracle_leg(wl)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": workload_config(wl),
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches,
        "roofline": head["roofline"],
        "stages_ms": head["stages_ms"],
        "eviction_pass": head["eviction_pass"],
        "decode": head["decode"],
        "single_pass_score": head.get("single_pass_score"),
        "streamed_pass": head.get("streamed_pass"),
        "cpu_baseline": cpu,
        "exp2_roof_probe": None if exp2_roof is None else exp2_roof[2],
        "workloads": workloads,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
