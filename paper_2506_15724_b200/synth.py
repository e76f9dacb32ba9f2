"""Seeded synthetic multimodal-shaped inputs for the MadaKV eviction pass.

This module only produces INPUTS (token layouts, Q/K/V values, decode-step vectors). It holds none of the method's
arithmetic and is the one module the CUDA path's callers and the CPU oracle's tests both use.

Values come from a counter-based generator: element ``idx`` of tensor ``tid`` under ``seed`` is
``table[top16(mix64(key(seed, tid) + idx * GOLDEN))]`` where ``table`` is the standard-normal quantile function
sampled at 65536 mid-points (computed once on the CPU in fp64, rounded to fp32). Integer hashing, one table lookup and
single fp32 additions are bit-identical on CPU and CUDA, so a tensor generated on either device holds the same bits,
and any slab can be regenerated independently of the rest.

The workloads stand in for the paper's evaluation inputs (MileBench samples run through LLaVA-1.5 / Qwen2.5-VL), which
are not available here; they take only that benchmark's shape: several images interleaved with short text, the
question at the end of the prompt.
"""
from dataclasses import dataclass, replace
import math

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

# tensor ids
TID_Q, TID_K, TID_V, TID_BETA, TID_DEC_Q, TID_DEC_K, TID_DEC_V = 1, 2, 3, 4, 5, 6, 7


def _s64(x):
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_py(z):
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def _lsr(z, s):
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix_t(z):
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


_table_cache = {}


def normal_table(device="cpu"):
    """65536 standard-normal quantiles at mid-points, fp32; always computed on the CPU, then moved."""
    key = str(device)
    if key not in _table_cache:
        if "cpu" not in _table_cache:
            p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
            _table_cache["cpu"] = torch.special.ndtri(p).to(torch.float32)
        _table_cache[key] = _table_cache["cpu"].to(device)
    return _table_cache[key]


def hash_normal(seed, tid, start, count, device="cpu"):
    """fp32 tensor of ``count`` N(0,1) samples: elements start..start+count-1 of tensor ``tid`` under ``seed``."""
    key = _mix_py(seed * 1000003 + tid)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    z = _mix_t(idx * _s64(_GOLDEN) + _s64(key))
    return normal_table(device)[_lsr(z, 48)]


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str  # "f32" | "bf16"
    B: int
    L: int
    Hq: int
    Hkv: int
    d: int
    n: int  # context length of every sequence (= max_seq_len)
    w: int
    budget: int  # nominal per-KV-head budget phi^1
    theta: float  # Eq. 9 threshold, calibrated so that layer-1 demand is close to the budget
    seed: int
    layout: str
    n_needles: int  # per modality
    max_new_tokens: int

    @property
    def g(self):
        return self.Hq // self.Hkv

    @property
    def units(self):
        return self.B * self.L * self.Hkv

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self):
        return 4 if self.dtype == "f32" else 2


# theta values: written by oracle/calibrate_theta.py (bisection on the CPU oracle, layer 1, demand ~ budget).
CONFIGS = {
    "tiny": Workload("tiny", "f32", 1, 1, 4, 4, 64, 512, 8, 128, 0.674536, 20250615, "tiny", 4, 16),
    "llava": Workload("llava", "bf16", 1, 32, 32, 32, 128, 8192, 32, 1638, 0.471452, 20250616, "llava", 16, 16),
    # second dense shape of the paper's model list (LLaVA-1.5-13B: 40 layers x 40 heads), same prompt recipe as llava
    "llava13b": Workload("llava13b", "bf16", 1, 40, 40, 40, 128, 8192, 32, 1638, 0.472339, 20250620, "llava", 16, 16),
    "qwen": Workload("qwen", "bf16", 1, 28, 28, 4, 128, 32768, 32, 2048, 0.324026, 20250617, "blocks70", 16, 16),
    # the other two points of the Qwen-shaped budget sweep {1024, 2048, 4096}: same prompt and K/V (same seed)
    "qwen1024": Workload("qwen1024", "bf16", 1, 28, 28, 4, 128, 32768, 32, 1024, 0.284623, 20250617, "blocks70", 16, 16),
    "qwen4096": Workload("qwen4096", "bf16", 1, 28, 28, 4, 128, 32768, 32, 4096, 0.395515, 20250617, "blocks70", 16, 16),
    "batched": Workload("batched", "bf16", 8, 28, 28, 4, 128, 16384, 32, 2048, 0.415580, 20250618, "blocks_rand", 16, 128),
    "long": Workload("long", "bf16", 1, 32, 32, 8, 128, 131072, 64, 4096, 0.218545, 20250619, "long", 16, 256),
}


def scaled(wl, **kw):
    """A reduced copy of a workload (fewer layers / heads / tokens) with the same recipe, for parity tests."""
    return replace(wl, **kw)


def _compose(rng, total, parts, minimum):
    """Split ``total`` into ``parts`` integers >= their ``minimum`` at seeded random cut points."""
    minimum = list(minimum)
    free = total - sum(minimum)
    assert free >= 0, (total, parts, minimum)
    cuts = np.sort(rng.randint(0, free + 1, size=parts - 1))
    sizes = np.diff(np.concatenate([[0], cuts, [free]]))
    return [int(s + m) for s, m in zip(sizes, minimum)]


def _interleave(text_sizes, image_sizes):
    """text, image, text, ..., image, text -> uint8 mask (1 = visual)."""
    assert len(text_sizes) == len(image_sizes) + 1
    segs = []
    for i, t in enumerate(text_sizes):
        segs.append(np.zeros(t, np.uint8))
        if i < len(image_sizes):
            segs.append(np.ones(image_sizes[i], np.uint8))
    return np.concatenate(segs)


def _blocks_layout(rng, n, w, visual_fraction):
    target = int(round(visual_fraction * n))
    blocks, tot = [], 0
    while True:
        b = int(rng.randint(256, 1025))
        if tot + b > target:
            rest = target - tot
            if rest >= 256 or not blocks:
                blocks.append(max(rest, 1))
            else:
                blocks[-1] += rest
            break
        blocks.append(b)
        tot += b
    n_vis = sum(blocks)
    text = _compose(rng, n - n_vis, len(blocks) + 1, [1] * len(blocks) + [max(w, 1)])
    return _interleave(text, blocks)


def layout(wl):
    """Token modality mask [B, n] uint8 (1 = visual) and seq_len [B] int32 of a workload."""
    rng = np.random.RandomState(wl.seed % (1 << 31))
    masks = []
    for _ in range(wl.B):
        if wl.layout == "tiny":
            assert wl.n >= 64 + 256 + wl.w
            m = _interleave([64, wl.n - 64 - 256], [256])
        elif wl.layout == "llava":
            n_img, img = 8, 576
            scale = wl.n / 8192.0
            img = max(8, int(round(img * scale)))
            lo, hi = max(1, int(100 * scale)), max(2, int(600 * scale))
            while True:
                text = [int(x) for x in rng.randint(lo, hi + 1, size=n_img)]
                last = wl.n - n_img * img - sum(text)
                if max(lo, wl.w) <= last <= hi:
                    break
            m = _interleave(text + [last], [img] * n_img)
        elif wl.layout == "blocks70":
            m = _blocks_layout(rng, wl.n, wl.w, 0.70)
        elif wl.layout == "blocks_rand":
            m = _blocks_layout(rng, wl.n, wl.w, float(rng.uniform(0.3, 0.9)))
        elif wl.layout == "long":
            n_img = max(1, wl.n // 1024)
            img = 768
            text = _compose(rng, wl.n - n_img * img, n_img + 1, [1] * n_img + [wl.w])
            m = _interleave(text, [img] * n_img)
        else:
            raise ValueError(wl.layout)
        assert m.shape[0] == wl.n, (m.shape, wl.n)
        assert not m[-wl.w:].any(), "the proxy-token window must be text"
        masks.append(m)
    return np.stack(masks), np.full(wl.B, wl.n, np.int32)


def needle_positions(wl, mask):
    """Per sequence: n_needles visual and n_needles text positions outside the window, ascending. [B, 2, n_needles]"""
    rng = np.random.RandomState((wl.seed + 7919) % (1 << 31))
    out = np.zeros((wl.B, 2, wl.n_needles), np.int64)
    for b in range(wl.B):
        body = mask[b, : wl.n - wl.w]
        for m, val in enumerate((1, 0)):
            cand = np.nonzero(body == val)[0]
            assert cand.size >= wl.n_needles
            out[b, m] = np.sort(rng.choice(cand, size=wl.n_needles, replace=False))
    return out


def make_q_win(wl):
    """Window queries [B, L, Hq, w, d] on the CPU, in the workload's dtype."""
    n = wl.B * wl.L * wl.Hq * wl.w * wl.d
    return hash_normal(wl.seed, TID_Q, 0, n).view(wl.B, wl.L, wl.Hq, wl.w, wl.d).to(wl.torch_dtype)


def make_kv(wl, q_win, mask, device="cpu", want_v=True):
    """K and V [B, L, Hkv, n, d] on ``device``.

    K = N(0,1) + (visual token ? beta[l,h,:] : 0) + (needle ? 4 * sqrt(d) * qbar / |qbar|^2 : 0), beta ~ N(0, 0.5^2)
    per (layer, KV head); qbar is the mean window query of the unit's query group, so a needle's logit is raised by
    about 4 for every window row. V = N(0,1). Built one (sequence, layer) slab at a time.
    """
    B, L, Hkv, n, d = wl.B, wl.L, wl.Hkv, wl.n, wl.d
    beta = 0.5 * hash_normal(wl.seed, TID_BETA, 0, L * Hkv * d).view(L, Hkv, 1, d)
    qbar = q_win.to(torch.float64).view(B, L, Hkv, wl.g * wl.w, d).mean(dim=3)  # CPU, so identical everywhere
    boost = (4.0 * math.sqrt(d) * qbar / (qbar * qbar).sum(-1, keepdim=True)).to(torch.float32)  # [B,L,Hkv,d]
    needles = needle_positions(wl, mask)
    k = torch.empty((B, L, Hkv, n, d), dtype=wl.torch_dtype, device=device)
    v = torch.empty((B, L, Hkv, n, d), dtype=wl.torch_dtype, device=device) if want_v else None
    slab = Hkv * n * d
    for b in range(B):
        vis = torch.from_numpy(mask[b].astype(np.float32)).to(device).view(1, n, 1)
        pos = torch.from_numpy(needles[b].reshape(-1)).to(device)
        for l in range(L):
            start = (b * L + l) * slab
            x = hash_normal(wl.seed, TID_K, start, slab, device).view(Hkv, n, d)
            x = x + vis * beta[l].to(device)
            x[:, pos, :] = x[:, pos, :] + boost[b, l].to(device).view(Hkv, 1, d)
            k[b, l] = x.to(wl.torch_dtype)
            if want_v:
                v[b, l] = hash_normal(wl.seed, TID_V, start, slab, device).view(Hkv, n, d).to(wl.torch_dtype)
    return k, v


def make_decode_step(wl, step, device="cpu"):
    """q [B,L,Hq,d], k_new, v_new [B,L,Hkv,d] of decode step ``step`` (fresh N(0,1) per step)."""
    nq = wl.B * wl.L * wl.Hq * wl.d
    nk = wl.B * wl.L * wl.Hkv * wl.d
    q = hash_normal(wl.seed, TID_DEC_Q, step * nq, nq, device).view(wl.B, wl.L, wl.Hq, wl.d)
    kn = hash_normal(wl.seed, TID_DEC_K, step * nk, nk, device).view(wl.B, wl.L, wl.Hkv, wl.d)
    vn = hash_normal(wl.seed, TID_DEC_V, step * nk, nk, device).view(wl.B, wl.L, wl.Hkv, wl.d)
    return q.to(wl.torch_dtype), kn.to(wl.torch_dtype), vn.to(wl.torch_dtype)


def make_inputs(wl, device="cpu", want_v=True):
    """Everything stages 1-4 read: dict(q_win (on device), k, v, mask [B,n] uint8, seq_len [B], budget [B])."""
    mask, seq_len = layout(wl)
    q_cpu = make_q_win(wl)
    k, v = make_kv(wl, q_cpu, mask, device, want_v)
    return dict(
        q_win=q_cpu.to(device),
        k=k,
        v=v,
        mask=torch.from_numpy(mask).to(device),
        seq_len=torch.from_numpy(seq_len).to(device),
        budget=torch.full((wl.B,), wl.budget, dtype=torch.int32, device=device),
    )
