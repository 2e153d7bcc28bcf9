"""Seeded synthetic inputs for the routed-expert layer.

This module holds no arithmetic of the layer itself: it only draws tensors with the
shapes and value distributions of the five workloads (activations ~ N(0,1) in bf16,
expert weights ~ N(0,0.02) in bf16, router weights ~ N(0,0.02) in fp32, router bias
~ N(0,0.01) or a skew-calibrated bias).  Both the CUDA path and the CPU checker are
fed from it, so they see identical bits.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

SCORE_SOFTMAX, SCORE_SIGMOID = 0, 1
BIAS_NONE, BIAS_POST_SCORE, BIAS_PRE_LOGIT = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    d: int
    E: int
    k: int
    f: int
    score_fn: int = SCORE_SOFTMAX
    bias_mode: int = BIAS_NONE
    bias_std: float = 0.0
    skew: bool = False       # Zipf(1.2)-calibrated bias with >= 10 % empty experts
    backward: bool = False
    seed: int = 0

    @property
    def M(self) -> int:
        return self.T * self.k


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", 256, 256, 8, 2, 512, seed=0),
    "c2_mid": Workload("c2_mid", 4096, 2048, 64, 6, 1408, seed=1),
    "c3_trillion": Workload("c3_trillion", 16384, 7168, 256, 8, 2048, SCORE_SIGMOID, BIAS_POST_SCORE, 0.01, seed=2),
    "c4_skew": Workload("c4_skew", 16384, 7168, 256, 8, 2048, SCORE_SIGMOID, BIAS_POST_SCORE, 0.01, skew=True,
                        seed=3),
    "c5_train": Workload("c5_train", 8192, 7168, 384, 8, 2048, SCORE_SIGMOID, BIAS_POST_SCORE, 0.01, backward=True,
                         seed=4),
}


def small(name: str, **kw) -> Workload:
    """A named workload with some sizes overridden (same distributions)."""
    return replace(WORKLOADS[name], **kw)


def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1_000_003 + stream)
    return g


def _normal_bf16(shape, std, gen, device, chunk_rows=None):
    """N(0, std) drawn in fp32 and rounded once to bf16, in slabs to bound temporaries."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    if out.numel() == 0:
        return out
    flat = out.view(shape[0], -1)
    step = chunk_rows or max(1, (1 << 28) // max(1, flat.shape[1]))
    for r0 in range(0, flat.shape[0], step):
        r1 = min(flat.shape[0], r0 + step)
        tmp = torch.randn((r1 - r0, flat.shape[1]), generator=gen, device=device, dtype=torch.float32)
        flat[r0:r1] = (tmp * std).to(torch.bfloat16)
    return out


def zipf_targets(T: int, E: int, k: int, dead: int, s: float = 1.2) -> torch.Tensor:
    """Zipf(s) loads over the live experts, water-filled under the cap T (an expert can get
    each token at most once).  Returns float64 targets of length E - dead, descending."""
    live = E - dead
    w = torch.arange(1, live + 1, dtype=torch.float64) ** (-s)
    M = float(T * k)
    capped = torch.zeros(live, dtype=torch.bool)
    tgt = torch.zeros(live, dtype=torch.float64)
    for _ in range(live):
        free_mass = M - float(capped.sum()) * T
        share = w.clone()
        share[capped] = 0
        tgt = torch.where(capped, torch.full_like(w, float(T)), share / share.sum() * free_mass)
        over = (tgt > T) & ~capped
        if not over.any():
            break
        capped |= over
    return tgt


def skew_bias(x: torch.Tensor, W_r: torch.Tensor, k: int, seed: int) -> torch.Tensor:
    """Post-score router bias that makes expert loads follow a capped Zipf(1.2) over a random
    expert order with ceil(0.1 E) experts empty.  A calibration loop on approximate scores
    (library matmul and sigmoid); it is an input recipe, not part of the layer."""
    T, E = x.shape[0], W_r.shape[1]
    dev = x.device
    s = torch.sigmoid(x.float() @ W_r)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed * 1_000_003 + 77)
    order = torch.randperm(E, generator=gen)
    dead = math.ceil(0.1 * E)
    live = E - dead
    tgt_sorted = zipf_targets(T, E, k, dead)
    target = torch.zeros(E, dtype=torch.float64)
    target[order[:live]] = tgt_sorted
    target = target.to(dev)
    b = torch.zeros(E, dtype=torch.float32, device=dev)
    deadmask = torch.zeros(E, dtype=torch.bool, device=dev)
    deadmask[order[live:].to(dev)] = True
    pinned = (target >= T) & ~deadmask
    free = ~deadmask & ~pinned
    b[deadmask] = -8.0
    b[pinned] = 8.0
    if k > int(pinned.sum()) and int(free.sum()) > 0:
        logt = torch.log(target.clamp_min(0.5)).float()
        for eta, iters in ((0.05, 300), (0.02, 500), (0.005, 700)):
            for _ in range(iters):
                sel = torch.topk(s + b, k, dim=1).indices
                load = torch.bincount(sel.reshape(-1), minlength=E).float()
                step = (logt - torch.log(load.clamp_min(0.5))).clamp(-1.0, 1.0)
                b = torch.where(free, b + eta * step, b)
                b = torch.where(free, b - b[free].mean(), b)
    return b


def make_inputs(w: Workload, device="cpu") -> dict:
    """All input tensors of one workload on `device` (generator streams are per tensor)."""
    dev = torch.device(device)
    out = {"workload": w}
    out["x"] = _normal_bf16((w.T, w.d), 1.0, _gen(w.seed, 1, dev), dev)
    out["W_r"] = torch.randn((w.d, w.E), generator=_gen(w.seed, 2, dev), device=dev, dtype=torch.float32) * 0.02
    out["W_gate"] = _normal_bf16((w.E, w.d, w.f), 0.02, _gen(w.seed, 3, dev), dev, chunk_rows=max(1, (1 << 27) // (w.d * w.f)))
    out["W_up"] = _normal_bf16((w.E, w.d, w.f), 0.02, _gen(w.seed, 4, dev), dev, chunk_rows=max(1, (1 << 27) // (w.d * w.f)))
    out["W_down"] = _normal_bf16((w.E, w.f, w.d), 0.02, _gen(w.seed, 5, dev), dev, chunk_rows=max(1, (1 << 27) // (w.d * w.f)))
    if w.bias_mode != BIAS_NONE:
        if w.skew:
            out["bias"] = skew_bias(out["x"], out["W_r"], w.k, w.seed)
        else:
            out["bias"] = torch.randn((w.E,), generator=_gen(w.seed, 6, dev), device=dev,
                                      dtype=torch.float32) * w.bias_std
    else:
        out["bias"] = None
    if w.backward:
        out["dY"] = _normal_bf16((w.T, w.d), 1.0, _gen(w.seed, 7, dev), dev)
    return out


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (on the host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
