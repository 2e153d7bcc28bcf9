#!/usr/bin/env python
"""Benchmark of the routed-expert MoE layer on B200: one step = one pass of the whole hot path
(route -> permute -> grouped SwiGLU GEMMs -> combine, plus the backward when the workload has one)
over one batch of seeded synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is useful TFLOP/s of the whole job with inputs resident in
HBM; `e2e` is the same metric through the host-buffer entry point of the C ABI (activations copied
from / to pinned host memory inside the timed region); `roofline` is for the kernel that takes the
largest share of the step; `cpu_baseline` is the CPU oracle timed on a bounded sample.
With N > 1 every rank runs the same workload on its own GPU (the layer has no collective; weak
scaling) and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import numpy as np
import torch

from paper_2607_01844_b200 import launch, synth

# fallback denominators if MEASURED_PEAKS.json is absent (an earlier measurement on this machine)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures, keyed by
# (kernel, workload).  Filled from the summaries under profiles/; None = not captured.
NCU_TRAFFIC_BYTES: dict = {
    # profiles/dram_traffic_gemm_kernels.md: one-pass captures of the full-size launches
    ("gemm_wgrad_gate_up", "c5_train"): 1477344768 + 45034986752,
    ("gemm_up_swiglu", "c3_trillion"): 24036303104 + 537853952,
    ("gemm_up_swiglu", "c4_skew"): 28745956608 + 538783744,
}


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def config_of(w):
    """The workload as both arms print it."""
    return {"workload": w.name, "T": w.T, "d": w.d, "E": w.E, "k": w.k, "f": w.f,
            "pass": "fwd+bwd" if w.backward else "fwd", "l2": "inputs larger than L2"}


def flops_per_step(w):
    return (18 if w.backward else 6) * w.M * w.d * w.f


def kernel_work(w, counts):
    """Algorithmic flops and bytes of one launch of each kernel (useful rows only, every tensor moved once)."""
    T, d, E, k, f, M = w.T, w.d, w.E, w.k, w.f, w.M
    live = int((counts > 0).sum())
    mdf = M * d * f
    stash = 3 if w.backward else 1
    return {
        "route_score": (2 * T * d * E, T * d * 2 + d * E * 4 + T * E * 4),
        "route_select": (0, T * E * 4 + T * k * 8),
        # tensor-core scoring: three bf16 pieces of W_r, x read once, logits written and read back once
        "route_score_tc": (3 * 2 * T * d * E, T * d * 2 + 3 * d * E * 2 + T * E * 4),
        "route_select_screen": (0, T * E * 4 + T * k * 8),
        "route_bwd_dwr": (2 * M * d, M * d * 2 + M * 4 + d * E * 4),
        "route_bwd_dx": (2 * M * d, 2 * T * d * 2 + T * k * 8 + d * E * 4),
        "permute_scatter_rows": (0, T * d * 2 + M * d * 2 + M * 4),
        "dy_scatter_rows": (0, T * d * 2 + M * d * 2 + M * 4),
        "combine_rows": (0, M * d * 2 + T * d * 2 + M * 4),
        "gemm_up_swiglu": (4 * mdf, live * 2 * d * f * 2 + M * d * 2 + stash * M * f * 2),
        "gemm_up_swiglu_gather": (4 * mdf, live * 2 * d * f * 2 + T * d * 2 + M * f * 2),
        "gemm_down_gate": (2 * mdf, live * d * f * 2 + M * f * 2 + M * d * 2),
        "gemm_dgrad_down_dswiglu": (2 * mdf, live * d * f * 2 + M * d * 2 + 6 * M * f * 2),
        "gemm_dgrad_gate_up": (4 * mdf, live * 2 * d * f * 2 + 2 * M * f * 2 + M * d * 2),
        "gemm_wgrad_down": (2 * mdf, E * d * f * 4 + M * f * 2 + M * d * 2),
        "gemm_wgrad_gate_up": (4 * mdf, 2 * E * d * f * 4 + M * d * 2 + 2 * M * f * 2),
    }


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region (read-only query)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(pw)) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- CPU oracle legs
def oracle_expert_sample(w, host_slices, n_experts, backward):
    """Time the oracle, as it stands, on the complete work of `n_experts` experts of this workload
    (every row routed to them: forward, and dgrad + wgrad when the workload has a backward).
    Returns (seconds, useful flops, rows)."""
    import oracle
    secs, flops, rows_total = 0.0, 0, 0
    for sl in host_slices[:n_experts]:
        rows = sl["x"].shape[0]
        if rows == 0:
            continue
        idx = np.zeros((rows, 1), np.int32)
        gate = sl["gate"].reshape(rows, 1).astype(np.float32)
        t0 = time.perf_counter()
        if backward:
            oracle.ffn_bwd_experts(sl["x"], sl["dY"], idx, gate, sl["Wg"], sl["Wu"], sl["Wd"], np.zeros(1, np.int32))
            oracle.ffn_bwd_tokens(sl["x"], sl["dY"], idx, gate, sl["Wg"], sl["Wu"], sl["Wd"])
        else:
            oracle.ffn_fwd(sl["x"], idx, gate, sl["Wg"], sl["Wu"], sl["Wd"])
        secs += time.perf_counter() - t0
        flops += rows * (18 if backward else 6) * w.d * w.f
        rows_total += rows
    return secs, flops, rows_total


def expert_slices(w, inp, idx, gate, experts):
    """Host copies of everything the oracle needs for the listed experts (rows routed to them)."""
    out = []
    flat = idx.reshape(-1)
    for e in experts:
        a = torch.nonzero(flat == e).reshape(-1)
        t = a // w.k
        sl = {"x": synth.bits(inp["x"][t]), "gate": gate.reshape(-1)[a].float().cpu().numpy(),
              "Wg": synth.bits(inp["W_gate"][e:e + 1]), "Wu": synth.bits(inp["W_up"][e:e + 1]),
              "Wd": synth.bits(inp["W_down"][e:e + 1])}
        if w.backward:
            sl["dY"] = synth.bits(inp["dY"][t])
        out.append(sl)
    return out


def run_reference(args, w):
    """The oracle on the host cores: each step is a bounded sample (the complete work of one expert)."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    oracle.build()
    dev = "cpu"
    torch.manual_seed(0)
    # inputs of the sampled experts only: same distributions, generated on the host
    rows = max(1, w.M // w.E)
    n_exp = args.steps + args.warmup
    g = torch.Generator().manual_seed(w.seed)
    def rnd(shape, std):
        return synth.bits((torch.randn(shape, generator=g) * std).to(torch.bfloat16))
    sl = {"x": rnd((rows, w.d), 1.0), "gate": np.full(rows, 1.0 / w.k, np.float32), "Wg": rnd((1, w.d, w.f), 0.02),
          "Wu": rnd((1, w.d, w.f), 0.02), "Wd": rnd((1, w.f, w.d), 0.02)}
    if w.backward:
        sl["dY"] = rnd((rows, w.d), 1.0)
    for _ in range(args.warmup):
        oracle_expert_sample(w, [sl], 1, w.backward)
    secs, flops = 0.0, 0
    for _ in range(args.steps):
        s, f, _ = oracle_expert_sample(w, [sl], 1, w.backward)
        secs += s; flops += f
    val = flops / secs / 1e12
    sample = f"{rows} rows of one expert per step ({'fwd+dgrad+wgrad' if w.backward else 'fwd'}), d={w.d}, f={w.f}"
    print(json.dumps({
        "impl": "reference", "metric": "moe_layer_tflops", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(w),
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------------------- second workload
def run_vocab(args):
    """Vocabulary projection with online log-likelihood (Eq. 5): N = 8192 tokens, H = 7168, V = 131072
    (--shape N,H,V overrides).  vocab_loss: one step = one forward; vocab_train: forward + backward
    (dX, dW_voc).  The N x V logits are never stored."""
    from paper_2607_01844_b200 import binding
    train = args.workload == "vocab_train"
    N, H, V = (int(v) for v in args.shape.split(",")) if args.shape else (8192, 7168, 131072)
    steps, warmup = args.steps or 10, max(3, args.warmup or 3)
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(5)
    X = torch.randn((N, H), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((H, V), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    t = torch.randint(0, V, (N,), generator=g, device="cuda", dtype=torch.int32)
    loss = torch.empty((N,), device="cuda")
    lse = torch.empty((N,), device="cuda")
    ws = binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse)
    stream = torch.cuda.current_stream()
    ws_b = None
    if train:
        dloss = torch.full((N,), -1.0 / N, device="cuda")
        dX = torch.empty_like(X)
        dW = torch.empty((H, V), device="cuda")
        ws_b = binding.mop_vocab_loss_bwd(0, X, W, t, lse, dloss, dX, dW)

    def step():
        binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse, ws, stream)
        if train:
            binding.mop_vocab_loss_bwd(0, X, W, t, lse, dloss, dX, dW, ws_b, stream)

    for _ in range(warmup):
        step()
    sampler = ClockSampler(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    pk, pk_kind = peaks()
    blocks = (V + 8191) // 8192
    # forward: one product; backward: logits again, dW_voc and dX: three more
    tf = (8.0 if train else 2.0) * N * H * V / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "vocab_train_tflops" if train else "vocab_loss_tflops", "value": tf, "unit": "TFLOP/s", "n_gpus": 1,
        "steps": steps, "warmup": warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": {"workload": args.workload, "N": N, "H": H, "V": V, "l2": "inputs larger than L2"},
        "clocks": clocks, "gpu_launches": (3 + (3 * blocks + 2 if train else 0)) * steps,
        "roofline": {"kernel": "vocab_logits_lse" + (" + vocab_dlogits + vocab_wgrad + vocab_dgrad" if train else ""),
                     "bound": "tensor", "achieved": tf, "peak": pk["bf16_tflops_sustained"],
                     "unit": "TFLOP/s", "frac": tf / pk["bf16_tflops_sustained"], "peak_source": pk_kind, "traffic": None,
                     "note": "whole call(s): tile table + GEMMs with their epilogues + merge / conversion"},
        "logits_never_stored_bytes": N * V * 2,
        "workspace_bytes": int(ws.numel()) + (int(ws_b.numel()) if train else 0),
    }))


# --------------------------------------------------------------------------------------- CUDA path
def bench_workload(w, args, steps, warmup, with_cpu_baseline):
    """One workload on this rank's GPU: device-resident timing with a per-kernel profile, the end-to-end
    host-buffer timing, the roofline of the dominant kernel and (optionally) the CPU baseline.  Returns the
    JSON record (rank 0) or None."""
    from paper_2607_01844_b200 import binding
    rank, local, world = launch.env_world()
    dev = torch.device("cuda", local)
    barrier = launch.barrier

    inp = synth.make_inputs(w, dev)
    if args.chunks:
        args.no_e2e = True      # the host-buffer entry points run the unchunked layer
    ctx = binding.context_for(w, device=local, host_io=0 if args.no_e2e else 2, gemm_path=args.gemm_path)
    buf = binding.LayerBuffers(w, device=dev)
    stream = torch.cuda.current_stream()

    rbwd = args.with_router_bwd and w.backward
    if rbwd:
        logits = torch.empty((w.T, w.E), dtype=torch.float32, device=dev)
        dW_r = torch.empty((w.d, w.E), dtype=torch.float32, device=dev)

    chunk_ws = None
    if args.chunks:
        chunk_ws = torch.empty(binding.mop_moe_chunked_workspace_bytes(ctx, args.chunks, w.backward), dtype=torch.uint8,
                               device=dev)

    def step():
        if args.chunks:
            binding.mop_moe_layer_fwd_chunked(ctx, args.chunks, inp["x"], inp["W_r"], inp["bias"], inp["W_gate"],
                                              inp["W_up"], inp["W_down"], buf.idx, buf.gate, buf.counts, buf.offsets,
                                              buf.perm_row, buf.row_src, buf.Y, chunk_ws, stream)
            if w.backward:
                binding.mop_moe_layer_bwd_chunked(ctx, args.chunks, inp["x"], inp["dY"], buf.gate, buf.offsets,
                                                  buf.perm_row, buf.row_src, inp["W_gate"], inp["W_up"], inp["W_down"],
                                                  buf.dX, buf.dW_gate, buf.dW_up, buf.dW_down, buf.dgate, chunk_ws, stream)
            return
        if rbwd:   # the router keeps its logits for the backward
            binding.mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], buf.idx, buf.gate, logits, stream)
            binding.mop_moe_permute(ctx, inp["x"], buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp,
                                    stream)
            binding.mop_moe_expert_ffn_fwd(ctx, buf.Xp, buf.offsets, buf.row_src, buf.gate, inp["W_gate"], inp["W_up"],
                                           inp["W_down"], buf.G, buf.U, buf.H, buf.Yp, stream)
            binding.mop_moe_combine(ctx, buf.Yp, buf.perm_row, buf.Y, stream)
        else:
            binding.forward(ctx, inp, buf, stream, gather=args.gather and not w.backward)
        if w.backward:
            binding.backward(ctx, inp, buf, stream)
        if rbwd:
            binding.mop_moe_route_bwd(ctx, logits, inp["bias"], buf.idx, buf.gate, buf.dgate, buf.Xp, buf.offsets,
                                      buf.perm_row, inp["W_r"], dW_r, None, buf.dX, stream)

    for _ in range(warmup):
        step()
    binding.mop_poll(ctx, stream)
    binding.mop_profile_enable(ctx, True)
    sampler = ClockSampler(local)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    sampler.start()
    l0 = ctx.launch_count
    ev0.record(stream)
    for _ in range(steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize(); barrier()
    launches = ctx.launch_count - l0
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    prof = binding.mop_profile_read(ctx, stream)
    binding.mop_profile_enable(ctx, False)
    binding.mop_poll(ctx, stream)
    ms = launch.max_over_ranks(ms, dev)
    ms_step = ms / steps
    value = launch.job_throughput(flops_per_step(w), ms_step, world) / 1e12

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        xh = inp["x"].cpu().pin_memory()
        Yh = torch.empty_like(xh).pin_memory()
        h2d, d2h = xh.numel() * 2, Yh.numel() * 2
        if w.backward:
            dYh = inp["dY"].cpu().pin_memory()
            dXh = torch.empty_like(xh).pin_memory()
            dgh = torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()
            h2d += dYh.numel() * 2
            d2h += dXh.numel() * 2 + dgh.numel() * 4

            def host_step():
                binding.mop_moe_train_step_host_async(ctx, xh, dYh, inp["W_r"], inp["bias"], inp["W_gate"],
                                                      inp["W_up"], inp["W_down"], Yh, dXh, dgh, buf.dW_gate,
                                                      buf.dW_up, buf.dW_down, stream)
        else:
            idxh = torch.empty((w.T, w.k), dtype=torch.int32).pin_memory()
            gh = torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()
            d2h += idxh.numel() * 4 + gh.numel() * 4

            def host_step():
                binding.mop_moe_forward_host_async(ctx, xh, inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"],
                                                   inp["W_down"], Yh, idxh, gh, stream)
        # Every step copies its inputs in from pinned host memory and its results back out; the
        # pipelined entry points overlap those copies with the neighbouring steps' kernels.  The
        # timed region ends when the last step's results are in host memory (mop_host_drain).
        for _ in range(2):
            host_step()
        binding.mop_host_drain(ctx, stream)
        n_e2e = steps
        barrier(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_e2e):
            host_step()
        binding.mop_host_drain(ctx, stream)
        e1.record(stream)
        torch.cuda.synchronize(); barrier()
        ems = e0.elapsed_time(e1)
        ems = launch.max_over_ranks(ems, dev)
        assert torch.equal(Yh, buf.Y.cpu()), "host entry point and device path disagree"
        e2e = {"value": launch.job_throughput(flops_per_step(w), ems / n_e2e, world) / 1e12, "unit": "TFLOP/s",
               "ms_per_step": ems / n_e2e, "steps": n_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "mop_moe_train_step_host_async" if w.backward else "mop_moe_forward_host_async",
               "overlap": "copies of step i+1 / i-1 run beside the kernels of step i (two buffer slots)"}

    if rank != 0:
        ctx.close()
        return None
    # ---- per-kernel table and the roofline of the dominant kernel
    pk, pk_kind = peaks()
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    counts = buf.counts.cpu().numpy()
    work = kernel_work(w, counts)
    kernels = {}
    for name, (tot, calls) in prof.items():
        avg_ms = tot / max(1, calls)
        fl, by = work.get(name, (0, 0))
        rec = {"ms": round(avg_ms, 4), "launches": calls, "share": round(tot / ms, 4)}
        if fl:
            rec["tflops"] = round(fl / (avg_ms * 1e-3) / 1e12, 1)
        if by:
            rec["gbs"] = round(by / (avg_ms * 1e-3) / 1e9, 1)
        if fl and by:   # fraction of this kernel's own roofline: the longer of its tensor time and its HBM time
            t_roof = max(fl / (pk["bf16_tflops_sustained"] * 1e12), by / (pk["hbm_gbs"] * 1e9))
            rec["roofline_frac"] = round(t_roof / (avg_ms * 1e-3), 3)
            rec["bound"] = "tensor" if fl / (pk["bf16_tflops_sustained"] * 1e12) >= by / (pk["hbm_gbs"] * 1e9) else "hbm"
        elif by:
            rec["roofline_frac"] = round(by / (pk["hbm_gbs"] * 1e9) / (avg_ms * 1e-3), 3)
            rec["bound"] = "hbm"
        kernels[name] = rec
    roofline = None
    if kernels:
        top = max(prof, key=lambda n: prof[n][0])
        avg_s = prof[top][0] / prof[top][1] * 1e-3
        fl, by = work.get(top, (0, 0))
        t_tensor = fl / (pk["bf16_tflops_sustained"] * 1e12)
        t_hbm = by / (pk["hbm_gbs"] * 1e9)
        if top == "route_score":
            # plain fp32 FMA chains: SMs x 128 lanes x 2 flop at the maximum SM clock
            peak = sm_count * 128 * 2 * 1.965e9 / 1e12
            roofline = {"kernel": top, "bound": "alu", "achieved": fl / avg_s / 1e12, "peak": peak, "unit": "TFLOP/s"}
        elif t_tensor >= t_hbm:
            roofline = {"kernel": top, "bound": "tensor", "achieved": fl / avg_s / 1e12,
                        "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s"}
        else:
            roofline = {"kernel": top, "bound": "hbm", "achieved": by / avg_s / 1e9, "peak": pk["hbm_gbs"],
                        "unit": "GB/s"}
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
        roofline["peak_source"] = pk_kind
        roofline["traffic"] = NCU_TRAFFIC_BYTES.get((top, w.name))
        roofline["ms"] = avg_s * 1e3

    # ---- CPU baseline: the oracle on a bounded sample (complete work of a few experts)
    cpu = None
    if world == 1 and with_cpu_baseline:
        import oracle
        oracle.build()
        order = np.argsort(-counts)
        mid = [int(e) for e in order[len(order) // 2: len(order) // 2 + 1]]      # a median-load expert
        sl = expert_slices(w, inp, buf.idx, buf.gate, mid)
        s1, f1, r1 = oracle_expert_sample(w, sl, 1, w.backward)
        n = int(max(1, min(16, 15.0 / max(s1, 1e-3))))
        more = [int(e) for e in order[len(order) // 2 + 1: len(order) // 2 + n]]
        s2, f2, r2 = oracle_expert_sample(w, expert_slices(w, inp, buf.idx, buf.gate, more), len(more), w.backward)
        cpu = {"value": (f1 + f2) / (s1 + s2) / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
               "seconds": round(s1 + s2, 2),
               "sample": f"{1 + len(more)} median-load experts, {r1 + r2} rows: "
                         f"{'fwd+dgrad+wgrad' if w.backward else 'fwd'} of every row routed to them"}
    # expert-contiguous activation buffers: whole layer (Xp, H, Yp; with a backward also the G, U stash and the
    # context's dYp, dG, dU, gH, dXp) against one group of experts at a time plus the fp32 accumulator
    M = w.T * w.k
    full_bytes = M * (2 * w.d + w.f) * 2 + (M * (2 * w.f + 2 * w.d + 3 * w.f) * 2 if w.backward else 0)
    memory = {"expert_contiguous_activation_bytes": full_bytes}
    if args.chunks:
        memory = {"chunks": args.chunks, "chunked_workspace_bytes": int(chunk_ws.numel()),
                  "unchunked_expert_contiguous_activation_bytes": full_bytes,
                  "ratio": chunk_ws.numel() / full_bytes}
    ctx.close()
    return {
        "metric": "moe_layer_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(w),
        "routing": {"load_cv": float(counts.std() / max(1e-9, counts.mean())), "empty_experts": int((counts == 0).sum()),
                    "rows_min": int(counts.min()), "rows_max": int(counts.max())},
        "frac_of_bf16_peak_nominal": value / world / 2250.0,
        "frac_of_bf16_peak_measured": value / world / pk["bf16_tflops_sustained"],
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "kernels": kernels,
        "cpu_baseline": cpu, "memory": memory,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(synth.WORKLOADS) + ["vocab_loss", "vocab_train"],
                    help="default: c5_train as the headline, followed by the forward workloads c2_mid, c3_trillion, "
                         "c4_skew as sub-records of the same JSON line")
    ap.add_argument("--shape", default=None,
                    help="T,d,E,k,f overriding the named workload's sizes (same distributions): small cases for "
                         "profiler captures")
    ap.add_argument("--gemm-path", type=int, default=0, help="mop_gemm_path (0 = library default)")
    ap.add_argument("--with-router-bwd", action="store_true",
                    help="also run the router backward (dgate -> dW_r, dX) in every step of a fwd+bwd workload")
    ap.add_argument("--gather", action="store_true",
                    help="forward-only workloads: up-projection gathers its rows from x (no permuted copy)")
    ap.add_argument("--chunks", type=int, default=0,
                    help="run the expert-chunked layer with this many groups of experts (buffers live for one group at a time)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra-workloads", action="store_true",
                    help="default invocation: skip the forward workloads that follow the headline")
    args = ap.parse_args()
    extra = (args.workload is None and args.shape is None and not args.no_extra_workloads and args.impl == "ours"
             and not args.chunks)
    args.workload = args.workload or "c5_train"
    if args.workload in ("vocab_loss", "vocab_train"):
        return run_vocab(args)
    w = synth.WORKLOADS[args.workload]
    if args.shape:
        T, d, E, k, f = (int(v) for v in args.shape.split(","))
        import dataclasses
        w = dataclasses.replace(w, T=T, d=d, E=E, k=k, f=f, name=f"{w.name}[{args.shape}]")
    if args.impl == "reference":
        args.steps = args.steps or 3
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args, w)
    args.steps = args.steps or 20
    args.warmup = max(3, args.warmup or 3)

    rank, local, world = launch.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local)
    launch.init("nccl", torch.device("cuda", local))

    out = bench_workload(w, args, args.steps, args.warmup, not args.no_cpu_baseline)
    if extra:
        # The tensor-bound forward configurations, one after the other on the freed GPU: sub-records of the
        # same line (metric, config and value of the line stay those of the training configuration).
        subs = {}
        for name in ("c2_mid", "c3_trillion", "c4_skew"):
            torch.cuda.empty_cache()
            sub = bench_workload(synth.WORKLOADS[name], args, min(args.steps, 20), 3, False)
            if sub is not None:
                subs[name] = {k: sub[k] for k in ("ms_per_step", "value", "unit", "steps", "config", "routing", "clocks", "e2e",
                                                  "gpu_launches", "roofline", "kernels",
                                                  "frac_of_bf16_peak_nominal", "frac_of_bf16_peak_measured")}
        if out is not None:
            out["workloads"] = subs
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
