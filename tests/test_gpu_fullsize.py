"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Config 2 is checked on every output element.  Configs 3-5 (11.5-17.3 TFLOP) are checked where the
oracle can follow in seconds: routing and permutation on ALL tokens (bit-exact), and the float
outputs on sampled tokens (Y, dX, dgate: the oracle recomputes those tokens through all their
experts) and sampled experts (dW: the oracle recomputes every row routed to them), plus properties
that hold at any size.  Inputs are generated on the GPU by the seeded generator and the slices the
oracle needs are downloaded, so both sides see the same bits.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth
from test_gpu_parity import MAX_ABS, check_float, check_layer

pytestmark = pytest.mark.gpu


def test_config2_every_element():
    check_layer(synth.WORKLOADS["c2_mid"], binding.GEMM_AUTO)


def _np_bias(inp):
    return None if inp["bias"] is None else inp["bias"].cpu().numpy()


def _token_problem(w, inp, buf, toks):
    """Reduced problem holding only the sampled tokens and the experts they use (ids remapped)."""
    tk = torch.as_tensor(toks, device=buf.idx.device)
    idx = buf.idx[tk].cpu().numpy()
    used = np.unique(idx)
    remap = np.full(w.E, -1, np.int32)
    remap[used] = np.arange(used.size, dtype=np.int32)
    ue = torch.as_tensor(used, device=buf.idx.device).long()
    prob = {"x": synth.bits(inp["x"][tk]), "idx": remap[idx], "gate": buf.gate[tk].cpu().numpy(),
            "Wg": synth.bits(inp["W_gate"][ue]), "Wu": synth.bits(inp["W_up"][ue]), "Wd": synth.bits(inp["W_down"][ue])}
    if w.backward:
        prob["dY"] = synth.bits(inp["dY"][tk])
    return prob


def _expert_problem(w, inp, buf, e):
    """Reduced problem: every row routed to expert e, as a one-expert top-1 layer."""
    a = torch.nonzero(buf.idx.reshape(-1) == e).reshape(-1)
    t = a // w.k
    rows = int(a.numel())
    return {"rows": rows, "x": synth.bits(inp["x"][t]), "dY": synth.bits(inp["dY"][t]),
            "idx": np.zeros((rows, 1), np.int32), "gate": buf.gate.reshape(-1)[a].cpu().numpy().reshape(rows, 1),
            "Wg": synth.bits(inp["W_gate"][e:e + 1]), "Wu": synth.bits(inp["W_up"][e:e + 1]),
            "Wd": synth.bits(inp["W_down"][e:e + 1])}


@pytest.mark.parametrize("name", ["c3_trillion", "c4_skew", "c5_train"])
def test_full_size_sampled(name):
    w = synth.WORKLOADS[name]
    inp = synth.make_inputs(w, "cuda")
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    binding.forward(ctx, inp, buf)
    if w.backward:
        binding.backward(ctx, inp, buf)
    binding.mop_poll(ctx)
    torch.cuda.synchronize()

    # ---- routing and permutation: all tokens, bit-exact
    xb = synth.bits(inp["x"])
    idx, gate = oracle.route(xb, inp["W_r"].cpu().numpy(), _np_bias(inp), w.k, w.score_fn, w.bias_mode)
    assert np.array_equal(buf.idx.cpu().numpy(), idx), "top-k indices"
    g = buf.gate.cpu().numpy()
    assert np.all(np.abs(g - gate) <= 1e-6 + 1e-5 * np.abs(gate)), "gates"
    counts, offsets, perm_row, row_src = oracle.permute(idx, w.E)
    assert np.array_equal(buf.counts.cpu().numpy(), counts)
    assert np.array_equal(buf.offsets.cpu().numpy(), offsets)
    assert np.array_equal(buf.perm_row.cpu().numpy(), perm_row)
    assert np.array_equal(buf.row_src.cpu().numpy(), row_src)
    assert counts.sum() == w.M
    if w.skew:
        assert (counts == 0).sum() >= 0.1 * w.E, "the skewed workload leaves at least 10 % of experts empty"
        assert counts.max() == w.T, "the heaviest expert receives every token"
    rng = np.random.default_rng(w.seed)
    rows = rng.choice(w.M, 64, replace=False)
    assert np.array_equal(synth.bits(buf.Xp[torch.as_tensor(rows, device="cuda")]), xb[row_src[rows] // w.k])
    del xb

    # ---- properties at full size
    assert torch.isfinite(buf.Y.float()).all()
    if w.backward:
        assert torch.isfinite(buf.dX.float()).all() and torch.isfinite(buf.dgate).all()
        empty = torch.as_tensor(np.nonzero(counts == 0)[0], device="cuda")
        if empty.numel():
            assert torch.all(buf.dW_gate[empty] == 0) and torch.all(buf.dW_down[empty] == 0)

    # ---- float outputs on sampled tokens
    toks = np.sort(rng.choice(w.T, 5, replace=False)).astype(np.int64)
    p = _token_problem(w, inp, buf, toks)
    tk = torch.as_tensor(toks, device="cuda")
    Y_e = oracle.ffn_fwd(p["x"], p["idx"], p["gate"], p["Wg"], p["Wu"], p["Wd"])
    Y_d = oracle.ffn_fwd(p["x"], p["idx"], p["gate"], p["Wg"], p["Wu"], p["Wd"], declared=True)
    print(name, "Y", check_float("Y", buf.Y[tk].float().cpu().numpy(), Y_e, Y_d))
    if w.backward:
        scale = lambda a: MAX_ABS * max(1.0, float(np.abs(a).max()))
        dX_e, dg_e = oracle.ffn_bwd_tokens(p["x"], p["dY"], p["idx"], p["gate"], p["Wg"], p["Wu"], p["Wd"])
        dX_d, dg_d = oracle.ffn_bwd_tokens(p["x"], p["dY"], p["idx"], p["gate"], p["Wg"], p["Wu"], p["Wd"],
                                           declared=True)
        print(name, "dX", check_float("dX", buf.dX[tk].float().cpu().numpy(), dX_e, dX_d, scale(dX_d)))
        print(name, "dgate", check_float("dgate", buf.dgate[tk].cpu().numpy(), dg_e, dg_d, scale(dg_d)))
        del p
        # ---- weight gradients of sampled experts (a light one and a heavy one)
        order = np.argsort(counts)
        live = order[counts[order] > 0]
        for e in (int(live[len(live) // 4]), int(live[-1])):
            q = _expert_problem(w, inp, buf, e)
            ex = np.zeros(1, np.int32)
            dW_e = oracle.ffn_bwd_experts(q["x"], q["dY"], q["idx"], q["gate"], q["Wg"], q["Wu"], q["Wd"], ex)
            dW_d = oracle.ffn_bwd_experts(q["x"], q["dY"], q["idx"], q["gate"], q["Wg"], q["Wu"], q["Wd"], ex,
                                          declared=True)
            for nm, got, a, b in zip(("dW_gate", "dW_up", "dW_down"), (buf.dW_gate, buf.dW_up, buf.dW_down), dW_e,
                                     dW_d):
                print(name, e, q["rows"], nm, check_float(nm, got[e].cpu().numpy(), a[0], b[0], scale(b)))


def test_full_size_router_backward():
    """Router backward at config 5's T, d, E, k (the expert width plays no part in it)."""
    w = synth.small("c5_train", f=64)
    dev = torch.device("cuda")
    x = synth._normal_bf16((w.T, w.d), 1.0, synth._gen(w.seed, 1, dev), dev)
    W_r = torch.randn((w.d, w.E), generator=synth._gen(w.seed, 2, dev), device=dev) * 0.02
    bias = torch.randn((w.E,), generator=synth._gen(w.seed, 6, dev), device=dev) * w.bias_std
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    logits = torch.empty((w.T, w.E), dtype=torch.float32, device=dev)
    binding.mop_moe_route(ctx, x, W_r, bias, buf.idx, buf.gate, logits)
    binding.mop_moe_permute(ctx, x, buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp)
    g = torch.Generator(device=dev).manual_seed(99)
    dgate = torch.randn((w.T, w.k), generator=g, device=dev) * 100.0          # dgate rms is about 140 at this size
    dX0 = torch.randn((w.T, w.d), generator=g, device=dev).to(torch.bfloat16)
    dX = dX0.clone()
    dWr = torch.empty((w.d, w.E), device=dev)
    binding.mop_moe_route_bwd(ctx, logits, bias, buf.idx, buf.gate, dgate, buf.Xp, buf.offsets, buf.perm_row, W_r, dWr,
                              None, dX)
    torch.cuda.synchronize()
    dz, dWr_ref, dXr_ref, _ = oracle.route_bwd(synth.bits(x), W_r.cpu().numpy(), bias.cpu().numpy(), w.k, w.score_fn,
                                               w.bias_mode, buf.idx.cpu().numpy(), dgate.cpu().numpy())
    r = np.linalg.norm(dWr.cpu().numpy() - dWr_ref) / np.linalg.norm(dWr_ref)
    assert r < 1e-5, r
    want = dX0.float().cpu().numpy().astype(np.float64) + dXr_ref
    got = dX.float().cpu().numpy()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 4e-3
    assert np.max(np.abs(got - want)) <= 2.0 ** -8 * np.abs(want).max()
