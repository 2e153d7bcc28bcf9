"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Config 2 is checked on every output element.  Configs 3-5 (11.5-17.3 TFLOP) are checked where the
oracle can follow in a minute: routing and permutation on ALL tokens (bit-exact); the float outputs
Y, dX, dgate on the tokens that own the first and the last row of EVERY live expert (the oracle
recomputes those tokens through all their experts, streaming the experts' weights); the weight
gradients of sixteen experts picked by row count (fewest, most, median, just below / above / at
multiples of 16, 64, 128, and experts whose elements lie beyond 2^31); plus properties that hold at
any size.  Inputs are generated on the GPU by the seeded generator and the slices the
oracle needs are downloaded, so both sides see the same bits.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth
from parity_util import check_float
from test_gpu_parity import check_layer

pytestmark = pytest.mark.gpu


def test_config2_every_element():
    check_layer(synth.WORKLOADS["c2_mid"], binding.GEMM_AUTO)


def _np_bias(inp):
    return None if inp["bias"] is None else inp["bias"].cpu().numpy()


def _expert_problem(w, inp, buf, e, rows=None):
    """Reduced problem: the rows routed to expert e (all, or the listed assignments), as a one-expert top-1 layer."""
    a = torch.nonzero(buf.idx.reshape(-1) == e).reshape(-1) if rows is None else rows
    t = a // w.k
    n = int(a.numel())
    q = {"rows": n, "x": synth.bits(inp["x"][t]), "idx": np.zeros((n, 1), np.int32),
         "gate": buf.gate.reshape(-1)[a].cpu().numpy().reshape(n, 1), "Wg": synth.bits(inp["W_gate"][e:e + 1]),
         "Wu": synth.bits(inp["W_up"][e:e + 1]), "Wd": synth.bits(inp["W_down"][e:e + 1])}
    if w.backward:
        q["dY"] = synth.bits(inp["dY"][t])
    return q


def _sampled_tokens(w, offsets, row_src):
    """Tokens that own the first and the last row of every live expert (at most 2 E of them)."""
    live = np.nonzero(np.diff(offsets) > 0)[0]
    rows = np.concatenate([offsets[live], offsets[live + 1] - 1])
    return np.unique(row_src[rows] // w.k).astype(np.int64)


def _oracle_on_sampled_tokens(w, inp, buf, toks, chunk=8):
    """Y (and dX, dgate) of the sampled tokens in both oracle modes.  The tokens use nearly every expert, so
    the experts are streamed in chunks: each chunk's weights are downloaded once and its (token, slot) pairs
    run through the oracle as a top-1 layer over the chunk; oracle.combine then sums a token's k rows."""
    n = toks.size
    tk = torch.as_tensor(toks, device=buf.idx.device)
    idx_s = buf.idx[tk].cpu().numpy()                      # [n, k]
    gate_s = buf.gate[tk].cpu().numpy()
    xs = synth.bits(inp["x"][tk])
    dys = synth.bits(inp["dY"][tk]) if w.backward else None
    modes = (False, True)
    Yp = {m: np.zeros((n, w.k, w.d), np.float32) for m in modes}
    dXp = {m: np.zeros((n, w.k, w.d), np.float32) for m in modes}
    dg = {m: np.zeros((n, w.k), np.float32) for m in modes}
    for e0 in range(0, w.E, chunk):
        e1 = min(w.E, e0 + chunk)
        q, j = np.nonzero((idx_s >= e0) & (idx_s < e1))    # pairs of this chunk: sampled token q, slot j
        if q.size == 0:
            continue
        sl = slice(e0, e1)
        Wg, Wu, Wd = (synth.bits(inp[nm][sl]) for nm in ("W_gate", "W_up", "W_down"))
        pidx = (idx_s[q, j] - e0).astype(np.int32).reshape(-1, 1)
        pgate = gate_s[q, j].reshape(-1, 1)
        for m in modes:
            Yp[m][q, j] = oracle.ffn_fwd(xs[q], pidx, pgate, Wg, Wu, Wd, declared=m)
            if w.backward:
                a, b = oracle.ffn_bwd_tokens(xs[q], dys[q], pidx, pgate, Wg, Wu, Wd, declared=m)
                dXp[m][q, j], dg[m][q, j] = a, b[:, 0]
    out = {"Y": tuple(oracle.combine(Yp[m], m) for m in modes)}
    if w.backward:
        out["dX"] = tuple(oracle.combine(dXp[m], m) for m in modes)
        out["dgate"] = (dg[False], dg[True])
    return out


def _experts_by_row_count(counts, n_max=16):
    """Experts whose row counts stress the tile edges: fewest and most rows, the median, the counts just
    below and just above multiples of 16, 64 and 128, and experts beyond index 146 (whose weight-gradient
    elements start past 2^31)."""
    live = np.nonzero(counts > 0)[0]
    order = live[np.argsort(counts[live], kind="stable")]
    pick = [int(order[0]), int(order[-1]), int(order[len(order) // 2])]
    for mod in (128, 64, 16):
        r = counts[live] % mod
        pick.append(int(live[np.argmax(r)]))                               # just below a multiple
        pick.append(int(live[np.argmin(np.where(r == 0, mod, r))]))        # just above a multiple
        if (r == 0).any():
            pick.append(int(live[np.argmax(r == 0)]))                      # exactly a multiple
    high = live[live > 146]
    pick += [int(e) for e in high[:: max(1, high.size // 5)][:5]] + ([int(high[-1])] if high.size else [])
    out = []
    for e in pick:
        if e not in out:
            out.append(e)
    return out[:n_max]


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

    # ---- float outputs of the tokens that own the first and the last row of EVERY live expert
    toks = _sampled_tokens(w, offsets, row_src)
    assert np.unique(idx[toks]).size == int((counts > 0).sum()), "the sample touches every live expert"
    tk = torch.as_tensor(toks, device="cuda")
    ref = _oracle_on_sampled_tokens(w, inp, buf, toks)
    case = f"{name}-full-{toks.size}tok"
    print(name, check_float("Y", buf.Y[tk].float().cpu().numpy(), *ref["Y"], case))
    if w.backward:
        print(name, check_float("dX", buf.dX[tk].float().cpu().numpy(), *ref["dX"], case))
        print(name, check_float("dgate", buf.dgate[tk].cpu().numpy(), *ref["dgate"], case))
        del ref
        # ---- weight gradients of experts picked by row count
        for e in _experts_by_row_count(counts):
            q = _expert_problem(w, inp, buf, e)
            ex = np.zeros(1, np.int32)
            dW_e = oracle.ffn_bwd_experts(q["x"], q["dY"], q["idx"], q["gate"], q["Wg"], q["Wu"], q["Wd"], ex)
            dW_d = oracle.ffn_bwd_experts(q["x"], q["dY"], q["idx"], q["gate"], q["Wg"], q["Wu"], q["Wd"], ex,
                                          declared=True)
            for nm, got, a, b in zip(("dW_gate", "dW_up", "dW_down"), (buf.dW_gate, buf.dW_up, buf.dW_down), dW_e,
                                     dW_d):
                print(name, e, q["rows"], check_float(nm, got[e].cpu().numpy(), a[0], b[0],
                                                      f"{name}-full-expert{e}-{q['rows']}rows"))


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
