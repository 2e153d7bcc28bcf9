"""Expert-chunked layer (the expert-contiguous buffers live for one group of experts at a time) against the
unchunked path and the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth
from parity_util import check_float
from test_gpu_parity import np_bias, run, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    synth.small("c2_mid", T=1500, d=256, E=6, k=2, f=320, backward=True, seed=70),          # 500 rows per expert
    synth.small("c3_trillion", T=600, d=192, E=40, k=8, f=128, backward=True, seed=71),     # sigmoid + bias, 120 rows each
    synth.small("c4_skew", T=1024, d=192, E=16, k=4, f=192, backward=True, seed=72),        # skewed: hot and empty experts
    synth.small("c1_tiny", T=3, d=64, E=5, k=1, f=64, backward=True, seed=73),              # fewer rows than experts
]


def chunked(w, inp, n_chunks):
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    for t in (buf.Xp, buf.H, buf.Yp):
        t.fill_(float("nan"))                                   # the chunked layer must not touch the full-size buffers
    nbytes = binding.mop_moe_chunked_workspace_bytes(ctx, n_chunks, True)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    binding.mop_moe_layer_fwd_chunked(ctx, n_chunks, inp["x"], inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"],
                                      inp["W_down"], buf.idx, buf.gate, buf.counts, buf.offsets, buf.perm_row, buf.row_src,
                                      buf.Y, ws)
    for t in (buf.dW_gate, buf.dW_up, buf.dW_down):
        t.fill_(3.0)
    binding.mop_moe_layer_bwd_chunked(ctx, n_chunks, inp["x"], inp["dY"], buf.gate, buf.offsets, buf.perm_row,
                                      buf.row_src, inp["W_gate"], inp["W_up"], inp["W_down"], buf.dX, buf.dW_gate,
                                      buf.dW_up, buf.dW_down, buf.dgate, ws)
    binding.mop_poll(ctx)
    torch.cuda.synchronize()
    assert torch.isnan(buf.Xp.float()).all() and torch.isnan(buf.Yp.float()).all()
    return ctx, buf, nbytes


@pytest.mark.parametrize("w", CASES, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}f{w.f}")
def test_chunked_layer_matches_the_unchunked_layer_and_the_oracle(w):
    host, inp, _, ref = run(w, binding.GEMM_AUTO)
    xb, Wg, Wu, Wd, dYb = (synth.bits(host[n]) for n in ("x", "W_gate", "W_up", "W_down", "dY"))
    sizes = []
    for n_chunks in (1, 2, 3, 8):
        ctx, buf, nbytes = chunked(w, inp, n_chunks)
        sizes.append(nbytes)
        for n in ("idx", "gate", "counts", "offsets", "perm_row", "row_src"):
            assert torch.equal(getattr(buf, n), getattr(ref, n)), (n_chunks, n)
        # each expert's rows go through the same kernels in the same order: weight gradients and dgate bit for bit
        for n in ("dW_gate", "dW_up", "dW_down", "dgate"):
            assert torch.equal(getattr(buf, n), getattr(ref, n)), (n_chunks, n)
        # Y and dX sum a token's experts in expert order instead of score order: equal up to that (one bf16 ulp)
        for n in ("Y", "dX"):
            a, b = getattr(buf, n).float(), getattr(ref, n).float()
            assert torch.all((a - b).abs() <= 2.0 ** -7 * b.abs() + 1e-30), (n_chunks, n)
        if n_chunks == 3:
            idx, gate = buf.idx.cpu().numpy(), buf.gate.cpu().numpy()
            case = f"chunked3-{w.name}-T{w.T}"
            check_float("Y", buf.Y.float().cpu().numpy(), oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd),
                        oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd, declared=True), case)
            dX_e, _ = oracle.ffn_bwd_tokens(xb, dYb, idx, gate, Wg, Wu, Wd)
            dX_d, _ = oracle.ffn_bwd_tokens(xb, dYb, idx, gate, Wg, Wu, Wd, declared=True)
            check_float("dX", buf.dX.float().cpu().numpy(), dX_e, dX_d, case)
    if w.T * w.k >= 64 * 8:
        assert sizes[3] < sizes[2] <= sizes[1] <= sizes[0]       # more chunks, smaller buffers


def test_chunked_layer_is_reproducible_and_refuses_what_it_cannot_do():
    w = CASES[1]
    inp = to_dev(synth.make_inputs(w, "cpu"))
    _, a, _ = chunked(w, inp, 4)
    _, b, _ = chunked(w, inp, 4)
    for n in ("Y", "dX", "dgate", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(getattr(a, n), getattr(b, n)), n
    ctx = binding.context_for(w)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_layer_fwd_chunked(ctx, 0, inp["x"], inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"],
                                          inp["W_down"], a.idx, a.gate, a.counts, a.offsets, a.perm_row, a.row_src, a.Y, ws)
    assert e.value.code == 1
    odd = synth.small("c1_tiny", T=77, d=72, E=5, k=2, f=40, seed=16)              # no tensor-core path for d = 72
    octx = binding.context_for(odd)
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_layer_fwd_chunked(octx, 2, inp["x"], inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"],
                                          inp["W_down"], a.idx, a.gate, a.counts, a.offsets, a.perm_row, a.row_src, a.Y, ws)
    assert e.value.code == 6
