"""Vocabulary projection with online log-likelihood (Eq. 5): the CUDA path against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth
from parity_util import check_float

pytestmark = pytest.mark.gpu


def _inputs(N, H, V, seed, std=0.02, device="cuda"):
    g = torch.Generator(device=device).manual_seed(seed)
    X = torch.randn((N, H), generator=g, device=device).to(torch.bfloat16)
    W = (torch.randn((H, V), generator=g, device=device) * std).to(torch.bfloat16)
    t = torch.randint(0, V, (N,), generator=g, device=device, dtype=torch.int32)
    return X, W, t


@pytest.mark.parametrize("N,H,V,std", [(1, 64, 64, 0.3), (300, 128, 1024, 0.2), (1000, 512, 4160, 0.05),
                                       (129, 192, 320, 2.0)])
def test_vocab_loss_matches_oracle(N, H, V, std):
    X, W, t = _inputs(N, H, V, seed=N + V, std=std)
    t[0] = 0
    t[-1] = V - 1                                                     # first and last column
    loss = torch.full((N,), 7.0, device="cuda")
    lse = torch.full((N,), 7.0, device="cuda")
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse)
    torch.cuda.synchronize()
    ref, ref_lse = oracle.vocab_loss(synth.bits(X), synth.bits(W), t.cpu().numpy())
    tol = 2e-3 * max(1.0, float(np.abs(ref_lse).max()))              # fp32 accumulation over H, __expf
    assert np.max(np.abs(lse.cpu().numpy() - ref_lse)) < tol
    assert np.max(np.abs(loss.cpu().numpy() - ref)) < tol
    # reproducible bit for bit
    loss2 = torch.empty_like(loss)
    binding.mop_vocab_loss_fwd(0, X, W, t, loss2, None)
    assert torch.equal(loss, loss2)


def test_vocab_loss_full_size_sampled_rows():
    N, H, V = 8192, 7168, 131072
    X, W, t = _inputs(N, H, V, seed=5)
    loss = torch.empty((N,), device="cuda")
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, None)
    torch.cuda.synchronize()
    assert torch.isfinite(loss).all() and bool((loss <= 0).all())
    rows = np.sort(np.random.default_rng(5).choice(N, 6, replace=False))
    r = torch.as_tensor(rows, device="cuda")
    ref, _ = oracle.vocab_loss(synth.bits(X[r]), synth.bits(W), t[r].cpu().numpy())
    assert np.max(np.abs(loss[r].cpu().numpy() - ref)) < 5e-3


def test_vocab_loss_rejects_bad_arguments():
    X, W, t = _inputs(64, 64, 64, seed=1)
    loss = torch.empty((64,), device="cuda")
    with pytest.raises(binding.MopError) as e:
        binding.mop_vocab_loss_fwd(0, X[:, :32].contiguous(), W[:32].contiguous(), t, loss)     # H = 32
    assert e.value.code == 6
    assert binding.mop_vocab_workspace_bytes(64, 64, 100) == 0


def test_a_wait_that_runs_out_in_a_vocabulary_call_is_reported_through_its_workspace():
    """The vocabulary calls have no context: the status word is the first word of the caller's workspace and
    mop_vocab_poll reads it.  A wait that nothing completes gives up after its limit (no fault), the poll
    reports it once, and the same workspace then serves a correct call."""
    N, H, V = 130, 64, 320
    X, W, t = _inputs(N, H, V, seed=9, std=0.3)
    loss = torch.empty((N,), device="cuda")
    ws = binding.mop_vocab_loss_fwd(0, X, W, t, loss)
    binding.mop_vocab_poll(0, ws)
    binding.mop_vocab_selftest_wait_timeout(0, ws, 20_000_000)
    with pytest.raises(binding.MopError) as e:
        binding.mop_vocab_poll(0, ws)
    assert e.value.code == 7
    binding.mop_vocab_poll(0, ws)                                     # cleared
    loss2 = torch.empty_like(loss)
    binding.mop_vocab_loss_fwd(0, X, W, t, loss2, None, ws)
    binding.mop_vocab_poll(0, ws)
    assert torch.equal(loss, loss2)


def _rel_fro(got, ref):
    n = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (n if n > 0 else 1.0))


@pytest.mark.parametrize("N,H,V,std", [(1, 64, 64, 0.3), (300, 128, 1024, 0.2), (200, 128, 8192 + 320, 0.1),
                                       (513, 256, 16384 + 64, 0.05), (129, 192, 320, 1.0)])
def test_vocab_loss_backward_matches_oracle(N, H, V, std):
    """dX and dW_voc against the fp64 oracle; the shapes span one, two and three vocabulary blocks with ragged tails."""
    X, W, t = _inputs(N, H, V, seed=N + V + 1, std=std)
    t[0] = 0
    t[-1] = V - 1
    g = torch.randn((N,), device="cuda") * 0.5 - 1.0
    loss = torch.empty((N,), device="cuda")
    lse = torch.empty((N,), device="cuda")
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse)
    dX = torch.full((N, H), 3.0, device="cuda", dtype=torch.bfloat16)
    dW = torch.full((H, V), 3.0, device="cuda")
    binding.mop_vocab_loss_bwd(0, X, W, t, lse, g, dX, dW)
    torch.cuda.synchronize()
    xb, wb, tn, gn = synth.bits(X), synth.bits(W), t.cpu().numpy(), g.cpu().numpy()
    dX_e, dW_e = oracle.vocab_loss_bwd(xb, wb, tn, gn)
    dX_d, dW_d = oracle.vocab_loss_bwd(xb, wb, tn, gn, declared=True)
    # against the declared-rounding mode only summation order, __expf and the final bf16 of dX remain
    case = f"vocab-N{N}H{H}V{V}std{std}"
    check_float("dX_voc", dX.float().cpu().numpy(), dX_e, dX_d, case)
    check_float("dW_voc", dW.cpu().numpy(), dW_e, dW_d, case)
    # reproducible bit for bit
    dX2, dW2 = torch.empty_like(dX), torch.empty_like(dW)
    binding.mop_vocab_loss_bwd(0, X, W, t, lse, g, dX2, dW2)
    assert torch.equal(dX, dX2) and torch.equal(dW, dW2)


def test_vocab_loss_backward_without_tokens_zeroes_the_weight_gradient():
    X, W, t = _inputs(0, 64, 128, seed=3)
    dW = torch.full((64, 128), 3.0, device="cuda")
    dX = torch.empty((0, 64), device="cuda", dtype=torch.bfloat16)
    e = torch.empty((0,), device="cuda")
    ws = torch.empty(max(256, binding.mop_vocab_bwd_workspace_bytes(0, 64, 128)), dtype=torch.uint8, device="cuda")
    binding.mop_vocab_loss_bwd(0, X, W, t, e, e, dX, dW, ws)
    torch.cuda.synchronize()
    assert float(dW.abs().max()) == 0.0


def test_vocab_loss_backward_full_width_every_element_of_the_weight_gradient():
    """Full H = 7168 and V = 131072 (sixteen vocabulary blocks, element offsets of dW_voc up to 9.4e8) with
    N = 128 tokens, so that the fp64 oracle can follow: every element of dW_voc and of dX."""
    N, H, V = 128, 7168, 131072
    X, W, t = _inputs(N, H, V, seed=8)
    t[0], t[-1] = 0, V - 1
    g = torch.randn((N,), device="cuda") * 0.5 - 1.0
    loss = torch.empty((N,), device="cuda")
    lse = torch.empty((N,), device="cuda")
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse)
    dX = torch.empty_like(X)
    dW = torch.empty((H, V), device="cuda")
    binding.mop_vocab_loss_bwd(0, X, W, t, lse, g, dX, dW)
    torch.cuda.synchronize()
    xb, wb, tn, gn = synth.bits(X), synth.bits(W), t.cpu().numpy(), g.cpu().numpy()
    got_X, got_W = dX.float().cpu().numpy(), dW.cpu().numpy()
    del dW, W
    # one mode at a time: each holds an fp64 copy of W_voc and of dW_voc (7.5 GB each)
    dX_d, dW_d = oracle.vocab_loss_bwd(xb, wb, tn, gn, declared=True)
    from parity_util import TOL
    atol, c_rms, rtol = TOL["dW_voc"]
    rms = float(np.sqrt(np.mean(dW_d * dW_d)))
    use, max_abs = 0.0, 0.0
    for h0 in range(0, H, 512):                           # row slabs keep the fp64 temporaries small
        ref = dW_d[h0:h0 + 512]
        err = np.abs(got_W[h0:h0 + 512] - ref)
        use = max(use, float((err / (atol + c_rms * rms + rtol * np.abs(ref))).max()))
        max_abs = max(max_abs, float(err.max()))
    dX_d = dX_d.astype(np.float32)
    del dW_d
    dX_e, dW_e = oracle.vocab_loss_bwd(xb, wb, tn, gn)
    num = sum(float(((got_W[h0:h0 + 512] - dW_e[h0:h0 + 512]) ** 2).sum()) for h0 in range(0, H, 512))
    rel = float(np.sqrt(num) / np.linalg.norm(dW_e))
    print("vocab full width: dW_voc rel-Fro vs exact", rel, "max-abs vs declared", max_abs, "rms", rms, "bound use", use)
    assert rel <= 1e-2 and use <= 1.0
    check_float("dX_voc", got_X, dX_e.astype(np.float32), dX_d, f"vocab-N{N}H{H}V{V}")


def test_vocab_loss_backward_full_size_sampled_rows_and_invariant():
    """N = 8192, H = 7168, V = 131072 (sixteen vocabulary blocks): dX of sampled tokens against the oracle,
    and the vocabulary sum of dW_voc, which vanishes because every row of dY sums to zero."""
    N, H, V = 8192, 7168, 131072
    X, W, t = _inputs(N, H, V, seed=6)
    loss = torch.empty((N,), device="cuda")
    lse = torch.empty((N,), device="cuda")
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse)
    g = torch.full((N,), -1.0, device="cuda")
    dX = torch.empty_like(X)
    dW = torch.empty((H, V), device="cuda")
    binding.mop_vocab_loss_bwd(0, X, W, t, lse, g, dX, dW)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(6).choice(N, 4, replace=False))
    r = torch.as_tensor(rows, device="cuda")
    dX_e, _ = oracle.vocab_loss_bwd(synth.bits(X[r]), synth.bits(W), t[r].cpu().numpy(), g[r].cpu().numpy())
    got = dX[r].float().cpu().numpy().astype(np.float64)
    assert _rel_fro(got, dX_e) <= 1e-2
    col_sum = dW.sum(1, dtype=torch.float64)
    scale = dW.abs().sum(1, dtype=torch.float64)
    assert float((col_sum.abs() / scale).max()) < 2e-3      # bf16 rounding of dY leaves a small residue
    assert torch.isfinite(dW).all()
