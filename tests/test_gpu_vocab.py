"""Vocabulary projection with online log-likelihood (Eq. 5): the CUDA path against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth

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
