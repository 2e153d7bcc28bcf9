"""The allocation-free permutation entry point, for callers that may not call cudaMalloc (a process
whose own arena holds all of HBM, or a loop that cannot take an allocation's device-wide
synchronisation).  Its scratch is an array compiled into the library, shared by every call, so the
check is made on two calls in a row with different shapes: whatever the first call left in the
array must not leak into the second.  Each call is compared, bit for bit, with mop_moe_permute.

This file is collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test."""
import pytest
import torch

from paper_2607_01844_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _reference(w, x, idx):
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w, backward=False)
    binding.mop_moe_permute(ctx, x, idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp)
    torch.cuda.synchronize()
    return buf


def _static(w, x, idx):
    buf = binding.LayerBuffers(w, backward=False)
    for t in (buf.counts, buf.offsets, buf.perm_row, buf.row_src):
        t.fill_(-7)
    buf.Xp.zero_()
    binding.mop_moe_permute_static(0, w.T, w.d, w.E, w.k, x, idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src,
                                   buf.Xp)
    torch.cuda.synchronize()
    return buf


def _random_topk(w, seed):
    g = torch.Generator().manual_seed(seed)
    idx = torch.stack([torch.randperm(w.E, generator=g)[:w.k] for _ in range(w.T)]).to(torch.int32)
    x = (torch.randn((w.T, w.d), generator=g)).to(torch.bfloat16)
    return x.cuda(), idx.cuda()


def test_static_permute_matches_context_permute_on_two_calls_in_a_row():
    first = synth.small("c2_mid", T=3000, d=128, E=96, k=6, f=64)     # 36 segments x 96 experts
    second = synth.small("c1_tiny", T=700, d=64, E=10, k=3, f=64)     # smaller: stale entries stay behind it
    for w, seed in ((first, 1), (second, 2)):
        x, idx = _random_topk(w, seed)
        got, ref = _static(w, x, idx), _reference(w, x, idx)
        for name in ("counts", "offsets", "perm_row", "row_src", "Xp"):
            assert torch.equal(getattr(got, name), getattr(ref, name)), (w.name, name)


def test_static_permute_at_the_edges_of_its_range():
    """Exactly 262144 scratch entries passes (256 segments x 1024 experts, the largest E), one segment more
    is refused; no tokens gives zero counts and offsets; Xp = None builds the tables only."""
    w = synth.small("c1_tiny", T=256 * 512 // 4, d=64, E=1024, k=4, f=64)           # 256 segments of 512
    x, idx = _random_topk(synth.small("c1_tiny", T=64, d=64, E=1024, k=4, f=64), 3)
    idx = idx.repeat(w.T // 64, 1).contiguous()
    x = x.repeat(w.T // 64, 1).contiguous()
    got, ref = _static(w, x, idx), _reference(w, x, idx)
    for name in ("counts", "offsets", "perm_row", "row_src", "Xp"):
        assert torch.equal(getattr(got, name), getattr(ref, name)), name
    w1 = synth.small("c1_tiny", T=w.T + 1, d=64, E=1024, k=4, f=64)                 # 257 segments
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_permute_static(0, w1.T, w1.d, w1.E, w1.k, x, idx, got.counts, got.offsets, got.perm_row,
                                       got.row_src, got.Xp)
    assert e.value.code == 2
    w0 = synth.small("c1_tiny", T=0, d=64, E=10, k=3, f=64)
    counts = torch.full((10,), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((11,), -7, dtype=torch.int32, device="cuda")
    binding.mop_moe_permute_static(0, 0, 64, 10, 3, None, None, counts, offsets, None, None, None)
    torch.cuda.synchronize()
    assert int(counts.abs().sum()) == 0 and int(offsets.abs().sum()) == 0
    w2 = synth.small("c1_tiny", T=700, d=64, E=10, k=3, f=64)
    x2, idx2 = _random_topk(w2, 4)
    ref2 = _reference(w2, x2, idx2)
    buf = binding.LayerBuffers(w2, backward=False)
    binding.mop_moe_permute_static(0, w2.T, w2.d, w2.E, w2.k, None, idx2, buf.counts, buf.offsets, buf.perm_row,
                                   buf.row_src, None)
    torch.cuda.synchronize()
    for name in ("counts", "offsets", "perm_row", "row_src"):
        assert torch.equal(getattr(buf, name), getattr(ref2, name)), name


def test_static_permute_rejects_sizes_beyond_its_scratch():
    w = synth.small("c1_tiny", T=40000, d=64, E=1000, k=8, f=64)      # 625 segments x 1000 experts > 262144
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_permute_static(0, w.T, w.d, w.E, w.k, dummy, dummy, dummy, dummy, dummy, dummy, dummy)
    assert e.value.code == 2
