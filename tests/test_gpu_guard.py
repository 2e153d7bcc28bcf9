"""Guard bands around everything the kernels write: a stand-in for a memory checker.

Every output and stash tensor of the caller is carved out of a larger allocation with a 4 KiB band of
a known pattern directly before and directly after it, and the context's own workspace carries such
bands between all of its buffers (mop_debug_guard_arm / mop_debug_guard_check).  After a forward and
a backward on every GEMM schedule all bands must be intact: a tail tile, a TMA store box or a row
loop that runs past the end of a buffer would leave its mark there, whether or not the next
allocation happens to absorb it.  Small shapes only.
"""
import numpy as np
import pytest
import torch

from paper_2607_01844_b200 import binding, synth
from test_gpu_parity import SMALL, to_dev

pytestmark = pytest.mark.gpu

BAND = 4096
PATTERN = 0xA5


class Guarded:
    """Allocator of device tensors that sit between two pattern bands."""

    def __init__(self):
        self.raw = []

    def empty(self, shape, dtype):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((BAND + nbytes + BAND,), PATTERN, dtype=torch.uint8, device="cuda")
        self.raw.append((raw, nbytes))
        return raw[BAND:BAND + nbytes].view(dtype).view(shape)

    def damaged(self):
        """Number of band bytes that no longer hold the pattern."""
        bad = 0
        for raw, nbytes in self.raw:
            bad += int((raw[:BAND] != PATTERN).sum()) + int((raw[BAND + nbytes:] != PATTERN).sum())
        return bad


def guarded_buffers(w, g):
    buf = binding.LayerBuffers(synth.small(w.name, T=0, d=w.d, E=w.E, k=w.k, f=w.f, backward=w.backward))
    M = w.T * w.k
    i32, b16, f32 = torch.int32, torch.bfloat16, torch.float32
    shapes = {"idx": ((w.T, w.k), i32), "gate": ((w.T, w.k), f32), "counts": ((w.E,), i32),
              "offsets": ((w.E + 1,), i32), "perm_row": ((M,), i32), "row_src": ((M,), i32), "Xp": ((M, w.d), b16),
              "H": ((M, w.f), b16), "Yp": ((M, w.d), b16), "Y": ((w.T, w.d), b16)}
    if w.backward:
        shapes.update({"G": ((M, w.f), b16), "U": ((M, w.f), b16), "dX": ((w.T, w.d), b16), "dgate": ((w.T, w.k), f32),
                       "dW_gate": ((w.E, w.d, w.f), f32), "dW_up": ((w.E, w.d, w.f), f32),
                       "dW_down": ((w.E, w.f, w.d), f32)})
    for name, (shape, dtype) in shapes.items():
        setattr(buf, name, g.empty(shape, dtype))
    return buf


CASES = SMALL + [
    synth.small("c4_skew", T=900, d=320, E=9, k=3, f=448, backward=True, seed=51),     # ragged: d, f = 5 and 7 x 64
    synth.small("c2_mid", T=1100, d=192, E=3, k=2, f=320, backward=True, seed=52),     # 700+ rows per expert
]
PATHS = [binding.GEMM_AUTO, binding.GEMM_SCALAR, binding.GEMM_TENSOR_1CTA, binding.GEMM_TENSOR_2CTA,
         binding.GEMM_TENSOR_MIXED, binding.GEMM_TENSOR_TN]


@pytest.mark.parametrize("w", CASES, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}f{w.f}")
def test_no_kernel_writes_outside_its_buffers(w):
    inp = to_dev(synth.make_inputs(w, "cpu"))
    ref = None
    for path in PATHS:
        if path not in (binding.GEMM_AUTO, binding.GEMM_SCALAR) and (w.d % 64 or w.f % 64):
            continue
        for mode in ((1, 2) if w.backward else (0,)):
            ctx = binding.Context(w.T, w.d, w.E, w.k, w.f, w.score_fn, w.bias_mode, mode, False, path)
            g = Guarded()
            buf = guarded_buffers(w, g)
            binding.mop_debug_guard_arm(ctx)
            assert binding.mop_debug_guard_check(ctx) == 0
            binding.forward(ctx, inp, buf)
            if w.backward:
                if mode == 2:      # recompute the up-projection in the backward instead of reading the stash
                    binding.mop_moe_expert_ffn_bwd(ctx, inp["dY"], buf.Xp, None, None, None, buf.offsets, buf.perm_row,
                                                   buf.row_src, buf.gate, inp["W_gate"], inp["W_up"], inp["W_down"],
                                                   buf.dX, buf.dW_gate, buf.dW_up, buf.dW_down, buf.dgate)
                else:
                    binding.backward(ctx, inp, buf)
            binding.mop_poll(ctx)
            assert binding.mop_debug_guard_check(ctx) == 0, f"workspace bands damaged (path {path}, mode {mode})"
            assert g.damaged() == 0, f"bands around the caller's tensors damaged (path {path}, mode {mode})"
            if ref is None:
                ref = buf
            else:              # the guarded runs also agree with each other where schedules are bit-identical
                assert torch.equal(buf.idx, ref.idx) and torch.equal(buf.perm_row, ref.perm_row)


def test_guard_check_notices_a_write_into_a_band():
    """The check itself: a byte written into a workspace band, and one behind a tensor, are both counted."""
    w = synth.small("c1_tiny", T=32, d=64, E=4, k=2, f=64, backward=True)
    ctx = binding.context_for(w)
    binding.mop_debug_guard_arm(ctx)
    inp = to_dev(synth.make_inputs(w, "cpu"))
    g = Guarded()
    buf = guarded_buffers(w, g)
    binding.forward(ctx, inp, buf)
    assert binding.mop_debug_guard_check(ctx) == 0 and g.damaged() == 0
    raw, nbytes = g.raw[0]
    raw[BAND + nbytes] = 0                    # the host plays the faulty kernel: first byte past the tensor
    assert g.damaged() == 1
    binding.mop_debug_guard_poke(ctx, 0, 4095)   # ... and the last byte before the first workspace buffer
    binding.mop_debug_guard_poke(ctx, 3, 17)
    assert binding.mop_debug_guard_check(ctx) == 2
    binding.mop_debug_guard_arm(ctx)
    assert binding.mop_debug_guard_check(ctx) == 0
    with pytest.raises(binding.MopError):
        binding.mop_debug_guard_poke(ctx, 1000, 0)


def test_gathering_forward_host_io_and_router_backward_stay_inside_their_buffers():
    w = synth.small("c3_trillion", T=300, d=192, E=40, k=8, f=64, backward=True, seed=53)
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    # gathering forward
    ctx = binding.context_for(w, backward=False)
    g = Guarded()
    buf = guarded_buffers(synth.small("c3_trillion", T=w.T, d=w.d, E=w.E, k=w.k, f=w.f, seed=53), g)
    binding.mop_debug_guard_arm(ctx)
    binding.forward(ctx, inp, buf, gather=True)
    binding.mop_poll(ctx)
    assert binding.mop_debug_guard_check(ctx) == 0 and g.damaged() == 0
    # router backward + pipelined host steps (buffers of the context)
    ctx = binding.context_for(w, host_io=2)
    g = Guarded()
    buf = guarded_buffers(w, g)
    logits = g.empty((w.T, w.E), torch.float32)
    dWr = g.empty((w.d, w.E), torch.float32)
    dbias = g.empty((w.E,), torch.float32)
    binding.mop_debug_guard_arm(ctx)
    binding.mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], buf.idx, buf.gate, logits)
    binding.mop_moe_permute(ctx, inp["x"], buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp)
    binding.mop_moe_expert_ffn_fwd(ctx, buf.Xp, buf.offsets, buf.row_src, buf.gate, inp["W_gate"], inp["W_up"],
                                   inp["W_down"], buf.G, buf.U, buf.H, buf.Yp)
    binding.mop_moe_combine(ctx, buf.Yp, buf.perm_row, buf.Y)
    binding.backward(ctx, inp, buf)
    binding.mop_moe_route_bwd(ctx, logits, inp["bias"], buf.idx, buf.gate, buf.dgate, buf.Xp, buf.offsets,
                              buf.perm_row, inp["W_r"], dWr, dbias, buf.dX)
    xh, dYh = host["x"].pin_memory(), host["dY"].pin_memory()
    Yh, dXh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
    dgh = torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()
    for _ in range(3):
        binding.mop_moe_train_step_host_async(ctx, xh, dYh, inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"],
                                              inp["W_down"], Yh, dXh, dgh, buf.dW_gate, buf.dW_up, buf.dW_down)
    binding.mop_host_drain(ctx)
    binding.mop_poll(ctx)
    assert binding.mop_debug_guard_check(ctx) == 0 and g.damaged() == 0


def test_vocabulary_calls_and_static_permute_stay_inside_their_buffers():
    g = Guarded()
    N, H, V = 300, 128, 8192 + 320
    gen = torch.Generator(device="cuda").manual_seed(3)
    X = torch.randn((N, H), generator=gen, device="cuda").to(torch.bfloat16)
    W = (torch.randn((H, V), generator=gen, device="cuda") * 0.1).to(torch.bfloat16)
    t = torch.randint(0, V, (N,), generator=gen, device="cuda", dtype=torch.int32)
    loss, lse = g.empty((N,), torch.float32), g.empty((N,), torch.float32)
    ws = g.empty((max(256, binding.mop_vocab_workspace_bytes(N, H, V)),), torch.uint8)
    binding.mop_vocab_loss_fwd(0, X, W, t, loss, lse, ws)
    dX, dW = g.empty((N, H), torch.bfloat16), g.empty((H, V), torch.float32)
    wsb = g.empty((max(256, binding.mop_vocab_bwd_workspace_bytes(N, H, V)),), torch.uint8)
    binding.mop_vocab_loss_bwd(0, X, W, t, lse, torch.full((N,), -1.0, device="cuda"), dX, dW, wsb)
    w = synth.small("c2_mid", T=3000, d=128, E=96, k=6, f=64)
    idx = torch.stack([torch.randperm(w.E)[:w.k] for _ in range(w.T)]).to(torch.int32).cuda()
    x = torch.randn((w.T, w.d), device="cuda").to(torch.bfloat16)
    buf = guarded_buffers(w, g)
    binding.mop_moe_permute_static(0, w.T, w.d, w.E, w.k, x, idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src,
                                   buf.Xp)
    torch.cuda.synchronize()
    assert g.damaged() == 0
