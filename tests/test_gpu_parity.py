"""Parity of the CUDA path (called through the C ABI) with the CPU oracle on the same seeded inputs.

Integers (top-k indices, counts, offsets, permutation) must match bit for bit.  Floats: relative
Frobenius error <= 1e-2 against the oracle's exact mode and max-abs error <= 2e-2 against its
declared-rounding mode (bf16 roundings at the tensors the interface declares bf16), per tensor.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import binding, synth
from parity_util import check_float, rel_fro

pytestmark = pytest.mark.gpu


def to_dev(host):
    return {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in host.items()}


def np_bias(host):
    return None if host["bias"] is None else host["bias"].cpu().numpy()


def run(w, gemm_path=binding.GEMM_AUTO, host=None):
    host = host or synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    ctx = binding.context_for(w, gemm_path=gemm_path)
    buf = binding.LayerBuffers(w)
    binding.forward(ctx, inp, buf)
    if w.backward:
        binding.backward(ctx, inp, buf)
    binding.mop_poll(ctx)
    torch.cuda.synchronize()
    return host, inp, ctx, buf


def check_integers(w, host, buf):
    xb = synth.bits(host["x"])
    idx, gate = oracle.route(xb, host["W_r"].numpy(), np_bias(host), w.k, w.score_fn, w.bias_mode)
    assert np.array_equal(buf.idx.cpu().numpy(), idx), "top-k indices"
    g = buf.gate.cpu().numpy()
    assert np.all(np.abs(g - gate) <= 1e-6 + 1e-5 * np.abs(gate)), "gates"
    counts, offsets, perm_row, row_src = oracle.permute(idx, w.E)
    assert np.array_equal(buf.counts.cpu().numpy(), counts), "counts"
    assert np.array_equal(buf.offsets.cpu().numpy(), offsets), "offsets"
    assert np.array_equal(buf.perm_row.cpu().numpy(), perm_row), "perm_row"
    assert np.array_equal(buf.row_src.cpu().numpy(), row_src), "row_src"
    Xp = synth.bits(buf.Xp)
    assert np.array_equal(Xp, xb[row_src // w.k]), "Xp rows"
    return idx, g


def check_layer(w, gemm_path):
    host, inp, ctx, buf = run(w, gemm_path)
    idx, gate = check_integers(w, host, buf)   # the float checks use the CUDA path's gates (<= 1e-5 apart)
    xb, Wg, Wu, Wd = (synth.bits(host[n]) for n in ("x", "W_gate", "W_up", "W_down"))
    case = f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}f{w.f}-path{gemm_path}"
    Y_e = oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd)
    Y_d = oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd, declared=True)
    check_float("Y", buf.Y.float().cpu().numpy(), Y_e, Y_d, case)
    if w.backward:
        dYb = synth.bits(host["dY"])
        ex = np.arange(w.E, dtype=np.int32)
        dX_e, dg_e = oracle.ffn_bwd_tokens(xb, dYb, idx, gate, Wg, Wu, Wd)
        dX_d, dg_d = oracle.ffn_bwd_tokens(xb, dYb, idx, gate, Wg, Wu, Wd, declared=True)
        dW_e = oracle.ffn_bwd_experts(xb, dYb, idx, gate, Wg, Wu, Wd, ex)
        dW_d = oracle.ffn_bwd_experts(xb, dYb, idx, gate, Wg, Wu, Wd, ex, declared=True)
        check_float("dX", buf.dX.float().cpu().numpy(), dX_e, dX_d, case)
        check_float("dgate", buf.dgate.cpu().numpy(), dg_e, dg_d, case)
        for name, got, e, dd in zip(("dW_gate", "dW_up", "dW_down"), (buf.dW_gate, buf.dW_up, buf.dW_down), dW_e,
                                    dW_d):
            check_float(name, got.cpu().numpy(), e, dd, case)
    return ctx, buf


SMALL = [
    synth.WORKLOADS["c1_tiny"],
    synth.small("c1_tiny", backward=True),
    synth.small("c2_mid", T=300, d=192, E=12, k=3, f=320, backward=True, seed=11),          # ragged tiles
    synth.small("c3_trillion", T=200, d=256, E=40, k=8, f=128, backward=True, seed=12),     # sigmoid + bias
    synth.small("c3_trillion", T=130, d=64, E=33, k=1, f=64, bias_mode=2, backward=True, seed=13),
    synth.small("c1_tiny", T=64, d=128, E=4, k=4, f=64, backward=True, seed=14),            # k = E
    synth.small("c1_tiny", T=1, d=64, E=3, k=2, f=64, backward=True, seed=15),              # one token
    synth.small("c1_tiny", T=77, d=72, E=5, k=2, f=40, backward=True, seed=16),             # d, f multiples of 8 only
]


@pytest.mark.parametrize("w", SMALL, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}f{w.f}{'b' if w.backward else ''}")
@pytest.mark.parametrize("path", [binding.GEMM_SCALAR, binding.GEMM_AUTO, binding.GEMM_TENSOR_TN],
                         ids=["scalar", "auto", "tokens_on_n"])
def test_small_layers_match_oracle(w, path):
    if path == binding.GEMM_TENSOR_TN and (w.d % 64 or w.f % 64):
        with pytest.raises(binding.MopError) as e:      # a forced tensor-core schedule refuses odd shapes
            binding.context_for(w, gemm_path=path)
        assert e.value.code == 6
        return
    check_layer(w, path)


@pytest.mark.parametrize("path", [binding.GEMM_TENSOR_2CTA, binding.GEMM_TENSOR_MIXED, binding.GEMM_TENSOR_TN],
                         ids=["2cta", "mixed", "tokens_on_n"])
def test_two_cta_schedules_match_oracle_and_the_one_cta_kernel(path):
    w = synth.small("c2_mid", T=1500, d=256, E=6, k=2, f=320, backward=True, seed=21)   # 500 rows per expert
    _, buf = check_layer(w, path)
    _, _, _, ref = run(w, binding.GEMM_TENSOR_1CTA)
    for n in ("H", "Yp", "Y", "dX", "dW_gate", "dW_up", "dW_down"):   # same accumulation order
        assert torch.equal(getattr(buf, n), getattr(ref, n)), n
    # dgate is a sum over f whose partial sums are grouped by the kernel's tile shape
    assert torch.allclose(buf.dgate, ref.dgate, rtol=1e-4, atol=1e-4 * float(ref.dgate.abs().max()))


GATHER = [
    synth.small("c3_trillion", T=200, d=256, E=40, k=8, f=128, seed=41),      # 40 rows per expert: one ragged tile each
    synth.small("c2_mid", T=1500, d=256, E=6, k=2, f=320, seed=42),           # 500 rows per expert: two tiles
    synth.small("c4_skew", T=1024, d=192, E=16, k=4, f=192, seed=43),         # skewed counts, hot and empty experts
    synth.small("c1_tiny", T=3, d=64, E=5, k=1, f=64, seed=44),               # fewer rows than experts
]


@pytest.mark.parametrize("w", GATHER, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}f{w.f}")
def test_gathering_forward_matches_oracle_and_the_permuting_forward(w):
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    ctx = binding.context_for(w, backward=False)
    buf = binding.LayerBuffers(w)
    buf.Xp.fill_(float("nan"))                       # the gathering form must not touch (or need) Xp
    binding.forward(ctx, inp, buf, gather=True)
    binding.mop_poll(ctx)
    torch.cuda.synchronize()
    assert torch.isnan(buf.Xp.float()).all()
    xb, Wg, Wu, Wd = (synth.bits(host[n]) for n in ("x", "W_gate", "W_up", "W_down"))
    idx, _ = oracle.route(xb, host["W_r"].numpy(), np_bias(host), w.k, w.score_fn, w.bias_mode)
    assert np.array_equal(buf.idx.cpu().numpy(), idx)
    gate = buf.gate.cpu().numpy()
    Y_e = oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd)
    Y_d = oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd, declared=True)
    check_float("Y", buf.Y.float().cpu().numpy(), Y_e, Y_d, f"gather-{w.name}-T{w.T}")
    _, _, _, ref = run(dataclasses.replace(w, backward=False), binding.GEMM_TENSOR_TN, host)
    for n in ("H", "Yp", "Y"):                       # same tiles, same accumulation order
        assert torch.equal(getattr(buf, n), getattr(ref, n)), n


def test_gathering_forward_refuses_the_scalar_path():
    w = synth.small("c1_tiny", T=77, d=72, E=5, k=2, f=40, seed=16)
    host, inp, ctx, buf = run(w)
    with pytest.raises(binding.MopError) as e:
        binding.forward(ctx, inp, buf, gather=True)
    assert e.value.code == 6


def test_tokens_on_n_kernels_with_three_token_tiles_and_half_filled_k_stages():
    """700 rows per expert (three token tiles of 240) with d = 320 and f = 192: K is 2.5 and 1.5 pipeline
    stages of 128, so the last stage of every GEMM is half zero fill; all four token-row GEMMs forced
    onto the tokens-on-N kernel, compared with the oracle and bit for bit with the one-CTA kernel."""
    w = synth.small("c2_mid", T=1400, d=320, E=4, k=2, f=192, backward=True, seed=45)
    _, buf = check_layer(w, binding.GEMM_TENSOR_TN)
    assert int(buf.counts.max()) > 512
    _, _, _, ref = run(w, binding.GEMM_TENSOR_1CTA)
    for n in ("H", "Yp", "Y", "dX", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(getattr(buf, n), getattr(ref, n)), n


def test_all_keys_equal_goes_to_lowest_ids_and_leaves_experts_empty():
    w = synth.small("c1_tiny", T=96, d=64, E=6, k=2, f=64, backward=True, seed=17)
    host = synth.make_inputs(w, "cpu")
    host["W_r"] = torch.zeros_like(host["W_r"])
    host, inp, ctx, buf = run(w, host=host)
    assert np.array_equal(buf.idx.cpu().numpy(), np.tile(np.arange(2, dtype=np.int32), (96, 1)))
    assert np.array_equal(buf.counts.cpu().numpy(), np.array([96, 96, 0, 0, 0, 0], np.int32))
    assert torch.all(buf.dW_gate[2:] == 0) and torch.all(buf.dW_down[2:] == 0)
    check_integers(w, host, buf)


def test_an_overflowing_expert_does_not_reach_its_neighbours_gradients():
    """Backward with non-finite upstream gradients for the tokens of ONE expert (k = 1, so a token has one
    expert): that expert's gradients are lost, every other expert's dW and every other token's dX and dgate
    keep the bits of the clean run.  The rows of an expert end inside a 16-row K group of the weight-gradient
    GEMMs for all but a few experts here, so the K tail of the expert before the poisoned one is exercised."""
    w = synth.small("c5_train", T=1500, d=128, E=7, k=1, f=192, backward=True, seed=41)
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    for path in (binding.GEMM_AUTO, binding.GEMM_TENSOR_1CTA):
        ctx = binding.context_for(w, gemm_path=path)
        clean, bad = binding.LayerBuffers(w), binding.LayerBuffers(w)
        binding.forward(ctx, inp, clean)
        binding.backward(ctx, inp, clean)
        counts = clean.counts.cpu().numpy()
        e0 = int(np.argsort(counts)[len(counts) // 2])                    # an expert with rows, not the first one
        if e0 == 0:
            e0 = 1
        assert counts[e0] > 0 and counts[e0 - 1] % 16 != 0
        poisoned = dict(inp)
        dY = inp["dY"].clone()
        mine = (clean.idx[:, 0] == e0)
        dY[mine] = float("inf")
        dY[mine.nonzero()[::2, 0]] = float("nan")
        poisoned["dY"] = dY
        binding.forward(ctx, poisoned, bad)
        binding.backward(ctx, poisoned, bad)
        binding.mop_poll(ctx)
        others = torch.ones(w.E, dtype=torch.bool, device="cuda")
        others[e0] = False
        for name in ("dW_gate", "dW_up", "dW_down"):
            a, b = getattr(clean, name), getattr(bad, name)
            assert torch.equal(a[others], b[others]), f"{name} of the other experts (path {path})"
            assert not torch.isfinite(b[e0]).all(), f"{name} of the poisoned expert should be lost"
        assert torch.equal(clean.dX[~mine], bad.dX[~mine]) and torch.equal(clean.dgate[~mine], bad.dgate[~mine])


@pytest.mark.parametrize("T,k,E", [(2048, 2, 24), (2049, 2, 24), (4096, 1, 1024), (1025, 4, 7), (4609, 1, 3)])
def test_permutation_tables_on_both_sides_of_the_single_block_limit(T, k, E):
    """Up to 8 units of 512 assignments the permutation runs in one block, beyond that in three kernels: the tables
    must be the oracle's on both sides of that limit (and where the single block would not have the memory)."""
    gen = torch.Generator().manual_seed(T + E)
    idx = torch.stack([torch.randperm(E, generator=gen)[:k] for _ in range(T)]).to(torch.int32)
    counts, offsets, perm_row, row_src = oracle.permute(idx.numpy(), E)
    ctx = binding.Context(T, 64, E, k, 64)
    dev = {n: torch.empty(s, dtype=torch.int32, device="cuda") for n, s in
           (("counts", (E,)), ("offsets", (E + 1,)), ("perm_row", (T * k,)), ("row_src", (T * k,)))}
    x = torch.randn((T, 64)).to(torch.bfloat16).cuda()
    Xp = torch.empty((T * k, 64), dtype=torch.bfloat16, device="cuda")
    binding.mop_moe_permute(ctx, x, idx.cuda(), dev["counts"], dev["offsets"], dev["perm_row"], dev["row_src"], Xp)
    binding.mop_poll(ctx)
    assert np.array_equal(dev["counts"].cpu().numpy(), counts) and np.array_equal(dev["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(dev["perm_row"].cpu().numpy(), perm_row) and np.array_equal(dev["row_src"].cpu().numpy(), row_src)
    assert torch.equal(Xp.cpu(), x.cpu()[torch.from_numpy(row_src // k).long()])


def test_zero_tokens_is_a_no_op():
    w = synth.small("c1_tiny", T=0, d=64, E=4, k=2, f=64, backward=True)
    host, inp, ctx, buf = run(w)
    assert torch.all(buf.offsets == 0) and torch.all(buf.counts == 0)
    assert torch.all(buf.dW_gate == 0) and torch.all(buf.dW_up == 0) and torch.all(buf.dW_down == 0)


def test_results_are_bitwise_reproducible():
    w = synth.small("c2_mid", T=512, d=256, E=16, k=4, f=256, backward=True, seed=18)
    _, _, _, a = run(w)
    _, _, _, b = run(w)
    for n in ("idx", "gate", "perm_row", "Xp", "H", "Yp", "Y", "dX", "dgate", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(getattr(a, n), getattr(b, n)), n


def test_dw_accumulate_adds_into_existing_gradients():
    w = synth.small("c1_tiny", T=128, d=64, E=4, k=2, f=64, backward=True, seed=19)
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    ctx = binding.context_for(w, dw_accumulate=True)
    buf = binding.LayerBuffers(w)
    for t in (buf.dW_gate, buf.dW_up, buf.dW_down):
        t.fill_(1.0)
    binding.forward(ctx, inp, buf)
    binding.backward(ctx, inp, buf)
    _, _, _, ref = run(w, host=host)
    for n in ("dW_gate", "dW_up", "dW_down"):
        assert torch.allclose(getattr(buf, n), getattr(ref, n) + 1.0, atol=1e-5), n


def test_bad_arguments_return_codes():
    w = synth.WORKLOADS["c1_tiny"]
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_combine(ctx, None, buf.perm_row, buf.Y)
    assert e.value.code == 1
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_combine(ctx, buf.Yp.data_ptr() + 2, buf.perm_row, buf.Y)
    assert e.value.code == 3
    with pytest.raises(binding.MopError) as e:   # backward on a forward-only context
        binding.mop_moe_expert_ffn_bwd(ctx, *([buf.Yp] * 17))
    assert e.value.code == 6
    with pytest.raises(binding.MopError) as e:
        binding.Context(16, 64, 4, 5, 64)
    assert e.value.code == 1


def test_the_step_can_be_captured_into_a_cuda_graph_and_replayed():
    """The device entry points allocate nothing and never synchronise, so a whole step captures."""
    w = synth.small("c2_mid", T=512, d=256, E=16, k=4, f=192, backward=True, seed=29)
    host, inp, ctx, ref = run(w)
    buf = binding.LayerBuffers(w)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            binding.forward(ctx, inp, buf, side)
            binding.backward(ctx, inp, buf, side)
    torch.cuda.synchronize()
    for _ in range(2):                                  # replays are steps of their own
        for n in ("Y", "dX", "dgate", "dW_gate", "dW_up", "dW_down"):
            getattr(buf, n).zero_()
        graph.replay()
        torch.cuda.synchronize()
        for n in ("idx", "gate", "Y", "dX", "dgate", "dW_gate", "dW_up", "dW_down"):
            assert torch.equal(getattr(buf, n), getattr(ref, n)), n
    binding.mop_poll(ctx)


def test_largest_expert_count_and_routing_degree():
    """E = 1024 and k = 32 are the limits of the selection kernel; most experts get zero to four rows."""
    w = synth.small("c1_tiny", T=48, d=64, E=1024, k=32, f=64, backward=True, seed=27)
    _, buf = check_layer(w, binding.GEMM_AUTO)
    assert int((buf.counts == 0).sum()) > 0
    w2 = synth.small("c3_trillion", T=40, d=64, E=1024, k=32, f=64, seed=28)      # sigmoid + bias at the limits
    check_layer(w2, binding.GEMM_AUTO)


def test_shapes_beyond_the_limits_are_refused():
    for args, code in (((16, 64, 1025, 2, 64), 2), ((64, 64, 64, 33, 64), 2), ((16, 60, 4, 2, 64), 3),
                       ((16, 64, 4, 2, 36), 3), ((-1, 64, 4, 2, 64), 1), ((16, 64, 0, 1, 64), 1)):
        with pytest.raises(binding.MopError) as e:
            binding.Context(*args)
        assert e.value.code == code, args


def test_forward_host_entry_point_matches_device_path():
    w = synth.small("c2_mid", T=256, d=128, E=8, k=2, f=192, seed=20)
    host, inp, _, buf = run(w)
    ctx = binding.context_for(w, host_io=True)
    xh = host["x"].pin_memory()
    Yh = torch.empty_like(xh).pin_memory()
    idxh = torch.empty((w.T, w.k), dtype=torch.int32).pin_memory()
    gh = torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()
    binding.mop_moe_forward_host(ctx, xh, inp["W_r"], inp["bias"], inp["W_gate"], inp["W_up"], inp["W_down"], Yh, idxh,
                                 gh)
    assert torch.equal(Yh, buf.Y.cpu()) and torch.equal(idxh, buf.idx.cpu()) and torch.equal(gh, buf.gate.cpu())


@pytest.mark.parametrize("backward", [False, True], ids=["fwd", "train"])
def test_pipelined_host_steps_match_the_device_path_step_by_step(backward):
    """Five steps with different inputs in flight through the two slots; every step's results are its own."""
    w = synth.small("c2_mid", T=300, d=128, E=8, k=2, f=192, seed=23, backward=backward)
    steps = 5
    hosts = [synth.make_inputs(dataclasses.replace(w, seed=100 + i), "cpu") for i in range(steps)]
    weights = to_dev(hosts[0])                      # one set of weights, per-step activations
    ctx = binding.context_for(w, host_io=2)
    outs = []
    for h in hosts:
        o = {"x": h["x"].pin_memory(), "Y": torch.empty_like(h["x"]).pin_memory(),
             "idx": torch.empty((w.T, w.k), dtype=torch.int32).pin_memory(),
             "gate": torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()}
        if backward:
            o["dY"] = h["dY"].pin_memory()
            o["dX"] = torch.empty_like(h["x"]).pin_memory()
            o["dgate"] = torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()
        outs.append(o)
    dW = [torch.empty_like(weights[n], dtype=torch.float32) for n in ("W_gate", "W_up", "W_down")]
    for o in outs:
        if backward:
            binding.mop_moe_train_step_host_async(ctx, o["x"], o["dY"], weights["W_r"], weights["bias"],
                                                  weights["W_gate"], weights["W_up"], weights["W_down"], o["Y"],
                                                  o["dX"], o["dgate"], *dW)
        else:
            binding.mop_moe_forward_host_async(ctx, o["x"], weights["W_r"], weights["bias"], weights["W_gate"],
                                               weights["W_up"], weights["W_down"], o["Y"], o["idx"], o["gate"])
    binding.mop_host_drain(ctx)
    binding.mop_poll(ctx)
    ref_ctx = binding.context_for(w)
    for i, (h, o) in enumerate(zip(hosts, outs)):
        inp = dict(weights)
        inp["x"] = h["x"].cuda()
        if backward:
            inp["dY"] = h["dY"].cuda()
        buf = binding.LayerBuffers(w)
        binding.forward(ref_ctx, inp, buf)
        if backward:
            binding.backward(ref_ctx, inp, buf)
        torch.cuda.synchronize()
        assert torch.equal(o["Y"], buf.Y.cpu()), f"Y of step {i}"
        if backward:
            assert torch.equal(o["dX"], buf.dX.cpu()) and torch.equal(o["dgate"], buf.dgate.cpu()), f"step {i}"
        else:
            assert torch.equal(o["idx"], buf.idx.cpu()) and torch.equal(o["gate"], buf.gate.cpu()), f"step {i}"
    if backward:   # dW holds the last step's gradients
        for got, name in zip(dW, ("dW_gate", "dW_up", "dW_down")):
            assert torch.equal(got, getattr(buf, name)), name


def test_pipelined_host_entry_points_need_their_context_mode():
    w = synth.small("c1_tiny", T=8, d=64, E=4, k=2, f=64, seed=24)
    ctx = binding.context_for(w, host_io=True)
    with pytest.raises(binding.MopError) as e:
        binding.mop_host_drain(ctx)
    assert e.value.code == 6


ROUTER_BWD = [
    synth.small("c1_tiny", T=200, d=128, E=8, k=2, f=64, backward=True, seed=30),                       # softmax
    synth.small("c3_trillion", T=300, d=192, E=40, k=8, f=64, backward=True, seed=31),                  # sigmoid + post bias
    synth.small("c3_trillion", T=130, d=64, E=33, k=3, f=64, bias_mode=2, backward=True, seed=32),      # sigmoid, pre-logit bias
    synth.small("c2_mid", T=257, d=72, E=12, k=12, f=64, bias_mode=2, bias_std=0.1, backward=True, seed=33),  # softmax, k = E
]


@pytest.mark.parametrize("w", ROUTER_BWD, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}s{w.score_fn}b{w.bias_mode}")
def test_router_backward_matches_oracle(w):
    host = synth.make_inputs(w, "cpu")
    if w.bias_mode and host["bias"] is None:
        host["bias"] = torch.randn(w.E) * 0.1
    inp = to_dev(host)
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    logits = torch.empty((w.T, w.E), dtype=torch.float32, device="cuda")
    binding.mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], buf.idx, buf.gate, logits)
    binding.mop_moe_permute(ctx, inp["x"], buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp)
    g = torch.Generator().manual_seed(w.seed)
    dgate = torch.randn((w.T, w.k), generator=g).cuda()
    dX0 = (torch.randn((w.T, w.d), generator=g) * 0.5).to(torch.bfloat16).cuda()
    dX = dX0.clone()
    dWr = torch.full((w.d, w.E), 7.0, device="cuda")
    dbias = torch.full((w.E,), 7.0, device="cuda")
    binding.mop_moe_route_bwd(ctx, logits, inp["bias"], buf.idx, buf.gate, dgate, buf.Xp, buf.offsets, buf.perm_row,
                              inp["W_r"], dWr, dbias, dX)
    torch.cuda.synchronize()
    bias = None if host["bias"] is None else host["bias"].numpy()
    idx = buf.idx.cpu().numpy()
    dz, dWr_ref, dXr_ref, db_ref = oracle.route_bwd(synth.bits(host["x"]), host["W_r"].numpy(), bias, w.k, w.score_fn,
                                                    w.bias_mode, idx, dgate.cpu().numpy())
    assert rel_fro(dWr.cpu().numpy(), dWr_ref) < 1e-5
    assert np.max(np.abs(dbias.cpu().numpy() - db_ref)) <= 1e-5 * max(1.0, np.abs(db_ref).max())
    # dX = bf16(dX_in + router part): one bf16 rounding of the sum
    want = dX0.float().cpu().numpy().astype(np.float64) + dXr_ref
    got = dX.float().cpu().numpy()
    assert np.max(np.abs(got - want)) <= 2.0 ** -8 * np.maximum(1.0, np.abs(want)).max()
    assert rel_fro(got, want) < 4e-3


def test_backward_with_recomputation_equals_backward_with_stash():
    """Activation checkpointing: forward without the G, U stash, backward recomputes them from Xp."""
    w = synth.small("c2_mid", T=700, d=256, E=10, k=3, f=192, backward=True, seed=40)
    host, inp, _, ref = run(w)
    ctx = binding.Context(w.T, w.d, w.E, w.k, w.f, w.score_fn, w.bias_mode, 2)
    buf = binding.LayerBuffers(w)
    binding.mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], buf.idx, buf.gate)
    binding.mop_moe_permute(ctx, inp["x"], buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp)
    binding.mop_moe_expert_ffn_fwd(ctx, buf.Xp, buf.offsets, buf.row_src, buf.gate, inp["W_gate"], inp["W_up"],
                                   inp["W_down"], None, None, buf.H, buf.Yp)
    binding.mop_moe_combine(ctx, buf.Yp, buf.perm_row, buf.Y)
    binding.mop_moe_expert_ffn_bwd(ctx, inp["dY"], buf.Xp, None, None, None, buf.offsets, buf.perm_row, buf.row_src,
                                   buf.gate, inp["W_gate"], inp["W_up"], inp["W_down"], buf.dX, buf.dW_gate, buf.dW_up,
                                   buf.dW_down, buf.dgate)
    binding.mop_poll(ctx)
    for n in ("Y", "dX", "dgate", "dW_gate", "dW_up", "dW_down"):
        assert torch.equal(getattr(buf, n), getattr(ref, n)), n
    plain = binding.context_for(w)                      # a context without the recompute buffers refuses
    with pytest.raises(binding.MopError) as e:
        binding.mop_moe_expert_ffn_bwd(plain, inp["dY"], buf.Xp, None, None, None, buf.offsets, buf.perm_row,
                                       buf.row_src, buf.gate, inp["W_gate"], inp["W_up"], inp["W_down"], buf.dX,
                                       buf.dW_gate, buf.dW_up, buf.dW_down, buf.dgate)
    assert e.value.code == 6


def test_random_small_shapes_match_oracle():
    """Seeded random shapes: E not a multiple of 32, k from 1 to E, d and f multiples of 8 (scalar
    kernels) or of 64 (tensor-core kernels), tokens that leave experts empty."""
    rng = np.random.default_rng(1234)
    for i in range(10):
        E = int(rng.integers(1, 70))
        k = int(rng.integers(1, min(E, 8) + 1))
        if i % 2:
            d, f = int(rng.integers(1, 5)) * 64, int(rng.integers(1, 5)) * 64
        else:
            d, f = int(rng.integers(2, 20)) * 8, int(rng.integers(2, 20)) * 8
        T = int(rng.integers(1, 400))
        mode = [(0, 0), (1, 1), (1, 2), (0, 2), (1, 0)][i % 5]
        w = synth.small("c1_tiny", T=T, d=d, E=E, k=k, f=f, score_fn=mode[0], bias_mode=mode[1], bias_std=0.05,
                        backward=True, seed=100 + i)
        check_layer(w, binding.GEMM_AUTO)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Failure path without a fault: a device-side wait on a barrier that nothing completes gives up
    after its limit, records a code, the kernel returns; mop_poll reports MOP_ERR_TIMEOUT once, and
    the same context then runs the layer correctly."""
    w = synth.small("c1_tiny", backward=True)
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    ctx = binding.context_for(w)
    buf = binding.LayerBuffers(w)
    binding.mop_selftest_wait_timeout(ctx, 20_000_000)          # about 10 ms of SM cycles
    with pytest.raises(binding.MopError) as e:
        binding.mop_poll(ctx)
    assert e.value.code == 7
    binding.mop_poll(ctx)                                        # the word was cleared
    binding.forward(ctx, inp, buf)
    binding.backward(ctx, inp, buf)
    binding.mop_poll(ctx)
    check_integers(w, host, buf)


FAST_ROUTE = [
    synth.small("c3_trillion", T=1000, d=512, E=256, k=8, f=64, seed=60),                  # sigmoid + post-score bias
    synth.small("c3_trillion", T=777, d=320, E=64, k=3, f=64, bias_mode=2, seed=61),        # sigmoid, bias before the score
    synth.small("c2_mid", T=900, d=256, E=128, k=6, f=64, seed=62),                         # softmax
    synth.small("c3_trillion", T=300, d=192, E=1024, k=32, f=64, seed=63),                  # the selection's limits
    synth.small("c2_mid", T=257, d=64, E=64, k=32, f=64, seed=64),                          # half of the experts picked
    synth.small("c3_trillion", T=130, d=7168, E=384, k=8, f=64, seed=65),                   # the long chains of configs 3-5
    synth.small("c3_trillion", T=600, d=448, E=64, k=4, f=64, seed=66),                     # one narrow tile of experts, K in halves
    synth.small("c3_trillion", T=520, d=512, E=320, k=8, f=64, seed=67),                    # a wide tile and 64 more experts
]


@pytest.mark.parametrize("w", FAST_ROUTE, ids=lambda w: f"{w.name}-T{w.T}d{w.d}E{w.E}k{w.k}s{w.score_fn}b{w.bias_mode}")
def test_tensor_core_scoring_gives_the_indices_of_the_exact_chains(w):
    """Logits from three bf16 pieces of W_r on the tensor cores, the contract's chain only where the order is in
    doubt: indices and their order equal the oracle's (and the exact path's) bit for bit, gates within tolerance,
    and the returned logits are the chain's value or within the documented bound of it."""
    host = synth.make_inputs(w, "cpu")
    inp = to_dev(host)
    out = {}
    for path in (binding.ROUTE_EXACT, binding.ROUTE_TENSOR):
        ctx = binding.context_for(w, route_path=path)
        idx = torch.empty((w.T, w.k), dtype=torch.int32, device="cuda")
        gate = torch.empty((w.T, w.k), dtype=torch.float32, device="cuda")
        logits = torch.empty((w.T, w.E), dtype=torch.float32, device="cuda")
        binding.mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], idx, gate, logits)
        binding.mop_poll(ctx)
        out[path] = (idx.cpu().numpy(), gate.cpu().numpy(), logits.cpu().numpy(), binding.mop_route_stats(ctx))
    xb = synth.bits(host["x"])
    ref_idx, ref_gate, ref_z, _ = oracle.route(xb, host["W_r"].numpy(), np_bias(host), w.k, w.score_fn, w.bias_mode,
                                               want_logits=True)
    for path, (idx, gate, z, stats) in out.items():
        assert np.array_equal(idx, ref_idx), f"indices, route path {path}"
        assert np.all(np.abs(gate - ref_gate) <= 1e-6 + 1e-5 * np.abs(ref_gate)), f"gates, route path {path}"
    assert np.array_equal(out[binding.ROUTE_EXACT][2], ref_z)                       # the chain, bit for bit
    assert out[binding.ROUTE_EXACT][3] == (0, 0, 0)
    # the approximate logits stay inside the bound the selection relies on (and far inside it)
    z = out[binding.ROUTE_TENSOR][2]
    xn = np.linalg.norm(oracle.bf16_bits_to_f64(xb), axis=1)
    wmax = np.linalg.norm(host["W_r"].numpy().astype(np.float64), axis=0).max()
    eps = 24.0 * 2.0 ** -24 * xn * wmax
    err = np.abs(z.astype(np.float64) - ref_z.astype(np.float64)).max(1)
    assert np.all(err <= eps), float((err / eps).max())
    tokens, chains, beyond = out[binding.ROUTE_TENSOR][3]
    print(f"{w.name} T={w.T} d={w.d} E={w.E}: logit error {err.max():.2e} = {float((err / eps).max()):.3f} of the bound; "
          f"{tokens} of {w.T} tokens re-evaluated, {chains} chains")
    assert 0 <= tokens <= w.T and chains >= tokens and beyond == 0
    assert float((err / eps).max()) < 0.5


def test_tensor_core_scoring_with_equal_and_duplicate_keys():
    """W_r = 0 makes all keys of a token equal (every expert is re-evaluated and the lower ids win); two equal
    columns of W_r make one exact tie per token that only the chain can order."""
    w = synth.small("c2_mid", T=96, d=128, E=64, k=4, f=64, seed=66)
    host = synth.make_inputs(w, "cpu")
    for mode in ("zero", "duplicate"):
        Wr = torch.zeros_like(host["W_r"]) if mode == "zero" else host["W_r"].clone()
        if mode == "duplicate":
            Wr[:, 40] = Wr[:, 3]
        ctx = binding.context_for(w, route_path=binding.ROUTE_TENSOR)
        idx = torch.empty((w.T, w.k), dtype=torch.int32, device="cuda")
        gate = torch.empty((w.T, w.k), dtype=torch.float32, device="cuda")
        binding.mop_moe_route(ctx, host["x"].cuda(), Wr.cuda(), None, idx, gate)
        binding.mop_poll(ctx)
        ref_idx, ref_gate = oracle.route(synth.bits(host["x"]), Wr.numpy(), None, w.k, w.score_fn, w.bias_mode)
        assert np.array_equal(idx.cpu().numpy(), ref_idx), mode
        assert np.all(np.abs(gate.cpu().numpy() - ref_gate) <= 1e-6 + 1e-5 * np.abs(ref_gate)), mode
        if mode == "zero":
            assert binding.mop_route_stats(ctx) == (w.T, w.T * w.E, 0)


def test_tensor_core_scoring_refuses_shapes_it_cannot_take():
    with pytest.raises(binding.MopError) as e:
        binding.Context(64, 64, 40, 2, 64, route_path=binding.ROUTE_TENSOR)      # E not a multiple of 64
    assert e.value.code == 6
