"""Pins for the CPU oracle: every function is checked against something other than itself --
brute force, closed forms, library routines on special cases, automatic differentiation and
finite differences.  None of these tests touches the CUDA path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_01844_b200 import synth


def _rand_bits(rng, shape, std=1.0):
    t = torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * std).to(torch.bfloat16)
    return synth.bits(t)


def _small(rng, T=12, d=16, E=4, k=2, f=24):
    x = _rand_bits(rng, (T, d))
    Wg = _rand_bits(rng, (E, d, f), 0.3)
    Wu = _rand_bits(rng, (E, d, f), 0.3)
    Wd = _rand_bits(rng, (E, f, d), 0.3)
    Wr = (rng.standard_normal((d, E)) * 0.5).astype(np.float32)
    return x, Wg, Wu, Wd, Wr


# ------------------------------------------------------------------------------ bf16 rounding
def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.0078125, 1.01171875, 3.3895314e38, 1e-40],
                                 np.float32)])
    got = oracle.f32_to_bf16_bits(v)
    ref = synth.bits(torch.from_numpy(v).to(torch.bfloat16))
    assert np.array_equal(got, ref)
    # halfway cases go to the even neighbour
    assert oracle.bf16_bits_to_f32(oracle.f32_to_bf16_bits(np.float32([1.00390625])))[0] == 1.0
    assert oracle.bf16_bits_to_f32(oracle.f32_to_bf16_bits(np.float32([1.01171875])))[0] == 1.015625


# ------------------------------------------------------------------------------ sigmoid contract
def test_sigmoid_contract_close_to_true_sigmoid_and_monotone():
    z = np.linspace(-30, 30, 20001).astype(np.float32)
    s = oracle.sigmoid_contract(z)
    ref = 1.0 / (1.0 + np.exp(-z.astype(np.float64)))
    assert np.max(np.abs(s - ref)) < 3e-7
    assert np.all(np.diff(s.astype(np.float64)) >= -1.2e-7)  # monotone up to one ulp near 1
    assert oracle.sigmoid_contract(np.float32([0.0]))[0] == 0.5
    # saturation is finite and ordered
    lo, hi = oracle.sigmoid_contract(np.float32([-200.0, 200.0]))
    assert 0.0 <= lo < 1e-30 and hi == 1.0


# ------------------------------------------------------------------------------ router
@pytest.mark.parametrize("score_fn,bias_mode", [(0, 0), (0, 2), (1, 0), (1, 1), (1, 2)])
def test_topk_matches_brute_force_sort(score_fn, bias_mode):
    rng = np.random.default_rng(1)
    for (T, d, E, k) in [(64, 16, 16, 4), (33, 24, 7, 7), (20, 8, 5, 1)]:
        x = _rand_bits(rng, (T, d))
        Wr = (rng.standard_normal((d, E)) * 0.4).astype(np.float32)
        b = (rng.standard_normal(E) * 0.05).astype(np.float32) if bias_mode else None
        idx, gate, z, key = oracle.route(x, Wr, b, k, score_fn, bias_mode, want_logits=True)
        # logits: exact value within fp32 accumulation error of the fp64 product
        zref = oracle.bf16_bits_to_f64(x) @ Wr.astype(np.float64)
        assert np.max(np.abs(z - zref)) < 1e-5
        # independent selection: full stable sort of (-key, id)
        for t in range(T):
            order = sorted(range(E), key=lambda e: (-float(key[t, e]), e))
            assert list(idx[t]) == order[:k]
        # gates: closed forms in fp64
        if score_fn == 0:
            zz = key.astype(np.float64)
            p = np.exp(zz - zz.max(1, keepdims=True))
            p /= p.sum(1, keepdims=True)
        else:
            zz = (z + b if bias_mode == 2 else z).astype(np.float64)
            p = 1 / (1 + np.exp(-zz))
        sel = np.take_along_axis(p, idx.astype(np.int64), 1)
        gref = sel / sel.sum(1, keepdims=True)
        assert np.max(np.abs(gate - gref)) < 1e-6
        assert np.all(gate > 0) and np.allclose(gate.sum(1), 1.0, atol=1e-6)
        if score_fn == 0:
            # renormalised softmax equals a softmax over the selected logits alone
            zs = np.take_along_axis(key.astype(np.float64), idx.astype(np.int64), 1)
            q = np.exp(zs - zs.max(1, keepdims=True))
            assert np.max(np.abs(gate - q / q.sum(1, keepdims=True))) < 1e-6


def test_logit_chain_is_the_sequential_fma_order():
    """The logit is one fused multiply-add per i, ascending; emulate it exactly in fp64:
    the product of a bf16 by an fp32 and its sum with an fp32 are exact in fp64 up to one
    rounding, and double rounding is excluded here by checking the result against both
    neighbours."""
    rng = np.random.default_rng(2)
    T, d, E = 8, 96, 5
    x = _rand_bits(rng, (T, d))
    Wr = (rng.standard_normal((d, E)) * 0.2).astype(np.float32)
    _, _, z, _ = oracle.route(x, Wr, None, 1, 0, 0, want_logits=True)
    xf = oracle.bf16_bits_to_f64(x)
    acc = np.zeros((T, E), np.float32)
    for i in range(d):
        exact = xf[:, i:i + 1] * Wr[i:i + 1, :].astype(np.float64) + acc.astype(np.float64)
        acc = exact.astype(np.float32)
    # a blocked (pairwise) order differs; the sequential order matches to the last bit
    # except where fp64 double rounding could occur (none observed for this seed)
    assert np.array_equal(acc, z)


def test_tie_break_goes_to_lower_expert_id():
    T, d, E, k = 9, 8, 6, 3
    x = _rand_bits(np.random.default_rng(3), (T, d))
    for score_fn, bias_mode in [(0, 0), (1, 0), (1, 1)]:
        b = np.zeros(E, np.float32) if bias_mode else None
        idx, gate = oracle.route(x, np.zeros((d, E), np.float32), b, k, score_fn, bias_mode)
        assert np.array_equal(idx, np.tile(np.arange(k, dtype=np.int32), (T, 1)))
        assert np.allclose(gate, 1.0 / k, atol=1e-7)
        counts, offsets, _, _ = oracle.permute(idx, E)
        assert list(counts) == [T] * k + [0] * (E - k)
    # two identical router columns: the lower id always precedes the higher one
    rng = np.random.default_rng(4)
    Wr = (rng.standard_normal((d, E)) * 0.4).astype(np.float32)
    Wr[:, 4] = Wr[:, 1]
    idx, _ = oracle.route(x, Wr, None, E, 0, 0)
    for t in range(T):
        row = list(idx[t])
        assert row.index(1) + 1 == row.index(4)


def test_k_equals_E_gives_full_softmax():
    rng = np.random.default_rng(5)
    T, d, E = 10, 12, 6
    x = _rand_bits(rng, (T, d))
    Wr = (rng.standard_normal((d, E)) * 0.4).astype(np.float32)
    idx, gate, z, _ = oracle.route(x, Wr, None, E, 0, 0, want_logits=True)
    p = torch.softmax(torch.from_numpy(z).double(), 1).numpy()
    assert np.max(np.abs(gate - np.take_along_axis(p, idx.astype(np.int64), 1))) < 1e-6


def test_select_agrees_with_route():
    rng = np.random.default_rng(6)
    x = _rand_bits(rng, (40, 16))
    Wr = (rng.standard_normal((16, 9)) * 0.4).astype(np.float32)
    b = (rng.standard_normal(9) * 0.05).astype(np.float32)
    idx, gate, z, key = oracle.route(x, Wr, b, 3, 1, 1, want_logits=True)
    idx2, gate2 = oracle.select(key, z, 3, 1)
    assert np.array_equal(idx, idx2) and np.array_equal(gate, gate2)


# ------------------------------------------------------------------------------ permutation
def test_permutation_is_the_stable_sort_by_expert():
    rng = np.random.default_rng(7)
    for (T, k, E) in [(50, 3, 7), (1, 1, 1), (64, 2, 16), (17, 4, 4)]:
        idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
        counts, offsets, perm_row, row_src = oracle.permute(idx, E)
        flat = idx.reshape(-1)
        assert counts.sum() == T * k and np.array_equal(counts, np.bincount(flat, minlength=E))
        assert offsets[0] == 0 and offsets[-1] == T * k and np.all(np.diff(offsets) == counts)
        order = np.argsort(flat, kind="stable").astype(np.int32)
        assert np.array_equal(row_src, order)
        assert np.array_equal(perm_row[row_src], np.arange(T * k))
        assert np.array_equal(row_src[perm_row], np.arange(T * k))
        for e in range(E):
            seg = row_src[offsets[e]:offsets[e + 1]]
            assert np.all(flat[seg] == e) and np.all(np.diff(seg) > 0)
        assert np.array_equal(np.sort(row_src // k), np.repeat(np.arange(T), k))


# ------------------------------------------------------------------------------ forward
def _torch_layer(x, idx, gate, Wg, Wu, Wd):
    """The layer written with library ops and automatic differentiation, in fp64."""
    T, k = idx.shape
    Y = torch.zeros(T, x.shape[1], dtype=torch.float64)
    for t in range(T):
        for j in range(k):
            e = int(idx[t, j])
            h = torch.nn.functional.silu(x[t] @ Wg[e]) * (x[t] @ Wu[e])
            Y[t] = Y[t] + gate[t, j] * (h @ Wd[e])
    return Y


def test_forward_single_expert_is_a_dense_swiglu_mlp():
    rng = np.random.default_rng(8)
    x, Wg, Wu, Wd, _ = _small(rng, T=9, d=16, E=1, k=1, f=40)
    idx = np.zeros((9, 1), np.int32)
    gate = np.ones((9, 1), np.float32)
    xf, g, u, dn = (oracle.bf16_bits_to_f64(a) for a in (x, Wg[0], Wu[0], Wd[0]))
    a = xf @ g
    ref = ((a / (1 + np.exp(-a))) * (xf @ u)) @ dn
    Y32 = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd)
    Y64 = oracle.ffn_fwd(xf, idx, gate, *(oracle.bf16_bits_to_f64(w) for w in (Wg, Wu, Wd)), fp64=True)
    assert np.max(np.abs(Y64 - ref)) < 1e-12
    assert np.max(np.abs(Y32 - ref)) < 1e-4 * max(1.0, np.abs(ref).max())


def test_forward_k_equals_E_is_the_dense_mixture_and_parts_are_consistent():
    rng = np.random.default_rng(9)
    x, Wg, Wu, Wd, Wr = _small(rng, T=7, d=16, E=3, k=3, f=24)
    idx, gate = oracle.route(x, Wr, None, 3, 0, 0)
    xf, Wgf, Wuf, Wdf = (oracle.bf16_bits_to_f64(a) for a in (x, Wg, Wu, Wd))
    A = np.einsum("td,edf->tef", xf, Wgf)
    Bm = np.einsum("td,edf->tef", xf, Wuf)
    Hm = A / (1 + np.exp(-A)) * Bm
    Om = np.einsum("tef,efd->ted", Hm, Wdf)
    p = np.zeros((7, 3))
    np.put_along_axis(p, idx.astype(np.int64), gate.astype(np.float64), 1)
    ref = np.einsum("te,ted->td", p, Om)
    Y, G, U, H, Yp = oracle.ffn_fwd(xf, idx, gate, Wgf, Wuf, Wdf, fp64=True, want_parts=True)
    assert np.max(np.abs(Y - ref)) < 1e-12
    for t in range(7):
        for j in range(3):
            e = idx[t, j]
            assert np.max(np.abs(G[t, j] - A[t, e])) < 1e-12
            assert np.max(np.abs(U[t, j] - Bm[t, e])) < 1e-12
            assert np.max(np.abs(H[t, j] - Hm[t, e])) < 1e-12
            assert np.max(np.abs(Yp[t, j] - gate[t, j].astype(np.float64) * Om[t, e])) < 1e-12
    assert np.max(np.abs(Yp.sum(1) - Y)) < 1e-12


def test_forward_invariances():
    rng = np.random.default_rng(10)
    x, Wg, Wu, Wd, Wr = _small(rng, T=10, d=16, E=5, k=2, f=24)
    idx, gate = oracle.route(x, Wr, None, 2, 0, 0)
    Y = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd)
    # W_down = 0 -> Y = 0
    assert np.all(oracle.ffn_fwd(x, idx, gate, Wg, Wu, np.zeros_like(Wd)) == 0)
    # linear in W_down: doubling is exact in binary floating point
    Wd2 = synth.bits((torch.from_numpy(oracle.bf16_bits_to_f32(Wd)) * 2).to(torch.bfloat16))
    assert np.array_equal(oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd2), 2 * Y)
    # token permutation equivariance (bitwise: each token is computed on its own)
    perm = rng.permutation(10)
    assert np.array_equal(oracle.ffn_fwd(x[perm], idx[perm], gate[perm], Wg, Wu, Wd), Y[perm])
    # expert relabelling invariance
    rel = rng.permutation(5)             # new id of old expert e is rel[e]
    inv = np.argsort(rel)
    assert np.array_equal(oracle.ffn_fwd(x, rel[idx].astype(np.int32), gate, Wg[inv], Wu[inv], Wd[inv]), Y)
    # token list = slice of the full result
    toks = np.array([7, 2, 2, 9], np.int32)
    assert np.array_equal(oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd, toks=toks), Y[toks])
    # fp32 and fp64 instantiations agree
    Y64 = oracle.ffn_fwd(oracle.bf16_bits_to_f64(x), idx, gate, *(oracle.bf16_bits_to_f64(w) for w in (Wg, Wu, Wd)),
                         fp64=True)
    assert np.linalg.norm(Y - Y64) / np.linalg.norm(Y64) < 1e-5


# ------------------------------------------------------------------------------ backward
def _setup_bwd(seed, T=6, d=12, E=3, k=2, f=16):
    rng = np.random.default_rng(seed)
    x, Wg, Wu, Wd, Wr = _small(rng, T=T, d=d, E=E, k=k, f=f)
    dY = _rand_bits(rng, (T, d))
    idx, gate = oracle.route(x, Wr, None, k, 0, 0)
    return x, dY, idx, gate, Wg, Wu, Wd


def test_backward_matches_automatic_differentiation_fp64():
    x, dY, idx, gate, Wg, Wu, Wd = _setup_bwd(11)
    E = Wg.shape[0]
    xf, dYf, Wgf, Wuf, Wdf = (oracle.bf16_bits_to_f64(a) for a in (x, dY, Wg, Wu, Wd))
    tx, tg, tWg, tWu, tWd = (torch.tensor(a, dtype=torch.float64, requires_grad=True)
                             for a in (xf, gate.astype(np.float64), Wgf, Wuf, Wdf))
    Y = _torch_layer(tx, idx, tg, tWg, tWu, tWd)
    (Y * torch.from_numpy(dYf)).sum().backward()
    dX, dgate = oracle.ffn_bwd_tokens(xf, dYf, idx, gate, Wgf, Wuf, Wdf, fp64=True)
    dWg, dWu, dWd = oracle.ffn_bwd_experts(xf, dYf, idx, gate, Wgf, Wuf, Wdf, np.arange(E), fp64=True)
    for got, ref in [(dX, tx.grad), (dgate, tg.grad), (dWg, tWg.grad), (dWu, tWu.grad), (dWd, tWd.grad)]:
        ref = ref.numpy()
        assert np.max(np.abs(got - ref)) <= 1e-10 * max(1.0, np.abs(ref).max())
    # the fp32 instantiation follows within single-precision error
    dX32, dgate32 = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd)
    dWg32, dWu32, dWd32 = oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, np.arange(E))
    for got, ref in [(dX32, dX), (dgate32, dgate), (dWg32, dWg), (dWu32, dWu), (dWd32, dWd)]:
        assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref)


def test_backward_matches_central_finite_differences_fp64():
    x, dY, idx, gate, Wg, Wu, Wd = _setup_bwd(12, T=4, d=8, E=3, k=2, f=8)
    E = Wg.shape[0]
    xf, R, Wgf, Wuf, Wdf = (oracle.bf16_bits_to_f64(a) for a in (x, dY, Wg, Wu, Wd))
    g64 = gate.astype(np.float64)

    def loss(xx, gg, a, b, c):
        return float((oracle.ffn_fwd(xx, idx, gg, a, b, c, fp64=True) * R).sum())

    dX, dgate = oracle.ffn_bwd_tokens(xf, R, idx, g64, Wgf, Wuf, Wdf, fp64=True)
    dWg, dWu, dWd = oracle.ffn_bwd_experts(xf, R, idx, g64, Wgf, Wuf, Wdf, np.arange(E), fp64=True)
    args = [xf, g64, Wgf, Wuf, Wdf]
    grads = [dX, dgate, dWg, dWu, dWd]
    rng = np.random.default_rng(13)
    h = 1e-5
    for which, (arr, grad) in enumerate(zip(args, grads)):
        for _ in range(12):
            pos = tuple(rng.integers(0, s) for s in arr.shape)
            up = [a.copy() for a in args]
            dn = [a.copy() for a in args]
            up[which][pos] += h
            dn[which][pos] -= h
            fd = (loss(*up) - loss(*dn)) / (2 * h)
            assert abs(fd - grad[pos]) <= 1e-6 * max(1.0, abs(grad[pos])), (which, pos, fd, grad[pos])


def test_backward_identities_and_untouched_experts():
    x, dY, idx, gate, Wg, Wu, Wd = _setup_bwd(14, T=8, d=12, E=6, k=2, f=16)
    idx = np.where(idx == 5, 0, idx).astype(np.int32)          # expert 5 receives nothing
    idx[:, 1] = np.where(idx[:, 1] == idx[:, 0], (idx[:, 0] + 1) % 5, idx[:, 1])
    Y = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd)
    dX, dgate = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd)
    dYf = oracle.bf16_bits_to_f32(dY)
    # sum_j g * dgate = <dY, Y> per token (Y is linear in the gates)
    lhs = (gate * dgate).sum(1)
    rhs = (dYf * Y).sum(1)
    assert np.max(np.abs(lhs - rhs)) < 1e-4 * max(1.0, np.abs(rhs).max())
    dWg, dWu, dWd = oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, np.array([5, 0], np.int32))
    assert np.all(dWg[0] == 0) and np.all(dWu[0] == 0) and np.all(dWd[0] == 0)
    assert np.abs(dWd[1]).max() > 0
    # token list = slice of the full result
    toks = np.array([5, 1], np.int32)
    dXs, dgs = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd, toks=toks)
    assert np.array_equal(dXs, dX[toks]) and np.array_equal(dgs, dgate[toks])


# ------------------------------------------------------------------------------ the two modes
def test_declared_rounding_mode_stays_close_to_exact_mode():
    rng = np.random.default_rng(15)
    T, d, E, k, f = 24, 64, 4, 2, 96
    x = _rand_bits(rng, (T, d))
    dY = _rand_bits(rng, (T, d))
    Wg, Wu = _rand_bits(rng, (E, d, f), 0.1), _rand_bits(rng, (E, d, f), 0.1)
    Wd = _rand_bits(rng, (E, f, d), 0.1)
    Wr = (rng.standard_normal((d, E)) * 0.2).astype(np.float32)
    idx, gate = oracle.route(x, Wr, None, k, 0, 0)
    ex = (oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd), *oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd),
          *oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, np.arange(E)))
    de = (oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd, declared=True),
          *oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd, declared=True),
          *oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, np.arange(E), declared=True))
    for a, b in zip(ex, de):
        rel = np.linalg.norm(a - b) / np.linalg.norm(a)
        assert 0 < rel < 5e-3
    # outputs declared bf16 are representable in bf16
    for b in de[:2]:
        assert np.array_equal(oracle.bf16_bits_to_f32(synth.bits(torch.from_numpy(b).to(torch.bfloat16))), b)


ROUNDING_POINTS = ("H", "G_save", "U_save", "Yp", "Y", "dG", "dU", "gH", "dXp", "dX")


def _layer_with_roundings(x, dY, idx, gate, Wg, Wu, Wd, points):
    """The layer and its backward written with library ops in fp64, rounding to bf16 (nearest even,
    through the library's own conversion) at exactly the tensors named in `points` and nowhere else.
    Returns the same outputs as the oracle: Y, G, U, H [T,k,f], Yp [T,k,d], dX, dgate, dW_gate, dW_up, dW_down."""
    def r(name, v):
        return v.to(torch.float32).to(torch.bfloat16).to(torch.float64) if name in points else v

    x, dY, Wg, Wu, Wd = (torch.from_numpy(oracle.bf16_bits_to_f64(a)) for a in (x, dY, Wg, Wu, Wd))
    g_all = torch.from_numpy(gate.astype(np.float64))
    T, k = idx.shape
    E, d, f = Wg.shape
    out = {"Y": torch.zeros(T, d, dtype=torch.float64), "G": torch.zeros(T, k, f, dtype=torch.float64),
           "U": torch.zeros(T, k, f, dtype=torch.float64), "H": torch.zeros(T, k, f, dtype=torch.float64),
           "Yp": torch.zeros(T, k, d, dtype=torch.float64), "dX": torch.zeros(T, d, dtype=torch.float64),
           "dgate": torch.zeros(T, k, dtype=torch.float64), "dW_gate": torch.zeros(E, d, f, dtype=torch.float64),
           "dW_up": torch.zeros(E, d, f, dtype=torch.float64), "dW_down": torch.zeros(E, f, d, dtype=torch.float64)}
    for t in range(T):
        y = torch.zeros(d, dtype=torch.float64)
        dx = torch.zeros(d, dtype=torch.float64)
        for j in range(k):
            e, g = int(idx[t, j]), g_all[t, j]
            G, U = x[t] @ Wg[e], x[t] @ Wu[e]                    # fp32 accumulators on the device: not rounded
            H = r("H", torch.nn.functional.silu(G) * U)          # H is made from the unrounded G, U
            Gs, Us = r("G_save", G), r("U_save", U)              # the stash that the backward reads
            Yp = r("Yp", g * (H @ Wd[e]))
            y = y + Yp
            dHu = Wd[e] @ dY[t]                                  # dY W_down^T, kept in fp32
            s = torch.sigmoid(Gs)
            dH = g * dHu
            dG = r("dG", dH * Us * s * (1 + Gs * (1 - s)))
            dU = r("dU", dH * (Gs * s))
            gH = r("gH", g * H)
            dXp = r("dXp", Wg[e] @ dG + Wu[e] @ dU)
            dx = dx + dXp
            out["G"][t, j], out["U"][t, j], out["H"][t, j], out["Yp"][t, j] = Gs, Us, H, Yp
            out["dgate"][t, j] = dHu @ H
            out["dW_gate"][e] += torch.outer(x[t], dG)
            out["dW_up"][e] += torch.outer(x[t], dU)
            out["dW_down"][e] += torch.outer(gH, dY[t])
        out["Y"][t] = r("Y", y)
        out["dX"][t] = r("dX", dx)
    return {n: v.numpy() for n, v in out.items()}


def test_declared_rounding_mode_rounds_at_exactly_the_declared_tensors():
    """Pin of the declared-rounding mode.  An independent restatement (library ops, fp64, the library's
    bf16 conversion) that rounds at the ten declared tensors must reproduce every output of the
    oracle's declared mode to fp32 round-off; the same restatement with any ONE rounding point
    removed must miss some output by far more than that, so a dropped or misplaced rounding in the
    oracle cannot pass.  With no rounding point at all it must reproduce the exact mode."""
    rng = np.random.default_rng(77)
    T, d, E, k, f = 8, 16, 3, 2, 16
    x, dY = _rand_bits(rng, (T, d)), _rand_bits(rng, (T, d))
    Wg, Wu, Wd = (_rand_bits(rng, s, 0.35) for s in ((E, d, f), (E, d, f), (E, f, d)))
    Wr = (rng.standard_normal((d, E)) * 0.5).astype(np.float32)
    idx, gate = oracle.route(x, Wr, None, k, 0, 0)
    ex = np.arange(E, dtype=np.int32)

    def oracle_outputs(declared):
        Y, G, U, H, Yp = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd, declared=declared, want_parts=True)
        dX, dgate = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd, declared=declared)
        dWg, dWu, dWd = oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, ex, declared=declared)
        return {"Y": Y, "G": G, "U": U, "H": H, "Yp": Yp, "dX": dX, "dgate": dgate, "dW_gate": dWg, "dW_up": dWu,
                "dW_down": dWd}

    def worst(a, b):
        """Largest error over the outputs, each relative to its tensor's largest magnitude."""
        return max(float(np.max(np.abs(a[n] - b[n])) / max(1.0, np.abs(b[n]).max())) for n in b)

    tol = 1e-6                                            # fp32 accumulation over 16 terms (realised: 5e-8); a bf16 ulp is 4e-3
    dec = oracle_outputs(True)
    full = _layer_with_roundings(x, dY, idx, gate, Wg, Wu, Wd, set(ROUNDING_POINTS))
    for n in dec:
        err = float(np.max(np.abs(full[n] - dec[n])) / max(1.0, np.abs(dec[n]).max()))
        assert err <= tol, f"declared mode, {n}: {err:.3e}"
    none = _layer_with_roundings(x, dY, idx, gate, Wg, Wu, Wd, set())
    assert worst(none, oracle_outputs(False)) <= tol
    # the bf16 tensors of the declared mode are representable in bf16
    for n in ("Y", "G", "U", "H", "Yp", "dX"):
        assert np.array_equal(oracle.bf16_bits_to_f32(synth.bits(torch.from_numpy(dec[n]).to(torch.bfloat16))), dec[n])
    # every single rounding point is visible: without it, some output is off by >= 500 x the tolerance
    for p in ROUNDING_POINTS:
        without = _layer_with_roundings(x, dY, idx, gate, Wg, Wu, Wd, set(ROUNDING_POINTS) - {p})
        assert worst(without, dec) >= 500 * tol, f"removing the rounding of {p} goes unnoticed"
    # and so is a rounding in a place that is not declared: dgate and the weight gradients stay fp32
    for n in ("dgate", "dW_gate", "dW_up", "dW_down"):
        as_bf16 = oracle.bf16_bits_to_f32(synth.bits(torch.from_numpy(dec[n].astype(np.float32)).to(torch.bfloat16)))
        assert np.max(np.abs(as_bf16 - dec[n])) > 500 * tol * max(1.0, np.abs(dec[n]).max()), n


def test_combine_of_the_per_assignment_rows_is_the_layer_output():
    """oracle.combine applied to the per-assignment rows reproduces the whole-layer routines bit for bit, in
    both modes: Y from Yp, and dX of a token from its k one-expert problems (the form the full-size GPU
    tests use, where the experts of the sampled tokens are streamed)."""
    x, dY, idx, gate, Wg, Wu, Wd = _setup_bwd(16, T=7, d=12, E=4, k=3, f=16)
    T, k = idx.shape
    for declared in (False, True):
        Y, _, _, _, Yp = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd, declared=declared, want_parts=True)
        assert np.array_equal(oracle.combine(Yp, declared), Y)
        dX, dgate = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd, declared=declared)
        parts = np.zeros((T, k, x.shape[1]), np.float32)
        for t in range(T):
            for j in range(k):
                e = int(idx[t, j])
                one = (x[t:t + 1], dY[t:t + 1], np.zeros((1, 1), np.int32), gate[t:t + 1, j:j + 1], Wg[e:e + 1],
                       Wu[e:e + 1], Wd[e:e + 1])
                dXp, dg = oracle.ffn_bwd_tokens(*one, declared=declared)
                parts[t, j] = dXp[0]
                assert dg[0, 0] == dgate[t, j]
        assert np.array_equal(oracle.combine(parts, declared), dX)
    # closed form: a plain sum, rounded once
    p3 = np.float32([[[1.0, 2.0 ** -9], [2.0 ** -9, 2.0 ** -9], [0.5, 1.0]]])
    assert np.array_equal(oracle.combine(p3), np.float32([[1.5 + 2.0 ** -9, 1.0 + 2.0 ** -8]]))
    assert np.array_equal(oracle.combine(p3, True), np.float32([[1.5, 1.0]]))      # ties go to the even neighbour


def test_streamed_assembly_of_sampled_tokens_equals_the_whole_layer_oracle():
    """The full-size GPU tests assemble the oracle's Y, dX, dgate of sampled tokens from expert chunks;
    on a small layer that assembly must equal the oracle's whole-layer routines bit for bit."""
    import types

    from test_gpu_fullsize import _experts_by_row_count, _oracle_on_sampled_tokens, _sampled_tokens
    w = synth.small("c3_trillion", T=40, d=16, E=11, k=3, f=24, backward=True, seed=5)
    inp = synth.make_inputs(w, "cpu")
    xb, dYb, Wg, Wu, Wd = (synth.bits(inp[n]) for n in ("x", "dY", "W_gate", "W_up", "W_down"))
    idx, gate = oracle.route(xb, inp["W_r"].numpy(), inp["bias"].numpy(), w.k, w.score_fn, w.bias_mode)
    counts, offsets, perm_row, row_src = oracle.permute(idx, w.E)
    toks = _sampled_tokens(w, offsets, row_src)
    assert np.unique(idx[toks]).size == int((counts > 0).sum())
    buf = types.SimpleNamespace(idx=torch.from_numpy(idx), gate=torch.from_numpy(gate))
    got = _oracle_on_sampled_tokens(w, inp, buf, toks, chunk=4)
    for m, declared in enumerate((False, True)):
        assert np.array_equal(got["Y"][m], oracle.ffn_fwd(xb, idx, gate, Wg, Wu, Wd, declared=declared, toks=toks))
        dX, dg = oracle.ffn_bwd_tokens(xb, dYb, idx, gate, Wg, Wu, Wd, declared=declared, toks=toks)
        assert np.array_equal(got["dX"][m], dX) and np.array_equal(got["dgate"][m], dg)
    picked = _experts_by_row_count(counts)
    assert len(set(picked)) == len(picked) and all(counts[e] > 0 for e in picked)
    assert counts[picked[0]] == counts[counts > 0].min() and counts[picked[1]] == counts.max()


# ------------------------------------------------------------------------------ router backward
@pytest.mark.parametrize("score_fn,bias_mode", [(0, 0), (0, 2), (1, 0), (1, 1), (1, 2)])
def test_router_backward_matches_automatic_differentiation_of_the_long_form(score_fn, bias_mode):
    """The oracle uses the closed form on the selected logits; autodiff differentiates the long
    form (scores over ALL experts, then renormalisation over the selected ones)."""
    rng = np.random.default_rng(20 + score_fn * 3 + bias_mode)
    T, d, E, k = 9, 12, 7, 3
    x = _rand_bits(rng, (T, d))
    Wr = (rng.standard_normal((d, E)) * 0.4).astype(np.float32)
    b = (rng.standard_normal(E) * 0.1).astype(np.float32) if bias_mode else None
    idx, gate = oracle.route(x, Wr, b, k, score_fn, bias_mode)
    dgate = rng.standard_normal((T, k))
    dz, dWr, dX, db = oracle.route_bwd(x, Wr, b, k, score_fn, bias_mode, idx, dgate)

    tx = torch.tensor(oracle.bf16_bits_to_f64(x), requires_grad=True)
    tW = torch.tensor(Wr.astype(np.float64), requires_grad=True)
    tb = torch.tensor(b.astype(np.float64), requires_grad=True) if bias_mode else None
    z = tx @ tW
    if bias_mode == 2:
        z = z + tb
    s = torch.softmax(z, 1) if score_fn == 0 else torch.sigmoid(z)
    sel = torch.gather(s, 1, torch.from_numpy(idx.astype(np.int64)))
    g = sel / sel.sum(1, keepdim=True)
    assert np.max(np.abs(g.detach().numpy() - gate)) < 1e-6          # same forward as the router
    (g * torch.from_numpy(dgate)).sum().backward()
    assert np.max(np.abs(dWr - tW.grad.numpy())) < 1e-12
    assert np.max(np.abs(dX - tx.grad.numpy())) < 1e-12
    if bias_mode == 2:
        assert np.max(np.abs(db - tb.grad.numpy())) < 1e-12
    else:
        assert np.all(db == 0)
        if bias_mode == 1:
            assert tb.grad is None                                       # selection only: no gradient
    # dz is supported on the selected experts and sums to zero per token for softmax
    mask = np.zeros((T, E), bool)
    np.put_along_axis(mask, idx.astype(np.int64), True, 1)
    assert np.all(dz[~mask] == 0)
    if score_fn == 0:
        assert np.max(np.abs(dz.sum(1))) < 1e-12


def test_router_backward_central_differences():
    rng = np.random.default_rng(31)
    T, d, E, k = 5, 8, 6, 2
    x = _rand_bits(rng, (T, d))
    Wr = (rng.standard_normal((d, E)) * 0.4).astype(np.float32)
    idx, _ = oracle.route(x, Wr, None, k, 1, 0)
    dgate = rng.standard_normal((T, k))
    _, dWr, _, _ = oracle.route_bwd(x, Wr, None, k, 1, 0, idx, dgate)
    xf = oracle.bf16_bits_to_f64(x)

    def loss(W):
        z = np.take_along_axis(xf @ W, idx.astype(np.int64), 1)
        s = 1 / (1 + np.exp(-z))
        return float(((s / s.sum(1, keepdims=True)) * dgate).sum())

    W0 = Wr.astype(np.float64)
    for _ in range(10):
        i, e = rng.integers(0, d), rng.integers(0, E)
        Wp, Wm = W0.copy(), W0.copy()
        Wp[i, e] += 1e-6
        Wm[i, e] -= 1e-6
        fd = (loss(Wp) - loss(Wm)) / 2e-6
        assert abs(fd - dWr[i, e]) <= 1e-6 * max(1.0, abs(dWr[i, e]))


# ------------------------------------------------------------------------------ vocabulary projection
def test_vocab_loss_matches_library_cross_entropy_and_closed_forms():
    rng = np.random.default_rng(40)
    N, H, V = 13, 24, 301
    x = _rand_bits(rng, (N, H))
    W = _rand_bits(rng, (H, V), 0.3)
    t = rng.integers(0, V, N)
    loss, lse = oracle.vocab_loss(x, W, t)
    Y = torch.tensor(oracle.bf16_bits_to_f64(x) @ oracle.bf16_bits_to_f64(W))
    ce = torch.nn.functional.cross_entropy(Y, torch.from_numpy(t), reduction="none").numpy()
    assert np.max(np.abs(loss + ce)) < 1e-12                      # the log-likelihood is minus the cross entropy
    assert np.max(np.abs(lse - torch.logsumexp(Y, 1).numpy())) < 1e-12
    # all-zero weights: every token has log-likelihood -log V
    l0, lse0 = oracle.vocab_loss(x, np.zeros_like(W), t)
    assert np.allclose(l0, -np.log(V)) and np.allclose(lse0, np.log(V))
    # a shift of all logits of a token leaves the loss unchanged and moves lse by the shift
    assert np.all(loss <= 0)
    # large logits do not overflow
    big = synth.bits((torch.from_numpy(oracle.bf16_bits_to_f32(W)) * 64).to(torch.bfloat16))
    lb, _ = oracle.vocab_loss(x, big, t)
    assert np.all(np.isfinite(lb))


def test_vocab_loss_backward_matches_autodiff_finite_differences_and_closed_forms():
    rng = np.random.default_rng(41)
    N, H, V = 11, 16, 203
    x = _rand_bits(rng, (N, H))
    W = _rand_bits(rng, (H, V), 0.3)
    t = rng.integers(0, V, N)
    g = rng.standard_normal(N)
    dX, dW = oracle.vocab_loss_bwd(x, W, t, g)
    # (1) library autodiff of the library's own cross entropy (the loss is minus the cross entropy)
    Xt = torch.tensor(oracle.bf16_bits_to_f64(x), requires_grad=True)
    Wt = torch.tensor(oracle.bf16_bits_to_f64(W), requires_grad=True)
    ce = torch.nn.functional.cross_entropy(Xt @ Wt, torch.from_numpy(t), reduction="none")
    (-(ce * torch.from_numpy(g)).sum()).backward()
    assert np.max(np.abs(dX - Xt.grad.numpy())) < 1e-11
    assert np.max(np.abs(dW - Wt.grad.numpy())) < 1e-11
    # (2) central finite differences of the forward oracle's definition written out here
    Xf, Wf = oracle.bf16_bits_to_f64(x), oracle.bf16_bits_to_f64(W)

    def total(Xa, Wa):
        Y = Xa @ Wa
        m = Y.max(1)
        lse = m + np.log(np.exp(Y - m[:, None]).sum(1))
        return float(((Y[np.arange(N), t] - lse) * g).sum())

    eps = 1e-6
    for (n, h) in ((0, 0), (3, 7), (10, 15)):
        E = np.zeros_like(Xf); E[n, h] = eps
        assert abs((total(Xf + E, Wf) - total(Xf - E, Wf)) / (2 * eps) - dX[n, h]) < 1e-6
    for (h, v) in ((0, int(t[0])), (5, 100), (15, 202)):
        E = np.zeros_like(Wf); E[h, v] = eps
        assert abs((total(Xf, Wf + E) - total(Xf, Wf - E)) / (2 * eps) - dW[h, v]) < 1e-6
    # (3) closed form at W = 0: p is uniform, dY = g ([v == t] - 1/V), so dX = 0 and
    #     dW[:, v] = sum_n x[n] g[n] ([v == t_n] - 1/V)
    dX0, dW0 = oracle.vocab_loss_bwd(x, np.zeros_like(W), t, g)
    assert np.max(np.abs(dX0)) == 0.0
    onehot = np.zeros((N, V)); onehot[np.arange(N), t] = 1.0
    assert np.max(np.abs(dW0 - Xf.T @ ((onehot - 1.0 / V) * g[:, None]))) < 1e-12
    # (4) every row of dY sums to zero: the gradient is orthogonal to a constant shift of a token's logits,
    #     i.e. dW summed over the vocabulary vanishes
    assert np.max(np.abs(dW.sum(1))) < 1e-10
    # (5) the declared-rounding mode differs from the exact one only by the bf16 rounding of dY
    dXd, dWd = oracle.vocab_loss_bwd(x, W, t, g, declared=True)
    assert 0 < np.max(np.abs(dXd - dX)) < 2e-2 * max(1.0, np.abs(dX).max())
    assert np.linalg.norm(dWd - dW) / np.linalg.norm(dW) < 1e-2
