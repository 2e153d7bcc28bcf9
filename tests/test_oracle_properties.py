"""Property tests of the oracle over random small shapes (hypothesis): the invariants that hold for
every routing and every shape, on top of the fixed cases of test_oracle_pins.py."""
import numpy as np
import torch
from hypothesis import given, settings, strategies as st

import oracle
from paper_2607_01844_b200 import synth


def _bits(rng, shape, std=1.0):
    return synth.bits(torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * std).to(torch.bfloat16))


shapes = st.tuples(st.integers(1, 40), st.sampled_from([8, 16, 24]), st.integers(1, 37), st.integers(1, 6),
                   st.sampled_from([8, 16]), st.integers(0, 2 ** 31 - 1))


@settings(max_examples=30, deadline=None)
@given(shapes, st.sampled_from([(0, 0), (0, 2), (1, 0), (1, 1), (1, 2)]))
def test_routing_and_permutation_invariants(shape, mode):
    T, d, E, k, f, seed = shape
    k = min(k, E)
    score_fn, bias_mode = mode
    rng = np.random.default_rng(seed)
    x = _bits(rng, (T, d))
    Wr = (rng.standard_normal((d, E)) * 0.5).astype(np.float32)
    b = (rng.standard_normal(E) * 0.05).astype(np.float32) if bias_mode else None
    idx, gate, z, key = oracle.route(x, Wr, b, k, score_fn, bias_mode, want_logits=True)
    assert idx.min() >= 0 and idx.max() < E
    for t in range(T):
        assert len(set(idx[t])) == k                                   # distinct experts
        ks = key[t, idx[t]]
        assert np.all(np.diff(ks) <= 0)                                # descending keys
        rest = np.delete(key[t], idx[t])
        assert rest.size == 0 or rest.max() <= ks[-1]                  # nothing better was left out
    assert np.all(gate > 0) and np.allclose(gate.sum(1), 1.0, atol=1e-6)
    counts, offsets, perm_row, row_src = oracle.permute(idx, E)
    assert counts.sum() == T * k and offsets[-1] == T * k and np.all(np.diff(offsets) == counts)
    assert np.array_equal(np.sort(perm_row), np.arange(T * k))
    assert np.array_equal(row_src[perm_row], np.arange(T * k))
    assert np.all(counts <= T)                                         # an expert gets each token at most once


@settings(max_examples=15, deadline=None)
@given(shapes)
def test_forward_backward_invariants(shape):
    T, d, E, k, f, seed = shape
    k = min(k, E)
    rng = np.random.default_rng(seed)
    x, dY = _bits(rng, (T, d)), _bits(rng, (T, d))
    Wg, Wu, Wd = _bits(rng, (E, d, f), 0.3), _bits(rng, (E, d, f), 0.3), _bits(rng, (E, f, d), 0.3)
    Wr = (rng.standard_normal((d, E)) * 0.5).astype(np.float32)
    idx, gate = oracle.route(x, Wr, None, k, 0, 0)
    Y = oracle.ffn_fwd(x, idx, gate, Wg, Wu, Wd)
    # the order of a token's (expert, gate) slots does not matter beyond fp32 summation order
    perm = rng.permutation(k)
    Y2 = oracle.ffn_fwd(x, idx[:, perm], gate[:, perm], Wg, Wu, Wd)
    assert np.max(np.abs(Y - Y2)) <= 1e-5 * max(1.0, np.abs(Y).max())
    # Y is linear in the gates
    assert np.allclose(oracle.ffn_fwd(x, idx, 2 * gate, Wg, Wu, Wd), 2 * Y, rtol=0, atol=0)
    dX, dgate = oracle.ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd)
    lhs = (gate * dgate).sum(1)
    rhs = (oracle.bf16_bits_to_f32(dY) * Y).sum(1)
    assert np.max(np.abs(lhs - rhs)) <= 2e-4 * max(1.0, np.abs(rhs).max())
    # the weight gradient of an expert that received no token is zero
    unused = [e for e in range(E) if not np.any(idx == e)]
    if unused:
        dWg, dWu, dWd = oracle.ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, np.array(unused[:2], np.int32))
        assert not dWg.any() and not dWu.any() and not dWd.any()
