"""ctypes front end of the CPU oracle (``mop_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg of
the benchmark may import this package; the CUDA product path never does, and this
package never imports the CUDA package.  Arrays are numpy; bf16 tensors travel as
``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "mop_oracle.cpp"
_LIB = _HERE / "libmop_oracle.so"

SCORE_SOFTMAX, SCORE_SIGMOID = 0, 1
BIAS_NONE, BIAS_POST_SCORE, BIAS_PRE_LOGIT = 0, 1, 2

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (contraction off, so every rounding is the written one)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-mavx2", "-mfma", "-fopenmp", "-fPIC", "-shared",
               "-o", str(_LIB), str(_SRC)]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.mop_oracle_bf16_to_f32.restype = ctypes.c_float
        _lib.mop_oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.mop_oracle_f32_to_bf16.restype = ctypes.c_uint16
        _lib.mop_oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.mop_oracle_sigmoid_contract.restype = ctypes.c_float
        _lib.mop_oracle_sigmoid_contract.argtypes = [ctypes.c_float]
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle's loops will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _check(rc, name):
    if rc != 0:
        raise ValueError(f"{name}: invalid arguments (rc={rc})")


# ----------------------------------------------------------------------------- helpers
def f32_to_bf16_bits(a) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns, through the oracle's own routine."""
    a = _c(a, np.float32)
    out = np.empty(a.shape, np.uint16)
    fn = lib().mop_oracle_f32_to_bf16_array
    fn.restype = None
    fn(ctypes.c_size_t(a.size), _p(a), _p(out))
    return out


def bf16_bits_to_f32(bits) -> np.ndarray:
    """Exact widening (vectorised: a bf16 is the upper half of an fp32)."""
    b = _c(bits, np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(bits) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def sigmoid_contract(z) -> np.ndarray:
    z = _c(z, np.float32)
    L = lib()
    out = np.empty(z.shape, np.float32)
    flat, o = z.reshape(-1), out.reshape(-1)
    for i in range(flat.size):
        o[i] = L.mop_oracle_sigmoid_contract(float(flat[i]))
    return out


# ----------------------------------------------------------------------------- router
def route(x_bits, W_r, bias, k, score_fn, bias_mode, want_logits=False):
    """x_bits [T,d] uint16, W_r [d,E] f32, bias [E] f32 or None.

    Returns (idx [T,k] i32, gate [T,k] f32) and, if want_logits, also (z, key) [T,E] f32.
    """
    x_bits = _c(x_bits, np.uint16)
    W_r = _c(W_r, np.float32)
    T, d = x_bits.shape
    E = W_r.shape[1]
    assert W_r.shape[0] == d
    b = None if bias is None else _c(bias, np.float32)
    idx = np.empty((T, k), np.int32)
    gate = np.empty((T, k), np.float32)
    z = np.empty((T, E), np.float32) if want_logits else None
    key = np.empty((T, E), np.float32) if want_logits else None
    rc = lib().mop_oracle_route(T, d, E, k, score_fn, bias_mode, _p(x_bits), _p(W_r), _p(b), _p(idx), _p(gate), _p(z),
                                _p(key))
    _check(rc, "route")
    return (idx, gate, z, key) if want_logits else (idx, gate)


def select(key, zg, k, score_fn):
    """Top-k and gates from given keys [T,E] and gate logits [T,E]."""
    key = _c(key, np.float32)
    zg = _c(zg, np.float32)
    T, E = key.shape
    idx = np.empty((T, k), np.int32)
    gate = np.empty((T, k), np.float32)
    _check(lib().mop_oracle_select(T, E, k, score_fn, _p(key), _p(zg), _p(idx), _p(gate)), "select")
    return idx, gate


def permute(idx, E):
    """idx [T,k] i32 -> counts [E], offsets [E+1], perm_row [T*k], row_src [T*k] (all i32)."""
    idx = _c(idx, np.int32)
    T, k = idx.shape
    counts = np.empty(E, np.int32)
    offsets = np.empty(E + 1, np.int32)
    perm_row = np.empty(T * k, np.int32)
    row_src = np.empty(T * k, np.int32)
    _check(lib().mop_oracle_permute(T, k, E, _p(idx), _p(counts), _p(offsets), _p(perm_row), _p(row_src)), "permute")
    return counts, offsets, perm_row, row_src


# ----------------------------------------------------------------------------- expert FFN
def _dims(x, Wg, idx):
    T, d = x.shape
    E, d2, f = Wg.shape
    assert d2 == d
    k = idx.shape[1]
    return T, d, E, k, f


def ffn_fwd(x, idx, gate, Wg, Wu, Wd, *, fp64=False, declared=False, toks=None, want_parts=False):
    """Forward of the routed layer on the listed tokens (all if toks is None).

    fp32 path: x, W* are uint16 bf16 bits, gate f32.  fp64 path: everything float64.
    Returns Y [n,d]; with want_parts also (G, U, H [n,k,f], Yp [n,k,d]) per assignment.
    """
    idx = _c(idx, np.int32)
    if fp64:
        dt, name = np.float64, "mop_oracle_ffn_fwd_f64"
        x, Wg, Wu, Wd = (_c(a, np.float64) for a in (x, Wg, Wu, Wd))
        gate = _c(gate, np.float64)
    else:
        dt, name = np.float32, "mop_oracle_ffn_fwd_f32"
        x, Wg, Wu, Wd = (_c(a, np.uint16) for a in (x, Wg, Wu, Wd))
        gate = _c(gate, np.float32)
    T, d, E, k, f = _dims(x, Wg, idx)
    assert Wu.shape == (E, d, f) and Wd.shape == (E, f, d) and gate.shape == (T, k)
    tk = None if toks is None else _c(toks, np.int32)
    n = T if tk is None else tk.size
    Y = np.empty((n, d), dt)
    parts = [np.empty((n, k, f), dt) for _ in range(3)] + [np.empty((n, k, d), dt)] if want_parts else [None] * 4
    fn = getattr(lib(), name)
    if fp64:
        rc = fn(T, d, E, k, f, _p(x), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(tk), _p(Y), *map(_p, parts))
    else:
        rc = fn(T, d, E, k, f, int(declared), _p(x), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(tk), _p(Y),
                *map(_p, parts))
    _check(rc, name)
    return (Y, *parts) if want_parts else Y


def ffn_bwd_tokens(x, dY, idx, gate, Wg, Wu, Wd, *, fp64=False, declared=False, toks=None):
    """dX [n,d] and dgate [n,k] for the listed tokens (all if toks is None)."""
    idx = _c(idx, np.int32)
    if fp64:
        dt, name = np.float64, "mop_oracle_ffn_bwd_tokens_f64"
        x, dY, Wg, Wu, Wd = (_c(a, np.float64) for a in (x, dY, Wg, Wu, Wd))
        gate = _c(gate, np.float64)
    else:
        dt, name = np.float32, "mop_oracle_ffn_bwd_tokens_f32"
        x, dY, Wg, Wu, Wd = (_c(a, np.uint16) for a in (x, dY, Wg, Wu, Wd))
        gate = _c(gate, np.float32)
    T, d, E, k, f = _dims(x, Wg, idx)
    tk = None if toks is None else _c(toks, np.int32)
    n = T if tk is None else tk.size
    dX = np.empty((n, d), dt)
    dgate = np.empty((n, k), dt)
    fn = getattr(lib(), name)
    if fp64:
        rc = fn(T, d, E, k, f, _p(x), _p(dY), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(tk), _p(dX), _p(dgate))
    else:
        rc = fn(T, d, E, k, f, int(declared), _p(x), _p(dY), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(tk),
                _p(dX), _p(dgate))
    _check(rc, name)
    return dX, dgate


def ffn_bwd_experts(x, dY, idx, gate, Wg, Wu, Wd, experts, *, fp64=False, declared=False):
    """dW_gate, dW_up [n,d,f] and dW_down [n,f,d] for the listed experts."""
    idx = _c(idx, np.int32)
    if fp64:
        dt, name = np.float64, "mop_oracle_ffn_bwd_experts_f64"
        x, dY, Wg, Wu, Wd = (_c(a, np.float64) for a in (x, dY, Wg, Wu, Wd))
        gate = _c(gate, np.float64)
    else:
        dt, name = np.float32, "mop_oracle_ffn_bwd_experts_f32"
        x, dY, Wg, Wu, Wd = (_c(a, np.uint16) for a in (x, dY, Wg, Wu, Wd))
        gate = _c(gate, np.float32)
    T, d, E, k, f = _dims(x, Wg, idx)
    ex = _c(experts, np.int32)
    n = ex.size
    dWg = np.empty((n, d, f), dt)
    dWu = np.empty((n, d, f), dt)
    dWd = np.empty((n, f, d), dt)
    fn = getattr(lib(), name)
    if fp64:
        rc = fn(T, d, E, k, f, _p(x), _p(dY), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(ex), _p(dWg), _p(dWu),
                _p(dWd))
    else:
        rc = fn(T, d, E, k, f, int(declared), _p(x), _p(dY), _p(idx), _p(gate), _p(Wg), _p(Wu), _p(Wd), n, _p(ex),
                _p(dWg), _p(dWu), _p(dWd))
    _check(rc, name)
    return dWg, dWu, dWd


def combine(parts, declared=False):
    """out[n] = sum_j parts[n, j] (fp32, j ascending); declared rounds the sum once to bf16.
    parts [n,k,d] f32: per-assignment rows, e.g. the Yp of ffn_fwd(want_parts=True)."""
    parts = _c(parts, np.float32)
    n, k, d = parts.shape
    out = np.empty((n, d), np.float32)
    _check(lib().mop_oracle_combine_f32(n, k, d, int(declared), _p(parts), _p(out)), "combine")
    return out


# ----------------------------------------------------------------------------- router backward
def route_bwd(x_bits, W_r, bias, k, score_fn, bias_mode, idx, dgate):
    """Backward of the router's gate computation with the selection held fixed (plain numpy, fp64).

    The gates of a token are g_j = s_j / sum_l s_l over its k selected experts, with s = softmax
    over all E of the logits (softmax router; the common denominator cancels, so g is a softmax
    over the selected logits) or s = sigmoid(logit) (sigmoid router); logit = z (+ bias when the
    bias enters before the score), z = x W_r.  Given dL/dgate this returns
        dz     [T,E]  (non-zero only at the selected experts),
        dW_r   [d,E] = x^T dz,   dX [T,d] = dz W_r^T,   dbias [E] (zero unless the bias is pre-logit).
    A bias added after the score only steers the selection and receives no gradient.
    """
    x = bf16_bits_to_f64(x_bits)
    W = np.asarray(W_r, np.float64)
    T, d = x.shape
    E = W.shape[1]
    idx = np.asarray(idx, np.int64)
    dg = np.asarray(dgate, np.float64)
    zz = x @ W
    if bias_mode == BIAS_PRE_LOGIT:
        zz = zz + np.asarray(bias, np.float64)[None, :]
    zs = np.take_along_axis(zz, idx, 1)                     # logits of the selected experts [T,k]
    if score_fn == SCORE_SOFTMAX:
        p = np.exp(zs - zs.max(1, keepdims=True))
        g = p / p.sum(1, keepdims=True)
        dzs = g * (dg - (g * dg).sum(1, keepdims=True))
    else:
        s = 1.0 / (1.0 + np.exp(-zs))
        S = s.sum(1, keepdims=True)
        g = s / S
        ds = (dg - (g * dg).sum(1, keepdims=True)) / S
        dzs = ds * s * (1.0 - s)
    dz = np.zeros((T, E))
    np.put_along_axis(dz, idx, dzs, 1)
    dbias = dz.sum(0) if bias_mode == BIAS_PRE_LOGIT else np.zeros(E)
    return dz, x.T @ dz, dz @ W.T, dbias


# ----------------------------------------------------------------------------- vocabulary projection
def vocab_loss(x_bits, W_bits, targets):
    """Per-token log-likelihood of the vocabulary projection (plain numpy, fp64):
        Y = X W_voc  [N,V],   loss[n] = Y[n, t_n] - log sum_v exp(Y[n, v]).
    x_bits [N,H], W_bits [H,V] bf16 bit patterns, targets [N] int.  Returns (loss [N], lse [N])."""
    X = bf16_bits_to_f64(x_bits)
    W = bf16_bits_to_f64(W_bits)
    t = np.asarray(targets, np.int64)
    Y = X @ W
    m = Y.max(1)
    lse = m + np.log(np.exp(Y - m[:, None]).sum(1))
    return Y[np.arange(Y.shape[0]), t] - lse, lse


def vocab_loss_bwd(x_bits, W_bits, targets, dloss, declared=False):
    """Gradients of the per-token log-likelihoods of vocab_loss (plain numpy, fp64), written out from
    Eq. 5: with p[n, v] = exp(Y[n, v] - lse[n]) and an upstream weight dloss[n] per token,
        dY[n, v] = dloss[n] * ([v == t_n] - p[n, v]),   dX = dY W_voc^T,   dW_voc = X^T dY.
    declared=True rounds dY to bf16 before the two products (the tensor the CUDA path hands to its
    tensor-core products in bf16).  Returns (dX [N,H], dW [H,V])."""
    X = bf16_bits_to_f64(x_bits)
    W = bf16_bits_to_f64(W_bits)
    t = np.asarray(targets, np.int64)
    g = np.asarray(dloss, np.float64)
    Y = X @ W
    m = Y.max(1)
    lse = m + np.log(np.exp(Y - m[:, None]).sum(1))
    dY = -np.exp(Y - lse[:, None])
    dY[np.arange(Y.shape[0]), t] += 1.0
    dY *= g[:, None]
    if declared:
        dY = bf16_bits_to_f64(f32_to_bf16_bits(dY.astype(np.float32)))
    return dY @ W.T, X.T @ dY

