"""Thin ctypes binding of the C ABI in ``include/mop_moe.h``: argument marshalling only.

Every function has the name of the C entry point it calls and takes torch tensors that already
live on the device (torch is used for memory and streams, nothing else).  There is no fallback:
if the shared library is missing, importing this module's `lib()` raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libmop_moe.so"

MOP_OK = 0
STATUS_NAMES = {0: "MOP_OK", 1: "MOP_ERR_INVALID_ARG", 2: "MOP_ERR_SHAPE", 3: "MOP_ERR_ALIGN", 4: "MOP_ERR_WORKSPACE",
                5: "MOP_ERR_CUDA", 6: "MOP_ERR_UNSUPPORTED", 7: "MOP_ERR_TIMEOUT"}
ROUTE_AUTO, ROUTE_EXACT, ROUTE_TENSOR = 0, 1, 2
GEMM_AUTO, GEMM_TENSOR, GEMM_SCALAR, GEMM_TENSOR_1CTA, GEMM_TENSOR_2CTA, GEMM_TENSOR_MIXED, GEMM_TENSOR_TN = 0, 1, 2, 3, 4, 5, 6


class MopShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("T", "d", "E", "k", "f", "score_fn", "bias_mode", "with_backward",
                                              "dw_accumulate", "gemm_path", "host_io", "route_path")]


class MopError(RuntimeError):
    def __init__(self, call, code):
        super().__init__(f"{call} failed: {STATUS_NAMES.get(code, code)} ({lib().mop_status_string(code).decode()})")
        self.code = code


_lib = None
_P = ctypes.c_void_p


def lib() -> ctypes.CDLL:
    """The CUDA library.  It must have been built (``python -m paper_2607_01844_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA extension first (no CPU fallback exists)")
        L = ctypes.CDLL(str(LIB_PATH))
        L.mop_status_string.restype = ctypes.c_char_p
        L.mop_status_string.argtypes = [ctypes.c_int]
        L.mop_workspace_bytes.restype = ctypes.c_size_t
        L.mop_workspace_bytes.argtypes = [ctypes.POINTER(MopShape)]
        L.mop_create.argtypes = [ctypes.POINTER(_P), ctypes.POINTER(MopShape), ctypes.c_int]
        L.mop_destroy.argtypes = [_P]
        L.mop_destroy.restype = None
        L.mop_poll.argtypes = [_P, _P]
        L.mop_launch_count.argtypes = [_P]
        L.mop_selftest_wait_timeout.argtypes = [_P, ctypes.c_int64, _P]
        L.mop_debug_guard_arm.argtypes = [_P, _P]
        L.mop_debug_guard_check.argtypes = [_P, ctypes.POINTER(ctypes.c_int64), _P]
        L.mop_debug_guard_poke.argtypes = [_P, ctypes.c_int32, ctypes.c_int32, _P]
        L.mop_launch_count.restype = ctypes.c_int64
        L.mop_moe_route.argtypes = [_P] * 8
        L.mop_route_stats.argtypes = [_P] + [ctypes.POINTER(ctypes.c_int64)] * 3 + [_P]
        L.mop_moe_permute.argtypes = [_P] * 9
        L.mop_moe_expert_ffn_fwd.argtypes = [_P] * 13
        L.mop_moe_expert_ffn_fwd_gather.argtypes = [_P] * 11
        L.mop_moe_combine.argtypes = [_P] * 5
        L.mop_moe_expert_ffn_bwd.argtypes = [_P] * 19
        L.mop_moe_forward_host.argtypes = [_P] * 11
        L.mop_moe_forward_host_async.argtypes = [_P] * 11
        L.mop_moe_train_step_host_async.argtypes = [_P] * 15
        L.mop_host_drain.argtypes = [_P] * 2
        L.mop_moe_route_bwd.argtypes = [_P] * 14
        L.mop_moe_chunked_workspace_bytes.argtypes = [ctypes.POINTER(MopShape), ctypes.c_int32, ctypes.c_int32]
        L.mop_moe_chunked_workspace_bytes.restype = ctypes.c_size_t
        L.mop_moe_layer_fwd_chunked.argtypes = [_P, ctypes.c_int32] + [_P] * 15
        L.mop_moe_layer_bwd_chunked.argtypes = [_P, ctypes.c_int32] + [_P] * 16
        L.mop_moe_train_step_host.argtypes = [_P] * 15
        L.mop_moe_permute_static.argtypes = [ctypes.c_int] + [ctypes.c_int32] * 4 + [_P] * 8
        L.mop_vocab_workspace_bytes.argtypes = [ctypes.c_int32] * 3
        L.mop_vocab_workspace_bytes.restype = ctypes.c_size_t
        L.mop_vocab_loss_fwd.argtypes = [ctypes.c_int] + [ctypes.c_int32] * 3 + [_P] * 7
        L.mop_vocab_poll.argtypes = [ctypes.c_int, _P, _P]
        L.mop_vocab_selftest_wait_timeout.argtypes = [ctypes.c_int, _P, ctypes.c_int64, _P]
        L.mop_vocab_bwd_workspace_bytes.argtypes = [ctypes.c_int32] * 3
        L.mop_vocab_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.mop_vocab_loss_bwd.argtypes = [ctypes.c_int] + [ctypes.c_int32] * 3 + [_P] * 9
        L.mop_profile_enable.argtypes = [_P, ctypes.c_int]
        L.mop_profile_read.argtypes = [_P, _P, ctypes.c_int32, ctypes.POINTER(ctypes.c_char_p),
                                       ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
        L.mop_profile_read.restype = ctypes.c_int32
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors cross the C ABI dense and row-major"
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(call, rc):
    if rc != MOP_OK:
        raise MopError(call, rc)


class Context:
    """Owns one mop_ctx (shape + workspace on one device)."""

    def __init__(self, T, d, E, k, f, score_fn=0, bias_mode=0, with_backward=False, dw_accumulate=False,
                 gemm_path=GEMM_AUTO, host_io=False, device=0, route_path=ROUTE_AUTO):
        self.shape = MopShape(T, d, E, k, f, score_fn, bias_mode, int(with_backward), int(dw_accumulate), gemm_path,
                              int(host_io), route_path)
        self.handle = _P()
        _check("mop_create", lib().mop_create(ctypes.byref(self.handle), ctypes.byref(self.shape), device))

    def close(self):
        if self.handle:
            lib().mop_destroy(self.handle)
            self.handle = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self):
        return lib().mop_workspace_bytes(ctypes.byref(self.shape))

    @property
    def launch_count(self):
        return lib().mop_launch_count(self.handle)


def mop_poll(ctx, stream=None):
    _check("mop_poll", lib().mop_poll(ctx.handle, _stream(stream)))


def mop_selftest_wait_timeout(ctx, limit_cycles=20_000_000, stream=None):
    _check("mop_selftest_wait_timeout", lib().mop_selftest_wait_timeout(ctx.handle, limit_cycles, _stream(stream)))


def mop_debug_guard_arm(ctx, stream=None):
    _check("mop_debug_guard_arm", lib().mop_debug_guard_arm(ctx.handle, _stream(stream)))


def mop_debug_guard_poke(ctx, band, byte, stream=None):
    _check("mop_debug_guard_poke", lib().mop_debug_guard_poke(ctx.handle, band, byte, _stream(stream)))


def mop_debug_guard_check(ctx, stream=None):
    """Bytes of the workspace's guard bands that were overwritten since they were armed."""
    bad = ctypes.c_int64(-1)
    _check("mop_debug_guard_check", lib().mop_debug_guard_check(ctx.handle, ctypes.byref(bad), _stream(stream)))
    return bad.value


def mop_moe_route(ctx, x, W_r, bias, topk_idx, topk_gate, logits=None, stream=None):
    _check("mop_moe_route", lib().mop_moe_route(ctx.handle, _ptr(x), _ptr(W_r), _ptr(bias), _ptr(topk_idx),
                                                _ptr(topk_gate), _ptr(logits), _stream(stream)))


def mop_route_stats(ctx, stream=None):
    """(tokens re-evaluated, chains evaluated, exact logits beyond half the assumed error bound) of the
    tensor-core scoring path since the last call."""
    a, b, c = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    _check("mop_route_stats", lib().mop_route_stats(ctx.handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                                    _stream(stream)))
    return a.value, b.value, c.value


def mop_moe_permute(ctx, x, topk_idx, counts, offsets, perm_row, row_src, Xp, stream=None):
    _check("mop_moe_permute", lib().mop_moe_permute(ctx.handle, _ptr(x), _ptr(topk_idx), _ptr(counts), _ptr(offsets),
                                                    _ptr(perm_row), _ptr(row_src), _ptr(Xp), _stream(stream)))


def mop_moe_expert_ffn_fwd(ctx, Xp, offsets, row_src, topk_gate, W_gate, W_up, W_down, G_save, U_save, H, Yp,
                           stream=None):
    _check("mop_moe_expert_ffn_fwd",
           lib().mop_moe_expert_ffn_fwd(ctx.handle, _ptr(Xp), _ptr(offsets), _ptr(row_src), _ptr(topk_gate),
                                        _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(G_save), _ptr(U_save), _ptr(H),
                                        _ptr(Yp), _stream(stream)))


def mop_moe_expert_ffn_fwd_gather(ctx, x, offsets, row_src, topk_gate, W_gate, W_up, W_down, H, Yp, stream=None):
    _check("mop_moe_expert_ffn_fwd_gather",
           lib().mop_moe_expert_ffn_fwd_gather(ctx.handle, _ptr(x), _ptr(offsets), _ptr(row_src), _ptr(topk_gate),
                                               _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(H), _ptr(Yp),
                                               _stream(stream)))


def mop_moe_combine(ctx, Yp, perm_row, Y, stream=None):
    _check("mop_moe_combine", lib().mop_moe_combine(ctx.handle, _ptr(Yp), _ptr(perm_row), _ptr(Y), _stream(stream)))


def mop_moe_expert_ffn_bwd(ctx, dY, Xp, G_save, U_save, H, offsets, perm_row, row_src, topk_gate, W_gate, W_up,
                           W_down, dX, dW_gate, dW_up, dW_down, dgate, stream=None):
    _check("mop_moe_expert_ffn_bwd",
           lib().mop_moe_expert_ffn_bwd(ctx.handle, _ptr(dY), _ptr(Xp), _ptr(G_save), _ptr(U_save), _ptr(H),
                                        _ptr(offsets), _ptr(perm_row), _ptr(row_src), _ptr(topk_gate), _ptr(W_gate),
                                        _ptr(W_up), _ptr(W_down), _ptr(dX), _ptr(dW_gate), _ptr(dW_up), _ptr(dW_down),
                                        _ptr(dgate), _stream(stream)))


def mop_moe_route_bwd(ctx, logits, bias, topk_idx, topk_gate, dgate, Xp, offsets, perm_row, W_r, dW_r, dbias, dX,
                      stream=None):
    _check("mop_moe_route_bwd",
           lib().mop_moe_route_bwd(ctx.handle, _ptr(logits), _ptr(bias), _ptr(topk_idx), _ptr(topk_gate), _ptr(dgate),
                                   _ptr(Xp), _ptr(offsets), _ptr(perm_row), _ptr(W_r), _ptr(dW_r), _ptr(dbias),
                                   _ptr(dX), _stream(stream)))


def mop_moe_chunked_workspace_bytes(ctx, n_chunks, with_backward=False):
    return lib().mop_moe_chunked_workspace_bytes(ctypes.byref(ctx.shape), n_chunks, int(with_backward))


def mop_moe_layer_fwd_chunked(ctx, n_chunks, x, W_r, bias, W_gate, W_up, W_down, topk_idx, topk_gate, counts, offsets,
                              perm_row, row_src, Y, workspace, stream=None):
    """Whole forward with the expert-contiguous buffers live for one group of experts at a time."""
    _check("mop_moe_layer_fwd_chunked",
           lib().mop_moe_layer_fwd_chunked(ctx.handle, n_chunks, _ptr(x), _ptr(W_r), _ptr(bias), _ptr(W_gate), _ptr(W_up),
                                           _ptr(W_down), _ptr(topk_idx), _ptr(topk_gate), _ptr(counts), _ptr(offsets),
                                           _ptr(perm_row), _ptr(row_src), _ptr(Y), _ptr(workspace), _stream(stream)))


def mop_moe_layer_bwd_chunked(ctx, n_chunks, x, dY, topk_gate, offsets, perm_row, row_src, W_gate, W_up, W_down, dX,
                              dW_gate, dW_up, dW_down, dgate, workspace, stream=None):
    """Whole backward of the chunked layer (recomputes the up-projection per group of experts)."""
    _check("mop_moe_layer_bwd_chunked",
           lib().mop_moe_layer_bwd_chunked(ctx.handle, n_chunks, _ptr(x), _ptr(dY), _ptr(topk_gate), _ptr(offsets),
                                           _ptr(perm_row), _ptr(row_src), _ptr(W_gate), _ptr(W_up), _ptr(W_down),
                                           _ptr(dX), _ptr(dW_gate), _ptr(dW_up), _ptr(dW_down), _ptr(dgate),
                                           _ptr(workspace), _stream(stream)))


def mop_moe_forward_host(ctx, x_host, W_r, bias, W_gate, W_up, W_down, Y_host, idx_host=None, gate_host=None,
                         stream=None):
    """x_host / Y_host / idx_host / gate_host are HOST tensors (pinned for full copy speed)."""
    _check("mop_moe_forward_host",
           lib().mop_moe_forward_host(ctx.handle, _ptr(x_host), _ptr(W_r), _ptr(bias), _ptr(W_gate), _ptr(W_up),
                                      _ptr(W_down), _ptr(Y_host), _ptr(idx_host), _ptr(gate_host), _stream(stream)))


def mop_moe_train_step_host(ctx, x_host, dY_host, W_r, bias, W_gate, W_up, W_down, Y_host, dX_host, dgate_host,
                            dW_gate, dW_up, dW_down, stream=None):
    """x_host, dY_host, Y_host, dX_host, dgate_host are HOST tensors; weights and dW are device tensors."""
    _check("mop_moe_train_step_host",
           lib().mop_moe_train_step_host(ctx.handle, _ptr(x_host), _ptr(dY_host), _ptr(W_r), _ptr(bias), _ptr(W_gate),
                                         _ptr(W_up), _ptr(W_down), _ptr(Y_host), _ptr(dX_host), _ptr(dgate_host),
                                         _ptr(dW_gate), _ptr(dW_up), _ptr(dW_down), _stream(stream)))


def mop_moe_forward_host_async(ctx, x_host, W_r, bias, W_gate, W_up, W_down, Y_host, idx_host=None, gate_host=None,
                               stream=None):
    """Enqueues one forward on PINNED host tensors and returns; results are valid after mop_host_drain."""
    _check("mop_moe_forward_host_async",
           lib().mop_moe_forward_host_async(ctx.handle, _ptr(x_host), _ptr(W_r), _ptr(bias), _ptr(W_gate),
                                            _ptr(W_up), _ptr(W_down), _ptr(Y_host), _ptr(idx_host), _ptr(gate_host),
                                            _stream(stream)))


def mop_moe_train_step_host_async(ctx, x_host, dY_host, W_r, bias, W_gate, W_up, W_down, Y_host, dX_host, dgate_host,
                                  dW_gate, dW_up, dW_down, stream=None):
    """Enqueues one training step on PINNED host tensors and returns; results are valid after mop_host_drain."""
    _check("mop_moe_train_step_host_async",
           lib().mop_moe_train_step_host_async(ctx.handle, _ptr(x_host), _ptr(dY_host), _ptr(W_r), _ptr(bias),
                                               _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(Y_host), _ptr(dX_host),
                                               _ptr(dgate_host), _ptr(dW_gate), _ptr(dW_up), _ptr(dW_down),
                                               _stream(stream)))


def mop_host_drain(ctx, stream=None):
    _check("mop_host_drain", lib().mop_host_drain(ctx.handle, _stream(stream)))


def mop_moe_permute_static(device, T, d, E, k, x, topk_idx, counts, offsets, perm_row, row_src, Xp, stream=None):
    """Permutation for callers that may not allocate: no context, scratch compiled into the library."""
    _check("mop_moe_permute_static",
           lib().mop_moe_permute_static(device, T, d, E, k, _ptr(x), _ptr(topk_idx), _ptr(counts), _ptr(offsets),
                                        _ptr(perm_row), _ptr(row_src), _ptr(Xp), _stream(stream)))


def mop_vocab_workspace_bytes(N, H, V):
    return lib().mop_vocab_workspace_bytes(N, H, V)


def mop_vocab_loss_fwd(device, X, W_voc, targets, loss, lse=None, workspace=None, stream=None):
    """loss[n] = (X W_voc)[n, t_n] - logsumexp_v (X W_voc)[n, v]; the logits are never stored."""
    N, H = X.shape
    V = W_voc.shape[1]
    if workspace is None:
        workspace = torch.empty(max(256, mop_vocab_workspace_bytes(N, H, V)), dtype=torch.uint8, device=X.device)
    _check("mop_vocab_loss_fwd",
           lib().mop_vocab_loss_fwd(device, N, H, V, _ptr(X), _ptr(W_voc), _ptr(targets), _ptr(loss), _ptr(lse),
                                    _ptr(workspace), _stream(stream)))
    return workspace


def mop_vocab_poll(device, workspace, stream=None):
    _check("mop_vocab_poll", lib().mop_vocab_poll(device, _ptr(workspace), _stream(stream)))


def mop_vocab_selftest_wait_timeout(device, workspace, limit_cycles=20_000_000, stream=None):
    _check("mop_vocab_selftest_wait_timeout",
           lib().mop_vocab_selftest_wait_timeout(device, _ptr(workspace), limit_cycles, _stream(stream)))


def mop_vocab_bwd_workspace_bytes(N, H, V):
    return lib().mop_vocab_bwd_workspace_bytes(N, H, V)


def mop_vocab_loss_bwd(device, X, W_voc, targets, lse, dloss, dX, dW_voc, workspace=None, stream=None):
    """dX, dW_voc of sum_n dloss[n] * loglik[n]; only an N x 8192 block of the logit gradients is ever live."""
    N, H = X.shape
    V = W_voc.shape[1]
    if workspace is None:
        workspace = torch.empty(max(256, mop_vocab_bwd_workspace_bytes(N, H, V)), dtype=torch.uint8, device=X.device)
    _check("mop_vocab_loss_bwd",
           lib().mop_vocab_loss_bwd(device, N, H, V, _ptr(X), _ptr(W_voc), _ptr(targets), _ptr(lse), _ptr(dloss),
                                    _ptr(dX), _ptr(dW_voc), _ptr(workspace), _stream(stream)))
    return workspace


def mop_profile_enable(ctx, on=True):
    _check("mop_profile_enable", lib().mop_profile_enable(ctx.handle, int(on)))


def mop_profile_read(ctx, stream=None, max_names=64):
    """{kernel name: (total milliseconds, launches)} since the last read."""
    names = (ctypes.c_char_p * max_names)()
    ms = (ctypes.c_float * max_names)()
    calls = (ctypes.c_int32 * max_names)()
    n = lib().mop_profile_read(ctx.handle, _stream(stream), max_names, names, ms, calls)
    if n < 0:
        raise RuntimeError("mop_profile_read failed")
    return {names[i].decode(): (float(ms[i]), int(calls[i])) for i in range(n)}


class LayerBuffers:
    """Device tensors of one layer invocation (allocated by torch, owned by the caller)."""

    def __init__(self, w, device="cuda", backward=None):
        T, d, E, k, f = w.T, w.d, w.E, w.k, w.f
        M = T * k
        backward = w.backward if backward is None else backward
        i32 = dict(dtype=torch.int32, device=device)
        b16 = dict(dtype=torch.bfloat16, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        self.idx = torch.empty((T, k), **i32)
        self.gate = torch.empty((T, k), **f32)
        self.counts = torch.empty((E,), **i32)
        self.offsets = torch.empty((E + 1,), **i32)
        self.perm_row = torch.empty((M,), **i32)
        self.row_src = torch.empty((M,), **i32)
        self.Xp = torch.empty((M, d), **b16)
        self.H = torch.empty((M, f), **b16)
        self.Yp = torch.empty((M, d), **b16)
        self.Y = torch.empty((T, d), **b16)
        self.G = self.U = None
        if backward:
            self.G = torch.empty((M, f), **b16)
            self.U = torch.empty((M, f), **b16)
            self.dX = torch.empty((T, d), **b16)
            self.dgate = torch.empty((T, k), **f32)
            self.dW_gate = torch.empty((E, d, f), **f32)
            self.dW_up = torch.empty((E, d, f), **f32)
            self.dW_down = torch.empty((E, f, d), **f32)


def forward(ctx, inp, buf, stream=None, gather=False):
    """route -> permute -> expert_ffn_fwd -> combine on device tensors (one pass of the forward path)."""
    mop_moe_route(ctx, inp["x"], inp["W_r"], inp["bias"], buf.idx, buf.gate, None, stream)
    if gather:
        # inference form: no expert-contiguous copy of x, no stash
        mop_moe_permute(ctx, None, buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, None, stream)
        mop_moe_expert_ffn_fwd_gather(ctx, inp["x"], buf.offsets, buf.row_src, buf.gate, inp["W_gate"], inp["W_up"],
                                      inp["W_down"], buf.H, buf.Yp, stream)
        mop_moe_combine(ctx, buf.Yp, buf.perm_row, buf.Y, stream)
        return
    mop_moe_permute(ctx, inp["x"], buf.idx, buf.counts, buf.offsets, buf.perm_row, buf.row_src, buf.Xp, stream)
    mop_moe_expert_ffn_fwd(ctx, buf.Xp, buf.offsets, buf.row_src, buf.gate, inp["W_gate"], inp["W_up"], inp["W_down"],
                           buf.G, buf.U, buf.H, buf.Yp, stream)
    mop_moe_combine(ctx, buf.Yp, buf.perm_row, buf.Y, stream)


def backward(ctx, inp, buf, stream=None):
    mop_moe_expert_ffn_bwd(ctx, inp["dY"], buf.Xp, buf.G, buf.U, buf.H, buf.offsets, buf.perm_row, buf.row_src,
                           buf.gate, inp["W_gate"], inp["W_up"], inp["W_down"], buf.dX, buf.dW_gate, buf.dW_up,
                           buf.dW_down, buf.dgate, stream)


def context_for(w, device=0, gemm_path=GEMM_AUTO, backward=None, host_io=False, dw_accumulate=False,
                route_path=ROUTE_AUTO):
    backward = w.backward if backward is None else backward
    return Context(w.T, w.d, w.E, w.k, w.f, w.score_fn, w.bias_mode, backward, dw_accumulate, gemm_path, host_io,
                   device, route_path)
