"""Binding of the recurrent-network workload (``include/rnn_bptt.h``): argument marshalling only.

``torch`` provides device memory and streams; every step runs in the CUDA library.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import torch

from .binding import JsError, JS_ERR_ARG, load_library, _stream_ptr

RNN_OK, RNN_ERR_INVALID, RNN_ERR_CUDA = 0, -1, -2
RNN_MAX_T, RNN_MAX_H, RNN_MAX_IO = 128, 128, 16

_ready = False


def _lib():
    global _ready
    lib = load_library()
    if not _ready:
        vp, ip = C.c_void_p, C.c_int
        lib.rnn_forward.argtypes = [vp] * 7 + [ip] * 5 + [vp] * 5
        lib.rnn_bptt_sequential.argtypes = [vp, vp, vp, ip, ip, ip, vp, vp]
        lib.rnn_bptt_jacobi.argtypes = [vp, vp, vp, ip, ip, ip, ip, vp, vp, vp]
        lib.rnn_param_grads.argtypes = [vp] * 4 + [ip] * 4 + [vp] * 4
        lib.rnn_last_error.restype = C.c_char_p
        _ready = True
    return lib


def _f32(t: Optional[torch.Tensor], what: str):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise JsError(JS_ERR_ARG, f"{what}: expected a contiguous CUDA tensor of float32")
    return C.c_void_p(t.data_ptr())


def _check(rc: int, what: str):
    if rc != RNN_OK:
        detail = _lib().rnn_last_error().decode() if rc == RNN_ERR_CUDA else "argument outside the documented limits"
        raise JsError(rc, f"{what}: {detail}")


def rnn_forward(Wh, Wx, b, Wo, bo, x, r, stream=None):
    """Forward pass; returns (h, d, l, loss) as new device tensors.  x [B,T,d_in], r [B,T,d_out]."""
    B, T, d_in = x.shape
    H, d_out = Wh.shape[0], r.shape[2]
    h = torch.empty((B, T, H), dtype=torch.float32, device=x.device)
    d = torch.empty_like(h)
    l = torch.empty_like(h)
    loss = torch.empty((B,), dtype=torch.float32, device=x.device)
    rc = _lib().rnn_forward(_f32(Wh, "Wh"), _f32(Wx, "Wx"), _f32(b, "b"), _f32(Wo, "Wo"), _f32(bo, "bo"), _f32(x, "x"),
                            _f32(r, "r"), B, T, H, d_in, d_out, _f32(h, "h"), _f32(d, "d"), _f32(l, "l"),
                            _f32(loss, "loss"), _stream_ptr(stream))
    _check(rc, "rnn_forward")
    return h, d, l, loss


def rnn_bptt_sequential(Wh, l, d, out=None, stream=None):
    """Exact state gradients s [B,T,H] by back-substitution."""
    B, T, H = l.shape
    s = torch.empty_like(l) if out is None else out
    _check(_lib().rnn_bptt_sequential(_f32(Wh, "Wh"), _f32(l, "l"), _f32(d, "d"), B, T, H, _f32(s, "s"),
                                      _stream_ptr(stream)), "rnn_bptt_sequential")
    return s


def rnn_bptt_jacobi(Wh, l, d, n_iters: int, s0=None, out=None, stream=None):
    """Jacobi_n: state gradients after n_iters Jacobi iterations from s0 (zeros if None)."""
    B, T, H = l.shape
    s = torch.empty_like(l) if out is None else out
    _check(_lib().rnn_bptt_jacobi(_f32(Wh, "Wh"), _f32(l, "l"), _f32(d, "d"), B, T, H, int(n_iters), _f32(s0, "s0"),
                                  _f32(s, "s"), _stream_ptr(stream)), "rnn_bptt_jacobi")
    return s


def rnn_param_grads(s, d, h, x, stream=None):
    """Per-sequence parameter gradients (dWh [B,H,H], dWx [B,H,d_in], db [B,H])."""
    B, T, H = s.shape
    d_in = x.shape[2]
    dWh = torch.empty((B, H, H), dtype=torch.float32, device=s.device)
    dWx = torch.empty((B, H, d_in), dtype=torch.float32, device=s.device)
    db = torch.empty((B, H), dtype=torch.float32, device=s.device)
    _check(_lib().rnn_param_grads(_f32(s, "s"), _f32(d, "d"), _f32(h, "h"), _f32(x, "x"), B, T, H, d_in, _f32(dWh, "dWh"),
                                  _f32(dWx, "dWx"), _f32(db, "db"), _stream_ptr(stream)), "rnn_param_grads")
    return dWh, dWx, db
