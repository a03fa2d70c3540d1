"""ctypes binding of ``libjacobi_sample.so``: same names as the C ABI, argument
marshalling only.  Fails loudly if the library is missing; there is no fallback."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

JS_JACOBI, JS_GAUSS_SEIDEL, JS_GS_JACOBI, JS_JACOBI_GS = 0, 1, 2, 3
JS_NOISE_UNIFORM_ICDF, JS_NOISE_LOGISTIC, JS_NOISE_GUMBEL, JS_NOISE_UNIFORM_CAT = 0, 1, 2, 3
JS_ACT_RELU, JS_ACT_GELU_TANH = 0, 1
JS_F32, JS_BF16 = 0, 1
JS_OK, JS_NOT_CONVERGED = 0, 1
JS_ERR_ARG, JS_ERR_UNSUPPORTED, JS_ERR_CUDA, JS_ERR_TIMEOUT = -1, -2, -3, -4
JS_OPT_FRONTIER_SKIP, JS_OPT_SEQ_SKIP, JS_OPT_SPIN_LIMIT, JS_OPT_PATH, JS_OPT_COMPACT, JS_OPT_TRACE = 0, 1, 2, 3, 4, 5

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libjacobi_sample.so")
_lib = None


class JsError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(what)


class _MadeDesc(C.Structure):
    _fields_ = [("T", C.c_int), ("C", C.c_int), ("L", C.c_int), ("H", C.POINTER(C.c_int)),
                ("act", C.c_int), ("prec", C.c_int),
                ("W", C.POINTER(C.POINTER(C.c_float))), ("b", C.POINTER(C.POINTER(C.c_float))),
                ("lut", C.POINTER(C.c_float)), ("n_lut", C.c_int),
                ("hidden_deg", C.POINTER(C.POINTER(C.c_int))), ("max_batch", C.c_int)]


class _ConvDesc(C.Structure):
    _fields_ = [("height", C.c_int), ("width", C.c_int), ("in_ch", C.c_int), ("ch", C.c_int),
                ("n_conv", C.c_int), ("C", C.c_int), ("prec", C.c_int),
                ("W", C.POINTER(C.POINTER(C.c_float))), ("b", C.POINTER(C.POINTER(C.c_float))),
                ("lut", C.POINTER(C.c_float)), ("n_lut", C.c_int), ("max_batch", C.c_int)]


class _NoallocMade(C.Structure):
    _fields_ = [("T", C.c_int), ("C", C.c_int), ("L", C.c_int), ("H", C.c_int * 8), ("act", C.c_int),
                ("W_dev", C.c_void_p * 9), ("b_dev", C.c_void_p * 9), ("lut_dev", C.c_void_p)]


class JsStats(C.Structure):
    _fields_ = [("iterations", C.c_int), ("batch_iters_max", C.c_int), ("final_frontier", C.c_int),
                ("tiles_issued", C.c_longlong), ("tiles_skipped", C.c_longlong), ("path", C.c_int),
                ("status", C.c_int), ("compactions", C.c_int), ("mma_flops", C.c_longlong), ("weight_bytes", C.c_longlong)]


def load_library():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise JsError(JS_ERR_CUDA, f"{_LIB_PATH} is missing: run __graft_entry__.build() "
                                   "(python -m paper_2002_03629_b200.build)")
    lib = C.CDLL(_LIB_PATH)
    vp, ip = C.c_void_p, C.c_int
    lib.js_made_create.argtypes = [C.POINTER(_MadeDesc), C.POINTER(vp)]
    lib.js_conv_create.argtypes = [C.POINTER(_ConvDesc), C.POINTER(vp)]
    lib.js_model_destroy.argtypes = [vp]
    lib.js_model_destroy.restype = None
    lib.jacobi_sample.argtypes = [vp, ip, vp, ip, vp, ip, ip, ip, vp, vp, vp]
    lib.jacobi_sample_host.argtypes = [vp, ip, vp, ip, vp, ip, ip, ip, vp, vp, vp]
    lib.sequential_sample.argtypes = [vp, ip, vp, ip, vp, vp]
    lib.js_forward_logits.argtypes = [vp, ip, vp, vp, vp]
    lib.jacobi_sample_real.argtypes = [vp, ip, vp, vp, ip, ip, ip, C.c_float, vp, vp, vp]
    lib.sequential_sample_real.argtypes = [vp, ip, vp, vp, vp]
    lib.js_forward_logits_real.argtypes = [vp, ip, vp, vp, vp]
    lib.js_set_option.argtypes = [vp, ip, ip]
    lib.js_get_stats.argtypes = [vp, C.POINTER(JsStats)]
    lib.js_get_trace.argtypes = [vp, vp, ip]
    lib.js_strerror.argtypes = [ip]
    lib.js_strerror.restype = C.c_char_p
    lib.js_last_cuda_error.restype = C.c_char_p
    lib.jacobi_sample_noalloc.argtypes = [C.POINTER(_NoallocMade), ip, vp, ip, vp, ip, vp, vp, vp]
    lib.js_noalloc_scratch_limit.restype = C.c_size_t
    lib.js_noalloc_scratch_needed.argtypes = [C.POINTER(_NoallocMade), ip]
    lib.js_noalloc_scratch_needed.restype = C.c_size_t
    lib.js_noalloc_last_error.restype = C.c_char_p
    _lib = lib
    return lib


def _check(rc: int, what: str) -> int:
    if rc < 0:
        lib = load_library()
        msg = lib.js_strerror(rc).decode()
        if rc == JS_ERR_CUDA:
            msg += ": " + lib.js_last_cuda_error().decode()
        raise JsError(rc, f"{what}: {msg}")
    return rc


def _fp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dev(t: Optional[torch.Tensor], dtype, what: str):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise JsError(JS_ERR_ARG, f"{what}: expected a contiguous CUDA tensor of {dtype}")
    return C.c_void_p(t.data_ptr())


class Model:
    """Owner of a ``js_model`` handle."""

    def __init__(self, handle: int, T: int, Cc: int):
        self._h = C.c_void_p(handle)
        self.T, self.C = T, Cc

    @classmethod
    def made(cls, T: int, Cc: int, H: Sequence[int], act: int, prec: int, W: List[np.ndarray],
             b: List[np.ndarray], lut: np.ndarray, max_batch: int,
             hidden_deg: Optional[List[np.ndarray]] = None) -> "Model":
        """js_made_create: W[l] unmasked float32 [out, in] host arrays; masks are applied by the library."""
        lib = load_library()
        L = len(H)
        W = [np.ascontiguousarray(w, dtype=np.float32) for w in W]
        b = [np.ascontiguousarray(v, dtype=np.float32) for v in b]
        lut = np.ascontiguousarray(lut, dtype=np.float32)
        widths = [T, *H, T * Cc]
        for l in range(L + 1):
            if W[l].shape != (widths[l + 1], widths[l]) or b[l].shape != (widths[l + 1],):
                raise JsError(JS_ERR_ARG, f"layer {l}: bad weight or bias shape")
        d = _MadeDesc()
        d.T, d.C, d.L, d.act, d.prec, d.max_batch = T, Cc, L, act, prec, max_batch
        Hs = (C.c_int * L)(*H)
        d.H = Hs
        Wp = (C.POINTER(C.c_float) * (L + 1))(*[_fp(w) for w in W])
        bp = (C.POINTER(C.c_float) * (L + 1))(*[_fp(v) for v in b])
        d.W, d.b, d.lut, d.n_lut = Wp, bp, _fp(lut), len(lut)
        keep = None
        if hidden_deg is not None:
            keep = [np.ascontiguousarray(x, dtype=np.int32) for x in hidden_deg]
            d.hidden_deg = (C.POINTER(C.c_int) * L)(*[x.ctypes.data_as(C.POINTER(C.c_int)) for x in keep])
        h = C.c_void_p()
        _check(lib.js_made_create(C.byref(d), C.byref(h)), "js_made_create")
        return cls(h.value, T, Cc)

    @classmethod
    def conv(cls, height: int, width: int, in_ch: int, ch: int, n_conv: int, Cc: int, prec: int,
             W: List[np.ndarray], b: List[np.ndarray], lut: np.ndarray, max_batch: int) -> "Model":
        """js_conv_create."""
        lib = load_library()
        W = [np.ascontiguousarray(w, dtype=np.float32) for w in W]
        b = [np.ascontiguousarray(v, dtype=np.float32) for v in b]
        lut = np.ascontiguousarray(lut, dtype=np.float32)
        d = _ConvDesc()
        d.height, d.width, d.in_ch, d.ch, d.n_conv, d.C, d.prec = height, width, in_ch, ch, n_conv, Cc, prec
        d.max_batch = max_batch
        Wp = (C.POINTER(C.c_float) * (n_conv + 1))(*[_fp(w) for w in W])
        bp = (C.POINTER(C.c_float) * (n_conv + 1))(*[_fp(v) for v in b])
        d.W, d.b, d.lut, d.n_lut = Wp, bp, _fp(lut), len(lut)
        h = C.c_void_p()
        _check(lib.js_conv_create(C.byref(d), C.byref(h)), "js_conv_create")
        return cls(h.value, height * width * in_ch, Cc)

    @classmethod
    def from_config(cls, cfg, W, b, lut, max_batch: Optional[int] = None) -> "Model":
        mb = cfg.batch if max_batch is None else max_batch
        if cfg.kind == "made":
            return cls.made(cfg.D, cfg.C, list(cfg.H), cfg.act, cfg.prec, W, b, lut, mb)
        return cls.conv(cfg.height, cfg.width, cfg.in_ch, cfg.ch, cfg.layers, cfg.C, cfg.prec, W, b, lut, mb)

    def set_option(self, option: int, value: int) -> None:
        _check(load_library().js_set_option(self._h, option, value), "js_set_option")

    def stats(self) -> JsStats:
        s = JsStats()
        _check(load_library().js_get_stats(self._h, C.byref(s)), "js_get_stats")
        return s

    def trace(self) -> np.ndarray:
        """js_get_trace: device timestamps [2 CTAs][256 phases][12 slots] of the last traced call."""
        buf = np.zeros((2, 256, 12), dtype=np.uint64)
        _check(load_library().js_get_trace(self._h, buf.ctypes.data_as(C.c_void_p), buf.size), "js_get_trace")
        return buf

    def close(self) -> None:
        if self._h:
            load_library().js_model_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def jacobi_sample(model: Model, noise: torch.Tensor, nk: int, init: Optional[torch.Tensor], mode: int,
                  block: int, max_iters: int, out_samples: torch.Tensor,
                  out_iters: Optional[torch.Tensor] = None, stream=None) -> int:
    """jacobi_sample of the C ABI on CUDA tensors.  Returns 0 or JS_NOT_CONVERGED; raises JsError on errors."""
    batch = out_samples.shape[0]
    rc = load_library().jacobi_sample(
        model._h, batch, _dev(noise, torch.float32, "noise"), nk, _dev(init, torch.uint8, "init"), mode, block,
        max_iters, _dev(out_samples, torch.uint8, "out_samples"), _dev(out_iters, torch.int32, "out_iters"),
        _stream_ptr(stream))
    return _check(rc, "jacobi_sample")


def _host(t: Optional[torch.Tensor], dtype, what: str):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise JsError(JS_ERR_ARG, f"{what}: expected a contiguous CPU tensor of {dtype}")
    return C.c_void_p(t.data_ptr())


def jacobi_sample_host(model: Model, noise: torch.Tensor, nk: int, init: Optional[torch.Tensor], mode: int,
                       block: int, max_iters: int, out_samples: torch.Tensor,
                       out_iters: Optional[torch.Tensor] = None, stream=None) -> int:
    """jacobi_sample_host of the C ABI: CPU tensors in and out (pinned ones upload asynchronously)."""
    batch = out_samples.shape[0]
    rc = load_library().jacobi_sample_host(
        model._h, batch, _host(noise, torch.float32, "noise"), nk, _host(init, torch.uint8, "init"), mode, block,
        max_iters, _host(out_samples, torch.uint8, "out_samples"), _host(out_iters, torch.int32, "out_iters"),
        _stream_ptr(stream))
    return _check(rc, "jacobi_sample_host")


def sequential_sample(model: Model, noise: torch.Tensor, nk: int, out_samples: torch.Tensor, stream=None) -> int:
    batch = out_samples.shape[0]
    rc = load_library().sequential_sample(model._h, batch, _dev(noise, torch.float32, "noise"), nk,
                                          _dev(out_samples, torch.uint8, "out_samples"), _stream_ptr(stream))
    return _check(rc, "sequential_sample")


def js_forward_logits(model: Model, x: torch.Tensor, logits: torch.Tensor, stream=None) -> int:
    batch = x.shape[0]
    rc = load_library().js_forward_logits(model._h, batch, _dev(x, torch.uint8, "x"),
                                          _dev(logits, torch.float32, "logits"), _stream_ptr(stream))
    return _check(rc, "js_forward_logits")


def jacobi_sample_real(model: Model, noise: torch.Tensor, init: Optional[torch.Tensor], mode: int, block: int,
                       max_iters: int, eps: float, out_states: torch.Tensor,
                       out_iters: Optional[torch.Tensor] = None, stream=None) -> int:
    """jacobi_sample_real of the C ABI: continuous states with logistic conditionals, stopping tolerance eps."""
    rc = load_library().jacobi_sample_real(
        model._h, out_states.shape[0], _dev(noise, torch.float32, "noise"), _dev(init, torch.float32, "init"), mode,
        block, max_iters, float(eps), _dev(out_states, torch.float32, "out_states"),
        _dev(out_iters, torch.int32, "out_iters"), _stream_ptr(stream))
    return _check(rc, "jacobi_sample_real")


def sequential_sample_real(model: Model, noise: torch.Tensor, out_states: torch.Tensor, stream=None) -> int:
    rc = load_library().sequential_sample_real(model._h, out_states.shape[0], _dev(noise, torch.float32, "noise"),
                                               _dev(out_states, torch.float32, "out_states"), _stream_ptr(stream))
    return _check(rc, "sequential_sample_real")


def js_forward_logits_real(model: Model, x: torch.Tensor, logits: torch.Tensor, stream=None) -> int:
    rc = load_library().js_forward_logits_real(model._h, x.shape[0], _dev(x, torch.float32, "x"),
                                               _dev(logits, torch.float32, "logits"), _stream_ptr(stream))
    return _check(rc, "js_forward_logits_real")


def _noalloc_net(T: int, Cc: int, H: Sequence[int], act: int, W: List[torch.Tensor], b: List[torch.Tensor],
                 lut: torch.Tensor) -> _NoallocMade:
    net = _NoallocMade()
    net.T, net.C, net.L, net.act = T, Cc, len(H), act
    for i, h in enumerate(H):
        net.H[i] = h
    for l in range(len(H) + 1):
        net.W_dev[l] = _dev(W[l], torch.float32, f"W[{l}]").value
        net.b_dev[l] = _dev(b[l], torch.float32, f"b[{l}]").value
    net.lut_dev = _dev(lut, torch.float32, "lut").value
    return net


def jacobi_sample_noalloc(T: int, Cc: int, H: Sequence[int], act: int, W: List[torch.Tensor],
                          b: List[torch.Tensor], lut: torch.Tensor, noise: torch.Tensor, nk: int,
                          init: Optional[torch.Tensor], max_iters: int, out_samples: torch.Tensor,
                          out_iters: Optional[torch.Tensor] = None, stream=None) -> int:
    """jacobi_sample_noalloc of the C ABI: for callers that may not allocate device memory.  Every
    tensor (unmasked fp32 weights included) is a CUDA tensor the caller already owns; the library
    allocates nothing and uses its built-in scratch array.  Calls must not overlap on the GPU."""
    lib = load_library()
    net = _noalloc_net(T, Cc, H, act, W, b, lut)
    rc = lib.jacobi_sample_noalloc(C.byref(net), out_samples.shape[0], _dev(noise, torch.float32, "noise"), nk,
                                   _dev(init, torch.uint8, "init"), max_iters,
                                   _dev(out_samples, torch.uint8, "out_samples"),
                                   _dev(out_iters, torch.int32, "out_iters"), _stream_ptr(stream))
    if rc < 0:
        raise JsError(rc, "jacobi_sample_noalloc: " + (lib.js_noalloc_last_error().decode()
                                                       or lib.js_strerror(rc).decode()))
    return rc


def noalloc_scratch_needed(T: int, Cc: int, H: Sequence[int], batch: int) -> int:
    net = _NoallocMade()
    net.T, net.C, net.L = T, Cc, len(H)
    for i, h in enumerate(H):
        net.H[i] = h
    return int(load_library().js_noalloc_scratch_needed(C.byref(net), batch))


def noalloc_scratch_limit() -> int:
    return int(load_library().js_noalloc_scratch_limit())
