"""ctypes front end of the CPU oracle (``jacobi_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this package and
this package never imports the CUDA library.

Every solver of the C file handles one sample; the ``*_batch`` helpers here loop
over samples, optionally on a thread pool (ctypes drops the GIL during a call).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "jacobi_oracle.c")
_LIB = os.path.join(_HERE, "libjacobi_oracle.so")

NOISE_UNIFORM_ICDF, NOISE_LOGISTIC, NOISE_GUMBEL, NOISE_UNIFORM_CAT = 0, 1, 2, 3
ACT_RELU, ACT_GELU_TANH = 0, 1
PREC_F32, PREC_BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        # ORACLE_LIB: a test plants mistakes in copies of the C source and points this at them,
        # to show that the pins notice (tests/test_oracle_mutants.py)
        _lib = C.CDLL(os.environ.get("ORACLE_LIB") or build())
        _lib.orc_made_create.restype = C.c_void_p
        _lib.orc_conv_create.restype = C.c_void_p
        _lib.orc_masked_weight.restype = C.POINTER(C.c_float)
        _lib.orc_degrees.restype = C.POINTER(C.c_int)
    return _lib


def _fptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _u8(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_uint8))


class Oracle:
    """A masked autoregressive network held by the oracle, plus its solvers."""

    def __init__(self, handle, T: int, Cc: int, keep):
        self._h = C.c_void_p(handle)
        self.T, self.C = T, Cc
        self._keep = keep

    # ---- construction -------------------------------------------------
    @classmethod
    def made(cls, D: int, Cc: int, H: Sequence[int], act: int, prec: int,
             W: List[np.ndarray], b: List[np.ndarray], lut: np.ndarray,
             hidden_deg: Optional[List[np.ndarray]] = None) -> "Oracle":
        L = len(H)
        W = [np.ascontiguousarray(w, dtype=np.float32) for w in W]
        b = [np.ascontiguousarray(v, dtype=np.float32) for v in b]
        lut = np.ascontiguousarray(lut, dtype=np.float32)
        widths = [D, *H, D * Cc]
        for l in range(L + 1):
            assert W[l].shape == (widths[l + 1], widths[l]), (l, W[l].shape)
            assert b[l].shape == (widths[l + 1],)
        Wp = (C.POINTER(C.c_float) * (L + 1))(*[_fptr(w) for w in W])
        bp = (C.POINTER(C.c_float) * (L + 1))(*[_fptr(v) for v in b])
        Hs = (C.c_int * L)(*H)
        degp = None
        keep = [W, b, lut]
        if hidden_deg is not None:
            hd = [np.ascontiguousarray(d, dtype=np.int32) for d in hidden_deg]
            degp = (C.POINTER(C.c_int) * L)(*[d.ctypes.data_as(C.POINTER(C.c_int)) for d in hd])
            keep.append(hd)
        h = lib().orc_made_create(D, Cc, L, Hs, act, prec, Wp, bp, _fptr(lut), len(lut), degp)
        assert h, "orc_made_create failed"
        o = cls(h, D, Cc, None)          # the C side copied everything it needs
        o.kind, o.L, o.widths = "made", L, widths
        return o

    @classmethod
    def conv(cls, height: int, width: int, in_ch: int, ch: int, n_conv: int, Cc: int, prec: int,
             W: List[np.ndarray], b: List[np.ndarray], lut: np.ndarray) -> "Oracle":
        W = [np.ascontiguousarray(w, dtype=np.float32) for w in W]
        b = [np.ascontiguousarray(v, dtype=np.float32) for v in b]
        lut = np.ascontiguousarray(lut, dtype=np.float32)
        assert len(W) == n_conv + 1
        Wp = (C.POINTER(C.c_float) * (n_conv + 1))(*[_fptr(w) for w in W])
        bp = (C.POINTER(C.c_float) * (n_conv + 1))(*[_fptr(v) for v in b])
        h = lib().orc_conv_create(height, width, in_ch, ch, n_conv, Cc, prec, Wp, bp, _fptr(lut), len(lut))
        assert h, "orc_conv_create failed"
        o = cls(h, height * width * in_ch, Cc, None)
        o.kind, o.L = "conv", n_conv
        return o

    def __del__(self):
        try:
            lib().orc_model_destroy(self._h)
        except Exception:
            pass

    # ---- introspection (tests recompute the forward pass from these) ---
    def masked_weight(self, l: int, shape) -> np.ndarray:
        p = lib().orc_masked_weight(self._h, l)
        n = int(np.prod(shape))
        return np.ctypeslib.as_array(p, shape=(n,)).reshape(shape).copy()

    def degrees(self, l: int) -> np.ndarray:
        p = lib().orc_degrees(self._h, l)
        return np.ctypeslib.as_array(p, shape=(self.widths[l],)).copy()

    # ---- single-sample calls -------------------------------------------
    def _noise(self, noise: np.ndarray, nk: int) -> np.ndarray:
        noise = np.ascontiguousarray(noise, dtype=np.float32)
        want = (self.T, self.C) if nk == NOISE_GUMBEL else (self.T,)
        assert noise.shape == want, (noise.shape, want)
        return noise

    def forward_logits(self, x: np.ndarray) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.uint8)
        assert x.shape == (self.T,)
        z = np.empty((self.T, self.C), dtype=np.float32)
        lib().orc_forward_logits(self._h, _u8(x), _fptr(z))
        return z

    def jacobi_step(self, x: np.ndarray, noise: np.ndarray, nk: int) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.uint8)
        noise = self._noise(noise, nk)
        out = np.empty(self.T, dtype=np.uint8)
        lib().orc_jacobi_step(self._h, _u8(x), _fptr(noise), nk, _u8(out))
        return out

    def margins(self, x: np.ndarray, noise: np.ndarray, nk: int) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.uint8)
        noise = self._noise(noise, nk)
        out = np.empty(self.T, dtype=np.float32)
        lib().orc_margins(self._h, _u8(x), _fptr(noise), nk, _fptr(out))
        return out

    def sequential(self, noise: np.ndarray, nk: int, literal: bool = False) -> np.ndarray:
        noise = self._noise(noise, nk)
        x = np.empty(self.T, dtype=np.uint8)
        f = lib().orc_sequential_literal if literal else lib().orc_sequential
        f(self._h, _fptr(noise), nk, _u8(x))
        return x

    def gauss_seidel(self, noise: np.ndarray, nk: int, init: Optional[np.ndarray] = None) -> np.ndarray:
        noise = self._noise(noise, nk)
        init = None if init is None else np.ascontiguousarray(init, dtype=np.uint8)
        x = np.empty(self.T, dtype=np.uint8)
        lib().orc_gauss_seidel(self._h, _fptr(noise), nk, _u8(init), _u8(x))
        return x

    def jacobi(self, noise: np.ndarray, nk: int, init: Optional[np.ndarray] = None, max_iters: int = 0,
               x_star: Optional[np.ndarray] = None):
        """Returns (x, iters, converged, k_correct)."""
        noise = self._noise(noise, nk)
        init = None if init is None else np.ascontiguousarray(init, dtype=np.uint8)
        xs = None if x_star is None else np.ascontiguousarray(x_star, dtype=np.uint8)
        x = np.empty(self.T, dtype=np.uint8)
        it, cv, kc = C.c_int(0), C.c_int(0), C.c_int(-1)
        lib().orc_jacobi(self._h, _fptr(noise), nk, _u8(init), max_iters, _u8(x),
                         C.byref(it), C.byref(cv), _u8(xs), C.byref(kc))
        return x, it.value, bool(cv.value), kc.value

    def _hybrid(self, fn, noise, nk, init, block, max_iters):
        noise = self._noise(noise, nk)
        init = None if init is None else np.ascontiguousarray(init, dtype=np.uint8)
        x = np.empty(self.T, dtype=np.uint8)
        it, cv = C.c_int(0), C.c_int(0)
        fn(self._h, _fptr(noise), nk, _u8(init), block, max_iters, _u8(x), C.byref(it), C.byref(cv))
        return x, it.value, bool(cv.value)

    def gs_jacobi(self, noise, nk, block: int, init=None, max_iters: int = 0):
        """Algorithm 3.  Returns (x, summed inner iterations, converged)."""
        return self._hybrid(lib().orc_gs_jacobi, noise, nk, init, block, max_iters)

    def jacobi_gs(self, noise, nk, block: int, init=None, max_iters: int = 0, literal: bool = False):
        """Algorithm 2.  Returns (x, outer iterations, converged)."""
        fn = lib().orc_jacobi_gs_literal if literal else lib().orc_jacobi_gs
        return self._hybrid(fn, noise, nk, init, block, max_iters)

    # ---- continuous states (C == 2: location and log-scale per position) ----
    def _real(self, a, n):
        a = np.ascontiguousarray(a, dtype=np.float32)
        assert a.shape == (n,), a.shape
        return a

    def forward_logits_real(self, x: np.ndarray) -> np.ndarray:
        assert self.C == 2
        x = self._real(x, self.T)
        z = np.empty((self.T, 2), dtype=np.float32)
        lib().orc_forward_logits_real(self._h, _fptr(x), _fptr(z))
        return z

    def jacobi_step_real(self, x: np.ndarray, noise: np.ndarray) -> np.ndarray:
        x, noise = self._real(x, self.T), self._real(noise, self.T)
        out = np.empty(self.T, dtype=np.float32)
        lib().orc_jacobi_step_real(self._h, _fptr(x), _fptr(noise), _fptr(out))
        return out

    def sequential_real(self, noise: np.ndarray) -> np.ndarray:
        noise = self._real(noise, self.T)
        x = np.empty(self.T, dtype=np.float32)
        lib().orc_sequential_real(self._h, _fptr(noise), _fptr(x))
        return x

    def jacobi_real(self, noise: np.ndarray, eps: float = 0.0, init: Optional[np.ndarray] = None, max_iters: int = 0):
        """Algorithm 1 on continuous states.  Returns (x, iters, converged)."""
        noise = self._real(noise, self.T)
        init = None if init is None else self._real(init, self.T)
        x = np.empty(self.T, dtype=np.float32)
        it, cv = C.c_int(0), C.c_int(0)
        lib().orc_jacobi_real(self._h, _fptr(noise), None if init is None else _fptr(init), C.c_float(eps), max_iters,
                              _fptr(x), C.byref(it), C.byref(cv))
        return x, it.value, bool(cv.value)

    def gs_jacobi_real(self, noise: np.ndarray, block: int, eps: float = 0.0, init: Optional[np.ndarray] = None,
                       max_iters: int = 0):
        """Algorithm 3 on continuous states.  Returns (x, summed inner iterations, converged)."""
        noise = self._real(noise, self.T)
        init = None if init is None else self._real(init, self.T)
        x = np.empty(self.T, dtype=np.float32)
        it, cv = C.c_int(0), C.c_int(0)
        lib().orc_gs_jacobi_real(self._h, _fptr(noise), None if init is None else _fptr(init), block, C.c_float(eps),
                                 max_iters, _fptr(x), C.byref(it), C.byref(cv))
        return x, it.value, bool(cv.value)

    # ---- batches ---------------------------------------------------------
    def map_batch(self, fn, n: int, threads: int = 1):
        """Run ``fn(i)`` for i in range(n), on a thread pool if threads > 1."""
        if threads <= 1:
            return [fn(i) for i in range(n)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            return list(ex.map(fn, range(n)))

    def sequential_batch(self, noise: np.ndarray, nk: int, threads: int = 1) -> np.ndarray:
        res = self.map_batch(lambda i: self.sequential(noise[i], nk), noise.shape[0], threads)
        return np.stack(res)

    def jacobi_batch(self, noise: np.ndarray, nk: int, init: Optional[np.ndarray] = None,
                     max_iters: int = 0, threads: int = 1):
        def one(i):
            return self.jacobi(noise[i], nk, None if init is None else init[i], max_iters)
        res = self.map_batch(one, noise.shape[0], threads)
        return (np.stack([r[0] for r in res]), np.array([r[1] for r in res], dtype=np.int32),
                np.array([r[2] for r in res]))


def from_config(cfg, W, b, lut) -> Oracle:
    """Oracle model for a workload description of ``synth_inputs``."""
    if cfg.kind == "made":
        return Oracle.made(cfg.D, cfg.C, list(cfg.H), cfg.act, cfg.prec, W, b, lut)
    return Oracle.conv(cfg.height, cfg.width, cfg.in_ch, cfg.ch, cfg.layers, cfg.C, cfg.prec, W, b, lut)
