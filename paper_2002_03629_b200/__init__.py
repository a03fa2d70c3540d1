"""B200 sampler for masked autoregressive networks by parallel fixed-point
iteration (Jacobi, Gauss-Seidel and block hybrids; arXiv 2002.03629).

The work is done by ``libjacobi_sample.so`` (hand-written CUDA for sm_100a,
C ABI in ``include/jacobi_sample.h``).  This package only marshals arguments:
``torch`` provides device memory and streams.
"""
from .binding import (  # noqa: F401
    JS_JACOBI, JS_GAUSS_SEIDEL, JS_GS_JACOBI, JS_JACOBI_GS,
    JS_NOISE_UNIFORM_ICDF, JS_NOISE_LOGISTIC, JS_NOISE_GUMBEL, JS_NOISE_UNIFORM_CAT,
    JS_ACT_RELU, JS_ACT_GELU_TANH, JS_F32, JS_BF16,
    JS_OK, JS_NOT_CONVERGED, JS_ERR_ARG, JS_ERR_UNSUPPORTED, JS_ERR_CUDA, JS_ERR_TIMEOUT,
    JS_OPT_FRONTIER_SKIP, JS_OPT_SEQ_SKIP, JS_OPT_SPIN_LIMIT, JS_OPT_PATH, JS_OPT_COMPACT, JS_OPT_TRACE,
    JsError, Model, load_library, jacobi_sample, jacobi_sample_host, sequential_sample, js_forward_logits,
    jacobi_sample_real, sequential_sample_real, js_forward_logits_real,
    jacobi_sample_noalloc, noalloc_scratch_needed, noalloc_scratch_limit,
)
