"""The shared library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    inc = os.path.join(ROOT, "include")
    text = "\n".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?[A-Za-z_][\w\s\*]*?\b(\w+)\s*\([^;{]*\)\s*;", text, flags=re.M)
    return sorted(set(names))


def test_header_declares_the_entry_points():
    names = declared_symbols()
    for must in ("jacobi_sample", "sequential_sample", "js_made_create", "js_conv_create", "js_model_destroy",
                 "js_forward_logits", "js_set_option", "js_get_stats", "js_strerror", "js_last_cuda_error",
                 "jacobi_sample_host", "jacobi_sample_real", "sequential_sample_real", "js_forward_logits_real",
                 "jacobi_sample_noalloc", "js_get_trace", "rnn_forward", "rnn_bptt_sequential", "rnn_bptt_jacobi",
                 "rnn_param_grads", "rnn_last_error"):
        assert must in names, names


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as ge
    ge.build()
    import paper_2002_03629_b200 as pkg
    lib = pkg.load_library()
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert lib.js_strerror(0) == b"ok"


def test_calls_fail_loudly_without_a_device():
    import numpy as np
    import torch
    import paper_2002_03629_b200 as pkg
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(pkg.JsError) as e:
        pkg.Model.made(4, 1, [8], 0, 0, [np.zeros((8, 4), np.float32), np.zeros((4, 8), np.float32)],
                       [np.zeros(8, np.float32), np.zeros(4, np.float32)], np.array([0, 1], np.float32), 4)
    assert e.value.code == pkg.JS_ERR_CUDA
