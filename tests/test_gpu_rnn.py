"""Parity of the recurrent-network CUDA path (include/rnn_bptt.h) with the float64 oracle, element by
element on the same seeded inputs (arXiv 2002.03629, Section 5.1).

Tolerance.  The CUDA path computes in fp32 with fused multiply-adds; every value is a sum of at most
H + d_in + 1 = 130 products per step, and the backward recursion contracts (the oracle's own Jacobi
iterates converge geometrically), so rounding errors do not build up over the steps.  A state or a
gradient of magnitude m is therefore matched to about 130 * 2^-24 * m ~ 1e-5 m; the tests allow
1e-4 of the array's largest magnitude plus 1e-4 relative.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import rnn_oracle as ro

pytestmark = pytest.mark.gpu


def close(got: torch.Tensor, want: np.ndarray, what=""):
    g = got.detach().cpu().double().numpy()
    scale = np.abs(want).max()
    np.testing.assert_allclose(g, want, rtol=1e-4, atol=1e-4 * scale + 1e-12, err_msg=what)


def case(name, **changes):
    cfg = si.RNN_CONFIGS[name]
    if changes:
        from dataclasses import replace
        cfg = replace(cfg, **changes)
    Wh, Wx, b, Wo, bo = si.rnn_weights(cfg)
    rng = np.random.default_rng(3)
    b = rng.normal(0, 0.1, b.shape).astype(np.float32)           # non-zero biases
    bo = rng.normal(0, 0.1, bo.shape).astype(np.float32)
    x, r = si.rnn_sequences(cfg)
    return cfg, (Wh, Wx, b, Wo, bo), x, r


def oracle_all(params, x, r):
    Wh, Wx, b, Wo, bo = params
    outs = [ro.forward(Wh, Wx, b, Wo, bo, x[i], r[i]) for i in range(x.shape[0])]
    return {k: np.stack([o[k] for o in outs]) for k in ("h", "d", "l")} | {"loss": np.array([o["loss"] for o in outs])}


def dev(*arrays):
    return [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda() for a in arrays]


CASES = [("rnn_small", {}), ("rnn_small", {"T": 1, "H": 4}), ("rnn_small", {"T": 128, "H": 128, "batch": 2}),
         ("rnn_small", {"T": 37, "H": 20, "d_in": 3, "d_out": 2, "batch": 5}), ("rnn_100", {}),
         ("rnn_100", {"batch": 6, "T": 100, "H": 124})]


@pytest.mark.parametrize("name,changes", CASES, ids=[f"{n}-{'-'.join(f'{k}{v}' for k, v in c.items()) or 'base'}" for n, c in CASES])
def test_forward_backward_and_jacobi_match_the_oracle(name, changes):
    import paper_2002_03629_b200.rnn as rnn
    cfg, params, x, r = case(name, **changes)
    Wh = params[0]
    want = oracle_all(params, x, r)
    dW = dev(*params)
    dx, dr = dev(x, r)
    h, d, l, loss = rnn.rnn_forward(*dW, dx, dr)
    close(h, want["h"], "h"); close(d, want["d"], "d"); close(l, want["l"], "l"); close(loss, want["loss"], "loss")
    # backward from the ORACLE's l and d (rounded to fp32), so that each step is compared on identical inputs
    l32, d32 = dev(want["l"], want["d"])
    lq, dq = l32.cpu().double().numpy(), d32.cpu().double().numpy()
    exact = np.stack([ro.backprop_exact(Wh, lq[i], dq[i]) for i in range(cfg.batch)])
    close(rnn.rnn_bptt_sequential(dW[0], l32, d32), exact, "sequential")
    for n in sorted({0, 1, 2, 5, min(17, cfg.T), cfg.T, cfg.T + 3}):
        wantn = np.stack([ro.backprop_jacobi(Wh, lq[i], dq[i], n) for i in range(cfg.batch)])
        close(rnn.rnn_bptt_jacobi(dW[0], l32, d32, n), wantn, f"jacobi_{n}")
    # from a given start iterate
    rng = np.random.default_rng(9)
    s0 = rng.normal(size=exact.shape).astype(np.float32)
    (s0d,) = dev(s0)
    for n in (0, 1, 3):
        wantn = np.stack([ro.backprop_jacobi(Wh, lq[i], dq[i], n, s0[i].astype(np.float64)) for i in range(cfg.batch)])
        close(rnn.rnn_bptt_jacobi(dW[0], l32, d32, n, s0=s0d), wantn, f"jacobi_{n} from s0")
    # parameter gradients from the oracle's exact states
    (s32,) = dev(exact)
    h32, = dev(want["h"])
    sq, hq = s32.cpu().double().numpy(), h32.cpu().double().numpy()
    dWh, dWx, db = rnn.rnn_param_grads(s32, d32, h32, dx)
    wg = [ro.param_grads(sq[i], dq[i], hq[i], x[i]) for i in range(cfg.batch)]
    close(dWh, np.stack([w[0] for w in wg]), "dWh")
    close(dWx, np.stack([w[1] for w in wg]), "dWx")
    close(db, np.stack([w[2] for w in wg]), "db")


def test_jacobi_has_the_finite_convergence_property_on_the_device():
    """Proposition 1 on the device's own arithmetic: after n iterations the last n states equal those of
    n + 1 iterations bit for bit, and T iterations reproduce themselves."""
    import paper_2002_03629_b200.rnn as rnn
    cfg, params, x, r = case("rnn_100")
    dW = dev(*params)
    dx, dr = dev(x, r)
    h, d, l, loss = rnn.rnn_forward(*dW, dx, dr)
    T = cfg.T
    prev = rnn.rnn_bptt_jacobi(dW[0], l, d, 1)
    for n in (2, 3, 10, 50):
        a = rnn.rnn_bptt_jacobi(dW[0], l, d, n)
        b = rnn.rnn_bptt_jacobi(dW[0], l, d, n + 1)
        assert torch.equal(a[:, T - n:], b[:, T - n:])
    full = rnn.rnn_bptt_jacobi(dW[0], l, d, T)
    assert torch.equal(full, rnn.rnn_bptt_jacobi(dW[0], l, d, T + 5))
    assert torch.equal(prev, l)                                      # one sweep from zero is the direct gradient
    # same run twice: reproducible
    assert torch.equal(full, rnn.rnn_bptt_jacobi(dW[0], l, d, T))
    seq = rnn.rnn_bptt_sequential(dW[0], l, d)
    assert (full - seq).abs().max().item() <= 1e-5 * seq.abs().max().item()


def test_full_batch_on_sampled_sequences():
    """The benchmark's batch (one sequence per thread block, several per SM in turn), checked on sampled
    sequences."""
    import paper_2002_03629_b200.rnn as rnn
    cfg, params, x, r = case("rnn_100_batch")
    Wh = params[0]
    dW = dev(*params)
    dx, dr = dev(x, r)
    h, d, l, loss = rnn.rnn_forward(*dW, dx, dr)
    s10 = rnn.rnn_bptt_jacobi(dW[0], l, d, 10)
    sx = rnn.rnn_bptt_sequential(dW[0], l, d)
    for i in (0, 1, 147, 148, 300, cfg.batch - 1):
        f = ro.forward(*params, x[i], r[i])
        close(h[i], f["h"], f"h[{i}]")
        close(sx[i], ro.backprop_exact(Wh, f["l"], f["d"]), f"exact[{i}]")
        close(s10[i], ro.backprop_jacobi(Wh, f["l"], f["d"], 10), f"jacobi_10[{i}]")


def test_argument_errors_launch_nothing():
    import paper_2002_03629_b200 as pkg
    import paper_2002_03629_b200.rnn as rnn
    lib = rnn._lib()
    t = torch.zeros(4 * 8 * 8, dtype=torch.float32, device="cuda")
    p = C.c_void_p(t.data_ptr())
    assert lib.rnn_bptt_jacobi(p, p, p, 1, 8, 6, 1, None, p, None) == rnn.RNN_ERR_INVALID      # H not a multiple of 4
    assert lib.rnn_bptt_jacobi(p, p, p, 1, 129, 8, 1, None, p, None) == rnn.RNN_ERR_INVALID    # T too large
    assert lib.rnn_bptt_jacobi(p, p, p, 1, 8, 8, -1, None, p, None) == rnn.RNN_ERR_INVALID
    assert lib.rnn_bptt_jacobi(None, p, p, 1, 8, 8, 1, None, p, None) == rnn.RNN_ERR_INVALID
    assert lib.rnn_bptt_sequential(p, p, p, 0, 8, 8, p, None) == rnn.RNN_ERR_INVALID
    assert lib.rnn_forward(p, p, p, p, p, p, p, 1, 8, 8, 17, 1, p, p, p, p, None) == rnn.RNN_ERR_INVALID
    assert lib.rnn_param_grads(p, p, p, p, 1, 8, 8, 0, p, p, p, None) == rnn.RNN_ERR_INVALID
    l3 = t.view(4, 8, 8)
    with pytest.raises(pkg.JsError):
        rnn.rnn_bptt_sequential(torch.zeros(8, 8), l3, l3)                                      # weights on the host
