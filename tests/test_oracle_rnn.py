"""Pins of the recurrent-network oracle (oracle/rnn_oracle.py) against what the mathematics fixes:
finite differences of the loss, an automatic-differentiation library, closed forms, and the
finite-convergence property of Jacobi iterations on a triangular system (Proposition 1).  A last
test plants mistakes in a copy of the oracle's source and checks that the pins notice each one."""
import os
import types

import numpy as np
import pytest

import synth_inputs as si
from oracle import rnn_oracle as ro

SRC = os.path.join(os.path.dirname(os.path.abspath(ro.__file__)), "rnn_oracle.py")


def setup(name="rnn_small", b=0):
    cfg = si.RNN_CONFIGS[name]
    Wh, Wx, bias, Wo, bo = si.rnn_weights(cfg)
    x, r = si.rnn_sequences(cfg)
    # non-zero biases so that a dropped bias term would show
    rng = np.random.default_rng(5)
    bias = rng.normal(0, 0.1, bias.shape)
    bo = rng.normal(0, 0.1, bo.shape)
    return cfg, (Wh.astype(np.float64), Wx.astype(np.float64), bias, Wo.astype(np.float64), bo), x[b].astype(np.float64), r[b].astype(np.float64)


# ---- the checks, each taking the module under test (the mutant test re-runs them on broken copies)
def check_param_grads_against_finite_differences(m):
    cfg, (Wh, Wx, b, Wo, bo), x, r = setup()
    f = m.forward(Wh, Wx, b, Wo, bo, x, r)
    s = m.backprop_exact(Wh, f["l"], f["d"])
    dWh, dWx, db = m.param_grads(s, f["d"], f["h"], x)
    eps = 1e-6
    rng = np.random.default_rng(0)

    def loss(Wh_, Wx_, b_):
        return m.forward(Wh_, Wx_, b_, Wo, bo, x, r)["loss"]

    for _ in range(12):
        j, i = rng.integers(0, cfg.H, 2)
        P = np.zeros_like(Wh); P[j, i] = eps
        fd = (loss(Wh + P, Wx, b) - loss(Wh - P, Wx, b)) / (2 * eps)
        assert abs(fd - dWh[j, i]) < 1e-7 * max(1.0, abs(fd)), (j, i, fd, dWh[j, i])
    for j in range(0, cfg.H, 5):
        P = np.zeros_like(Wx); P[j, 0] = eps
        fd = (loss(Wh, Wx + P, b) - loss(Wh, Wx - P, b)) / (2 * eps)
        assert abs(fd - dWx[j, 0]) < 1e-7 * max(1.0, abs(fd))
        P = np.zeros_like(b); P[j] = eps
        fd = (loss(Wh, Wx, b + P) - loss(Wh, Wx, b - P)) / (2 * eps)
        assert abs(fd - db[j]) < 1e-7 * max(1.0, abs(fd))


def check_state_grads_against_autograd(m):
    torch = pytest.importorskip("torch")
    cfg, (Wh, Wx, b, Wo, bo), x, r = setup()
    tWh, tWx, tb, tWo, tbo, tx, tr = (torch.tensor(v, dtype=torch.float64) for v in (Wh, Wx, b, Wo, bo, x, r))
    hs = []
    tWh.requires_grad_(True)
    prev = torch.zeros(cfg.H, dtype=torch.float64)
    loss = torch.zeros((), dtype=torch.float64)
    for t in range(cfg.T):
        h = torch.nn.functional.softplus(tWh @ prev + tWx @ tx[t] + tb)
        h.retain_grad()
        hs.append(h)
        loss = loss + 0.5 * torch.sum((tWo @ h + tbo - tr[t]) ** 2)
        prev = h
    loss.backward()
    want = np.stack([h.grad.numpy() for h in hs])
    f = m.forward(Wh, Wx, b, Wo, bo, x, r)
    assert abs(f["loss"] - loss.item()) < 1e-10 * max(1.0, loss.item())
    got = m.backprop_exact(Wh, f["l"], f["d"])
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)


def check_scalar_closed_form(m):
    # H = 1, constant derivative c: s_t = sum_j (w c)^j l_{t+j}
    T, w, c = 9, 0.7, 0.6
    l = np.arange(1.0, T + 1.0).reshape(T, 1)
    d = np.full((T, 1), c)
    want = np.array([[sum((w * c) ** j * l[t + j, 0] for j in range(T - t))] for t in range(T)])
    np.testing.assert_allclose(m.backprop_exact(np.array([[w]]), l, d), want, rtol=1e-13)
    # a non-symmetric 2x2 case by hand: one step back from the last state
    Wh = np.array([[0.5, -1.0], [2.0, 0.25]])
    l2 = np.array([[1.0, 2.0], [3.0, -1.0]])
    d2 = np.array([[0.1, 0.2], [0.5, 0.25]])
    g = d2[1] * l2[1]                                    # (1.5, -0.25)
    want0 = l2[0] + np.array([Wh[0, 0] * g[0] + Wh[1, 0] * g[1], Wh[0, 1] * g[0] + Wh[1, 1] * g[1]])
    got = m.backprop_exact(Wh, l2, d2)
    np.testing.assert_allclose(got[1], l2[1])
    np.testing.assert_allclose(got[0], want0)
    np.testing.assert_allclose(m.jacobi_step(Wh, l2, d2, got), got)


def check_jacobi_properties(m):
    cfg, (Wh, Wx, b, Wo, bo), x, r = setup()
    f = m.forward(Wh, Wx, b, Wo, bo, x, r)
    l, d, T = f["l"], f["d"], cfg.T
    exact = m.backprop_exact(Wh, l, d)
    np.testing.assert_allclose(m.backprop_jacobi(Wh, l, d, 1), l)              # one sweep from zero
    for n in (1, 2, 3, 7, T - 1):
        sn = m.backprop_jacobi(Wh, l, d, n)
        # Proposition 1 on the reversed chain: after n sweeps the last n states are final
        np.testing.assert_allclose(sn[T - n:], exact[T - n:], rtol=1e-13, atol=1e-15)
        assert np.abs(sn[:T - n] - exact[:T - n]).max() > 1e-9
    rng = np.random.default_rng(1)
    s0 = rng.normal(size=l.shape)
    np.testing.assert_allclose(m.backprop_jacobi(Wh, l, d, T, s0), exact, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(m.jacobi_step(Wh, l, d, exact), exact, rtol=1e-13, atol=1e-15)
    # truncation = back-propagation through n - 1 steps: an independent unrolling of the sum
    n = 4
    want = np.zeros_like(l)
    for t in range(T):
        term = None
        for j in range(min(n, T - t)):
            term = l[t + j].copy() if j == 0 else term
            if j > 0:
                v = l[t + j].copy()
                for q in range(t + j, t, -1):
                    v = Wh.T @ (d[q] * v)
                want[t] += v
            else:
                want[t] += term
    np.testing.assert_allclose(m.backprop_jacobi(Wh, l, d, n), want, rtol=1e-12, atol=1e-14)


CHECKS = [check_param_grads_against_finite_differences, check_state_grads_against_autograd,
          check_scalar_closed_form, check_jacobi_properties]


@pytest.mark.parametrize("check", CHECKS, ids=lambda c: c.__name__)
def test_pins(check):
    check(ro)


def test_convergence_is_geometric_on_the_paper_sized_model():
    cfg = si.RNN_CONFIGS["rnn_100"]
    Wh, Wx, b, Wo, bo = si.rnn_weights(cfg)
    x, r = si.rnn_sequences(cfg)
    f = ro.forward(Wh, Wx, b, Wo, bo, x[0], r[0])
    exact = ro.backprop_exact(Wh, f["l"], f["d"])
    errs = [np.linalg.norm(ro.backprop_jacobi(Wh, f["l"], f["d"], n) - exact) for n in (5, 10, 20, 100)]
    assert errs[0] > errs[1] > errs[2] > errs[3] == 0.0
    assert errs[2] < 1e-3 * errs[0]


MUTANTS = [
    ("transposed recurrence in the back-substitution", "s[t] = l[t] + Wh.T @ (d[t + 1] * s[t + 1])", "s[t] = l[t] + Wh @ (d[t + 1] * s[t + 1])"),
    ("derivative taken at the wrong step", "s[t] = l[t] + Wh.T @ (d[t + 1] * s[t + 1])", "s[t] = l[t] + Wh.T @ (d[t] * s[t + 1])"),
    ("derivative dropped", "s[t] = l[t] + Wh.T @ (d[t + 1] * s[t + 1])", "s[t] = l[t] + Wh.T @ (s[t + 1])"),
    ("direct term dropped", "s[t] = l[t] + Wh.T @ (d[t + 1] * s[t + 1])", "s[t] = Wh.T @ (d[t + 1] * s[t + 1])"),
    ("Jacobi sweep reads the new iterate", "s[t] = l[t] + (Wh.T @ (d[t + 1] * s_prev[t + 1]) if t + 1 < T else 0.0)",
     "t = T - 1 - t; s[t] = l[t] + (Wh.T @ (d[t + 1] * s[t + 1]) if t + 1 < T else 0.0)"),
    ("Jacobi sweep reads the same step", "s[t] = l[t] + (Wh.T @ (d[t + 1] * s_prev[t + 1]) if t + 1 < T else 0.0)",
     "s[t] = l[t] + (Wh.T @ (d[t] * s_prev[t]) if t + 1 < T else 0.0)"),
    ("Jacobi sweep transposed", "s[t] = l[t] + (Wh.T @ (d[t + 1] * s_prev[t + 1]) if t + 1 < T else 0.0)",
     "s[t] = l[t] + (Wh @ (d[t + 1] * s_prev[t + 1]) if t + 1 < T else 0.0)"),
    ("weight gradient pairs the same step", "dWh += np.outer(g[t], h[t - 1])", "dWh += np.outer(g[t], h[t])"),
    ("weight gradient transposed", "dWh += np.outer(g[t], h[t - 1])", "dWh += np.outer(h[t - 1], g[t])"),
    ("gradient without the activation derivative", "g = d * s", "g = s"),
    ("direct gradient without the output weights", '"l": e @ Wo,', '"l": e @ np.ones_like(Wo),'),
    ("derivative of the wrong activation", '"d": sigmoid(a)}', '"d": softplus(a)}'),
    ("bias dropped in the forward pass", "a[t] = Wh @ prev + Wx @ x[t] + b", "a[t] = Wh @ prev + Wx @ x[t]"),
    ("recurrence uses the input state twice", "prev = h[t]", "prev = h[max(t - 1, 0)]"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_notice_planted_mistakes(name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, name
    mod = types.ModuleType("rnn_oracle_mutant")
    exec(compile(src.replace(old, new), "rnn_oracle_mutant.py", "exec"), mod.__dict__)
    failed = 0
    for check in CHECKS:
        try:
            check(mod)
        except AssertionError:
            failed += 1
    assert failed > 0, f"no pin noticed: {name}"
