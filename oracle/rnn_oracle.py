"""CPU oracle of the recurrent-network workload: back-propagation through time as a triangular
system solved by truncated Jacobi iterations (arXiv 2002.03629, Section 5.1 and the appendix
sections "Backpropagation" and "Extra Experimental Details: RNN").

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the benchmark's CPU leg.
Plain numpy in float64, one sequence at a time, the recursions written out step by step.

Model (one hidden layer, SoftPlus, as in the paper's experiment):

    a_t = W_h h_{t-1} + W_x x_t + b,   h_t = softplus(a_t),   h_0 = 0,          t = 1..T
    y_t = W_o h_t + b_o,               loss = 1/2 sum_t |y_t - r_t|^2

so the loss touches every time step.  With  l_t = W_o^T (y_t - r_t)  (the direct part of
d loss / d h_t) and  d_t = softplus'(a_t) = sigmoid(a_t),  the states of the backward pass are
s_t = d loss / d h_t:

    s_T = l_T,      s_t = l_t + W_h^T (d_{t+1} * s_{t+1})                         (back-substitution)

which is the feedforward computation of Eq. 1 with the states taken from t = T downwards.  One
Jacobi iteration (Algorithm 1) applies the right-hand side to every t at once from the previous
iterate; "Jacobi_n" is the iterate after n of them, started from zero.
"""
from __future__ import annotations

import numpy as np


def softplus(a: np.ndarray) -> np.ndarray:
    return np.logaddexp(0.0, a)


def sigmoid(a: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-a))


def forward(Wh, Wx, b, Wo, bo, x, r):
    """Forward pass of one sequence.  x [T, d_in], r [T, d_out].  Returns a dict with the hidden
    states h [T, H] (h[t] is h_{t+1} of the text), pre-activations a, outputs y, the loss, the direct
    gradients l [T, H] and the activation derivatives d [T, H]."""
    Wh, Wx, b, Wo, bo, x, r = (np.asarray(v, dtype=np.float64) for v in (Wh, Wx, b, Wo, bo, x, r))
    T, H = x.shape[0], Wh.shape[0]
    h = np.zeros((T, H))
    a = np.zeros((T, H))
    prev = np.zeros(H)
    for t in range(T):
        a[t] = Wh @ prev + Wx @ x[t] + b
        h[t] = softplus(a[t])
        prev = h[t]
    y = h @ Wo.T + bo
    e = y - r
    return {"h": h, "a": a, "y": y, "loss": 0.5 * float(np.sum(e * e)), "l": e @ Wo, "d": sigmoid(a)}


def backprop_exact(Wh, l, d):
    """s_t = d loss / d h_t for every t by back-substitution, last step first."""
    Wh, l, d = (np.asarray(v, dtype=np.float64) for v in (Wh, l, d))
    T = l.shape[0]
    s = np.zeros_like(l)
    s[T - 1] = l[T - 1]
    for t in range(T - 2, -1, -1):
        s[t] = l[t] + Wh.T @ (d[t + 1] * s[t + 1])
    return s


def jacobi_step(Wh, l, d, s_prev):
    """One Jacobi iteration (Algorithm 1): every state from the previous iterate, all t at once."""
    Wh, l, d, s_prev = (np.asarray(v, dtype=np.float64) for v in (Wh, l, d, s_prev))
    T = l.shape[0]
    s = np.empty_like(l)
    for t in range(T):
        s[t] = l[t] + (Wh.T @ (d[t + 1] * s_prev[t + 1]) if t + 1 < T else 0.0)
    return s


def backprop_jacobi(Wh, l, d, n, s0=None):
    """Jacobi_n: the iterate after n Jacobi iterations from s0 (zeros if not given)."""
    s = np.zeros_like(np.asarray(l, dtype=np.float64)) if s0 is None else np.asarray(s0, dtype=np.float64)
    for _ in range(n):
        s = jacobi_step(Wh, l, d, s)
    return s


def param_grads(s, d, h, x):
    """Gradients of the loss with respect to W_h, W_x and b from the state gradients s:
    with g_t = d_t * s_t (= d loss / d a_t),  dW_h = sum_t g_t h_{t-1}^T,  dW_x = sum_t g_t x_t^T,
    db = sum_t g_t."""
    s, d, h, x = (np.asarray(v, dtype=np.float64) for v in (s, d, h, x))
    T, H = s.shape
    g = d * s
    dWh = np.zeros((H, H))
    dWx = np.zeros((H, x.shape[1]))
    db = np.zeros(H)
    for t in range(T):
        if t > 0:
            dWh += np.outer(g[t], h[t - 1])
        dWx += np.outer(g[t], x[t])
        db += g[t]
    return dWh, dWx, db
