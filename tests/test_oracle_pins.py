"""Pins of the CPU oracle against facts it does not compute itself.

Each test names what fixes the expected value: a hand computation, an
independent numpy/torch recomputation from the stated mask rule, brute-force
enumeration, a proposition of Section 3 or a worked example of Section 4.1.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from oracle import Oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ helpers
def bf16(a):
    """Round-to-nearest-even to bf16 by a library routine (torch), back to float32."""
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def made_masks(D, C, H):
    """Masks from the degree rule, written independently of the oracle."""
    deg = [np.arange(1, D + 1)]
    for h in H:
        deg.append(1 + (np.arange(h) * (D - 1)) // h)
    deg.append(np.repeat(np.arange(1, D + 1), C))
    masks = []
    for l in range(len(H) + 1):
        if l == len(H):
            masks.append(deg[l + 1][:, None] > deg[l][None, :])
        else:
            masks.append(deg[l + 1][:, None] >= deg[l][None, :])
    return masks


def numpy_made_logits(cfg, W, b, lut, x):
    masks = made_masks(cfg.D, cfg.C, cfg.H)
    rnd = bf16 if cfg.prec == si.PREC_BF16 else (lambda v: np.asarray(v, dtype=np.float32))
    a = rnd(lut)[x].astype(np.float64)
    for l in range(len(cfg.H)):
        pre = (rnd(W[l] * masks[l]).astype(np.float64) @ a + b[l]).astype(np.float32).astype(np.float64)
        if cfg.act == si.ACT_RELU:
            act = np.maximum(pre, 0)
        else:
            act = 0.5 * pre * (1 + np.tanh(np.sqrt(2 / np.pi) * (pre + 0.044715 * pre ** 3)))
        a = rnd(act.astype(np.float32)).astype(np.float64)
    z = rnd(W[-1] * masks[-1]).astype(np.float64) @ a + b[-1]
    return z.astype(np.float32).reshape(cfg.D, cfg.C)


def small_made(prec=si.PREC_F32, D=12, C=1, H=(24, 20), act=si.ACT_RELU, nk=si.NOISE_LOGISTIC, index=11,
               w_var_scale=8.0):
    cfg = si.MadeConfig("t", index, D=D, C=C, H=H, act=act, prec=prec, batch=6, noise_kind=nk,
                        w_var_scale=w_var_scale, b_var=0.1)
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    return cfg, W, b, lut, oracle.from_config(cfg, W, b, lut)


def small_conv(index=21, height=4, width=5, ch=12, layers=3, C=4):
    cfg = si.ConvConfig("c", index, height=height, width=width, in_ch=3, ch=ch, layers=layers, C=C, batch=3)
    W, b = si.conv_weights(cfg)
    W = [w * 3.0 for w in W]           # stronger coupling so that iterations are not trivial
    lut = si.conv_lut(cfg)
    return cfg, W, b, lut, oracle.from_config(cfg, W, b, lut)


# --------------------------------------------------------- forward pass pins
def test_hand_computed_network():
    rows = np.loadtxt(os.path.join(GOLD, "made3_hand.txt"))
    W = [np.ones((3, 3), np.float32), np.array([[1, 1, 1], [2, 3, 5], [7, 11, 13]], np.float32)]
    b = [np.array([0.5, -0.5, -1], np.float32), np.array([0.25, -1, -2], np.float32)]
    m = Oracle.made(3, 1, [3], si.ACT_RELU, si.PREC_F32, W, b, np.array([0, 1], np.float32))
    for r in rows:
        z = m.forward_logits(r[:3].astype(np.uint8))[:, 0]
        np.testing.assert_array_equal(z, r[3:].astype(np.float32))


@pytest.mark.parametrize("prec", [si.PREC_F32, si.PREC_BF16])
@pytest.mark.parametrize("act,C", [(si.ACT_RELU, 1), (si.ACT_GELU_TANH, 5)])
def test_forward_matches_numpy_recomputation(prec, act, C):
    nk = si.NOISE_GUMBEL if C > 1 else si.NOISE_LOGISTIC
    cfg, W, b, lut, m = small_made(prec=prec, C=C, act=act, nk=nk)
    rng = np.random.default_rng(0)
    for _ in range(5):
        x = rng.integers(0, cfg.n_symbols, cfg.D, dtype=np.uint8)
        z = m.forward_logits(x)
        ref = numpy_made_logits(cfg, W, b, lut, x)
        # GELU goes through tanh of two libraries; bf16 rounding may flip one unit by an ulp
        tol = 0 if (act == si.ACT_RELU) else (2e-2 if prec == si.PREC_BF16 else 1e-5)
        np.testing.assert_allclose(z, ref, rtol=tol, atol=tol)


def test_default_degrees_and_masked_weights():
    cfg, W, b, lut, m = small_made()
    masks = made_masks(cfg.D, cfg.C, cfg.H)
    widths = [cfg.D, *cfg.H, cfg.D * cfg.C]
    for l in range(len(W)):
        got = m.masked_weight(l, (widths[l + 1], widths[l]))
        np.testing.assert_array_equal(got, W[l] * masks[l])
    np.testing.assert_array_equal(m.degrees(1), 1 + (np.arange(cfg.H[0]) * (cfg.D - 1)) // cfg.H[0])


@pytest.mark.parametrize("maker", [small_made, small_conv])
def test_autoregressive_property(maker):
    """Logits of position t ignore positions >= t and do react to some position < t."""
    cfg, W, b, lut, m = maker()
    n_sym = 2 if cfg.C == 1 else cfg.C
    rng = np.random.default_rng(1)
    x = rng.integers(0, n_sym, m.T, dtype=np.uint8)
    z = m.forward_logits(x)
    reacts = np.zeros(m.T, bool)
    for t in range(m.T):
        y = x.copy()
        y[t] = (y[t] + 1) % n_sym
        zy = m.forward_logits(y)
        np.testing.assert_array_equal(zy[: t + 1], z[: t + 1])     # bit-unchanged
        if t + 1 < m.T:
            reacts[t + 1] = np.any(zy[t + 1] != z[t + 1])
    # the direct predecessor matters for most positions (guards against over-masking)
    assert reacts[1:].mean() > 0.5


def test_conv_forward_matches_torch_conv2d():
    cfg, W, b, lut, m = small_conv()
    ch, n_in = cfg.ch, cfg.in_ch
    grp = (n_in * np.arange(ch)) // ch
    x = np.random.default_rng(2).integers(0, cfg.C, m.T, dtype=np.uint8)
    a = torch.from_numpy(bf16(lut)[x].reshape(cfg.height, cfg.width, n_in)).permute(2, 0, 1)[None].double()
    for l in range(cfg.layers):
        gi = np.arange(n_in) if l == 0 else grp
        mask = np.zeros((ch, 3, 3, len(gi)), bool)
        mask[:, 0, :, :] = True
        mask[:, 1, 0, :] = True
        mask[:, 1, 1, :] = (gi[None, :] < grp[:, None]) if l == 0 else (gi[None, :] <= grp[:, None])
        wt = torch.from_numpy(bf16(W[l] * mask)).permute(0, 3, 1, 2).double()      # [co, ci, ky, kx]
        pre = torch.nn.functional.conv2d(a, wt, torch.from_numpy(b[l]).double(), padding=1)
        a = torch.from_numpy(bf16(torch.relu(pre.float()).numpy())).double()
    hmask = grp[None, :] <= (np.arange(n_in * cfg.C) // cfg.C)[:, None]
    wh = torch.from_numpy(bf16(W[-1] * hmask)).double()
    z = torch.einsum("oc,chw->hwo", wh, a[0]) + torch.from_numpy(b[-1]).double()
    ref = z.float().numpy().reshape(m.T, cfg.C)
    got = m.forward_logits(x)
    # summation order differs (conv2d vs index order): allow float rounding of the last step
    np.testing.assert_allclose(got, ref, rtol=2e-2, atol=2e-3)
    assert np.mean(got == ref) > 0.5


# ------------------------------------------------------------- brute force
def test_brute_force_unique_fixed_point_and_normalisation():
    """All 2^16 outcomes of the tiny model: exactly one is a fixed point of the
    parallel update for given noise, every solver returns it, and the chain-rule
    probabilities sum to one."""
    cfg = si.CONFIGS["made_tiny"]
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    m = oracle.from_config(cfg, W, b, lut)
    noise = si.draw_noise(cfg)
    D = cfg.D
    allx = ((np.arange(2 ** D)[:, None] >> np.arange(D)[None, :]) & 1).astype(np.uint8)
    Z = np.stack([m.forward_logits(v)[:, 0] for v in allx]).astype(np.float64)      # [65536, D]
    P1 = 1.0 / (1.0 + np.exp(-Z))
    prob = np.prod(np.where(allx == 1, P1, 1.0 - P1), axis=1)
    assert abs(prob.sum() - 1.0) < 1e-12
    for s in range(cfg.batch):
        u = noise[s]
        G = (u[None, :].astype(np.float64) < P1).astype(np.uint8)       # parallel update of every outcome
        fixed = np.nonzero(np.all(G == allx, axis=1))[0]
        assert len(fixed) == 1
        xstar = allx[fixed[0]]
        nk = cfg.noise_kind
        np.testing.assert_array_equal(m.sequential(u, nk), xstar)
        np.testing.assert_array_equal(m.sequential(u, nk, literal=True), xstar)
        np.testing.assert_array_equal(m.gauss_seidel(u, nk), xstar)
        np.testing.assert_array_equal(m.jacobi(u, nk)[0], xstar)
        np.testing.assert_array_equal(m.gs_jacobi(u, nk, 4)[0], xstar)
        np.testing.assert_array_equal(m.jacobi_gs(u, nk, 4)[0], xstar)


# ------------------------------------------------------------ sampler laws
@pytest.mark.parametrize("nk", [si.NOISE_UNIFORM_ICDF, si.NOISE_LOGISTIC, si.NOISE_GUMBEL])
def test_sampler_law_chi_square(nk):
    """Over many noise draws the sequential sampler's outcome frequencies follow
    the model's chain-rule probabilities."""
    C = 3 if nk == si.NOISE_GUMBEL else 1
    D = 3 if C > 1 else 4
    cfg = si.MadeConfig("law", 31 + nk, D=D, C=C, H=(8,), act=si.ACT_RELU, prec=si.PREC_F32, batch=1,
                        noise_kind=nk, w_var_scale=6.0, b_var=0.3)
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    m = oracle.from_config(cfg, W, b, lut)
    n_sym = cfg.n_symbols
    outcomes = list(itertools.product(range(n_sym), repeat=D))
    p = []
    for o in outcomes:
        z = m.forward_logits(np.array(o, np.uint8)).astype(np.float64)
        if C == 1:
            p1 = 1 / (1 + np.exp(-z[:, 0]))
            p.append(np.prod(np.where(np.array(o) == 1, p1, 1 - p1)))
        else:
            sm = np.exp(z - z.max(1, keepdims=True))
            sm /= sm.sum(1, keepdims=True)
            p.append(np.prod(sm[np.arange(D), o]))
    p = np.array(p)
    assert abs(p.sum() - 1) < 1e-9
    N = 40000
    noise = si.draw_noise(cfg, batch=N)
    counts = np.zeros(len(outcomes))
    index = {o: i for i, o in enumerate(outcomes)}
    for i in range(N):
        counts[index[tuple(int(v) for v in m.sequential(noise[i], nk))]] += 1
    expected = p * N
    keep = expected > 5
    chi2 = np.sum((counts[keep] - expected[keep]) ** 2 / expected[keep])
    dof = keep.sum() - 1
    # mean dof, variance 2*dof: six standard deviations is a safe yet sharp bound
    assert chi2 < dof + 6 * np.sqrt(2 * dof), (chi2, dof)
