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


def made_masks(D, C, H, hidden_deg=None):
    """Masks from the degree rule, written independently of the oracle."""
    deg = [np.arange(1, D + 1)]
    for i, h in enumerate(H):
        deg.append(1 + (np.arange(h) * (D - 1)) // h if hidden_deg is None else np.asarray(hidden_deg[i]))
    deg.append(np.repeat(np.arange(1, D + 1), C))
    masks = []
    for l in range(len(H) + 1):
        if l == len(H):
            masks.append(deg[l + 1][:, None] > deg[l][None, :])
        else:
            masks.append(deg[l + 1][:, None] >= deg[l][None, :])
    return masks


def numpy_made_logits(cfg, W, b, lut, x, hidden_deg=None):
    masks = made_masks(cfg.D, cfg.C, cfg.H, hidden_deg)
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
@pytest.mark.parametrize("nk", [si.NOISE_UNIFORM_ICDF, si.NOISE_LOGISTIC, si.NOISE_GUMBEL, si.NOISE_UNIFORM_CAT])
def test_sampler_law_chi_square(nk):
    """Over many noise draws the sequential sampler's outcome frequencies follow
    the model's chain-rule probabilities."""
    C = 3 if nk in (si.NOISE_GUMBEL, si.NOISE_UNIFORM_CAT) else 1
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


# ------------------------------------------ custom (unsorted) hidden degrees
def shuffled_degrees(cfg, seed=5):
    """Degrees 1..D-1 in random order for every hidden layer (every degree present at least once
    when the layer is wide enough)."""
    rng = np.random.default_rng(seed)
    out = []
    for h in cfg.H:
        d = 1 + (np.arange(h) * (cfg.D - 1)) // h
        out.append(rng.permutation(d).astype(np.int32))
    return out


@pytest.mark.parametrize("prec", [si.PREC_F32, si.PREC_BF16])
def test_custom_hidden_degrees(prec):
    """Caller-given degrees replace the default rule: the masked weights follow them, the forward pass
    equals a numpy recomputation with those degrees, the logits of position t still ignore positions
    >= t, and every solver still returns the feedforward sample."""
    cfg = si.MadeConfig("deg", 13, D=12, C=1, H=(24, 20), act=si.ACT_RELU, prec=prec, batch=4,
                        noise_kind=si.NOISE_LOGISTIC, w_var_scale=8.0, b_var=0.1)
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    hd = shuffled_degrees(cfg)
    m = Oracle.made(cfg.D, cfg.C, list(cfg.H), cfg.act, cfg.prec, W, b, lut, hidden_deg=hd)
    np.testing.assert_array_equal(m.degrees(1), hd[0])
    np.testing.assert_array_equal(m.degrees(2), hd[1])
    masks = made_masks(cfg.D, cfg.C, cfg.H, hd)
    widths = [cfg.D, *cfg.H, cfg.D]
    rnd = bf16 if prec == si.PREC_BF16 else (lambda v: v)
    for l in range(3):
        np.testing.assert_array_equal(m.masked_weight(l, (widths[l + 1], widths[l])), rnd(W[l] * masks[l]))
    rng = np.random.default_rng(3)
    x = rng.integers(0, 2, cfg.D, dtype=np.uint8)
    z = m.forward_logits(x)
    np.testing.assert_array_equal(z, numpy_made_logits(cfg, W, b, lut, x, hd))
    for t in range(cfg.D):
        y = x.copy()
        y[t] ^= 1
        np.testing.assert_array_equal(m.forward_logits(y)[: t + 1], z[: t + 1])
    # the shuffled masks differ from the default ones (otherwise this test would pin nothing)
    assert any(np.any(a != b2) for a, b2 in zip(masks, made_masks(cfg.D, cfg.C, cfg.H)))
    noise = si.draw_noise(cfg)
    for s_ in range(cfg.batch):
        ref = m.sequential(noise[s_], cfg.noise_kind, literal=True)
        np.testing.assert_array_equal(m.sequential(noise[s_], cfg.noise_kind), ref)
        np.testing.assert_array_equal(m.jacobi(noise[s_], cfg.noise_kind)[0], ref)
        np.testing.assert_array_equal(m.jacobi_gs(noise[s_], cfg.noise_kind, 4)[0], ref)
        np.testing.assert_array_equal(m.gs_jacobi(noise[s_], cfg.noise_kind, 4)[0], ref)


# ----------------------------------------------------- decision margins
def _margin_case(nk):
    C = 1 if nk in (si.NOISE_UNIFORM_ICDF, si.NOISE_LOGISTIC) else 6
    cfg = si.MadeConfig("mg", 41 + nk, D=10, C=C, H=(16,), act=si.ACT_RELU, prec=si.PREC_F32, batch=8,
                        noise_kind=nk, w_var_scale=6.0, b_var=0.3)
    W, b = si.made_weights(cfg)
    m = oracle.from_config(cfg, W, b, si.made_lut(cfg))
    return cfg, m, si.draw_noise(cfg)


def test_margin_binary_kinds_against_numpy():
    """|z + eps| for logistic noise, |z - logit(u)| for a uniform number, recomputed from the logits."""
    for nk in (si.NOISE_LOGISTIC, si.NOISE_UNIFORM_ICDF):
        cfg, m, noise = _margin_case(nk)
        rng = np.random.default_rng(7)
        for s_ in range(cfg.batch):
            x = rng.integers(0, 2, cfg.D, dtype=np.uint8)
            z = m.forward_logits(x)[:, 0]
            got = m.margins(x, noise[s_], nk)
            if nk == si.NOISE_LOGISTIC:
                want = np.abs(z + noise[s_])
                np.testing.assert_array_equal(got, want.astype(np.float32))
            else:
                u = noise[s_].astype(np.float64)
                want = np.abs(z.astype(np.float64) - (np.log(u) - np.log1p(-u)))
                np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-7)
            assert np.all(got > 0)


def test_margin_gumbel_is_top_two_gap():
    cfg, m, noise = _margin_case(si.NOISE_GUMBEL)
    rng = np.random.default_rng(8)
    for s_ in range(cfg.batch):
        x = rng.integers(0, cfg.C, cfg.D, dtype=np.uint8)
        sc = m.forward_logits(x) + noise[s_]                  # float32 sums, as the decision takes them
        part = np.partition(sc, cfg.C - 2, axis=1)
        want = part[:, -1] - part[:, -2]
        np.testing.assert_array_equal(m.margins(x, noise[s_], si.NOISE_GUMBEL), want)
    # the largest value first, then last: `second` has to follow `top` both ways
    z = np.zeros((cfg.D, cfg.C), np.float32)
    g = np.tile(np.array([5, 1, 4, 0, 2, 3], np.float32), (cfg.D, 1))
    m0 = Oracle.made(cfg.D, cfg.C, [4], si.ACT_RELU, si.PREC_F32,
                     [np.zeros((4, cfg.D), np.float32), np.zeros((cfg.D * cfg.C, 4), np.float32)],
                     [np.zeros(4, np.float32), z.reshape(-1)], si.made_lut(cfg))
    np.testing.assert_array_equal(m0.margins(np.zeros(cfg.D, np.uint8), g, si.NOISE_GUMBEL), np.ones(cfg.D, np.float32))
    np.testing.assert_array_equal(m0.margins(np.zeros(cfg.D, np.uint8), g[:, ::-1].copy(), si.NOISE_GUMBEL),
                                  np.ones(cfg.D, np.float32))


def test_margin_uniform_cat_is_twice_the_gap_to_the_nearest_boundary():
    cfg, m, noise = _margin_case(si.NOISE_UNIFORM_CAT)
    rng = np.random.default_rng(9)
    for s_ in range(cfg.batch):
        x = rng.integers(0, cfg.C, cfg.D, dtype=np.uint8)
        z = m.forward_logits(x).astype(np.float64)
        p = np.exp(z - z.max(1, keepdims=True))
        cdf = np.cumsum(p, 1) / p.sum(1, keepdims=True)
        u = noise[s_].astype(np.float64)
        lo = np.concatenate([np.full((cfg.D, 1), -np.inf), cdf[:, :-1]], 1)
        hi = np.concatenate([cdf[:, :-1], np.full((cfg.D, 1), np.inf)], 1)
        k = m.jacobi_step(x, noise[s_], si.NOISE_UNIFORM_CAT)
        idx = np.arange(cfg.D)
        want = 2 * np.minimum(u - lo[idx, k], hi[idx, k] - u)
        np.testing.assert_allclose(m.margins(x, noise[s_], si.NOISE_UNIFORM_CAT), want, rtol=1e-5, atol=1e-7)


@pytest.mark.parametrize("nk", [si.NOISE_LOGISTIC, si.NOISE_UNIFORM_ICDF, si.NOISE_GUMBEL, si.NOISE_UNIFORM_CAT])
def test_margin_is_the_distance_to_a_flipped_decision(nk):
    """Moving the noise by a little less than the margin keeps every decision, by a little more flips
    the decision of that position (and of no earlier one)."""
    cfg, m, noise = _margin_case(nk)
    rng = np.random.default_rng(10)
    x = rng.integers(0, cfg.n_symbols, cfg.D, dtype=np.uint8)
    u = noise[0]
    base = m.jacobi_step(x, u, nk)
    mg = m.margins(x, u, nk).astype(np.float64)
    z = m.forward_logits(x).astype(np.float64)
    for t in range(cfg.D):
        for scale, flips in ((0.98, False), (1.02, True)):
            v = u.astype(np.float64).copy()
            d = scale * mg[t]
            if nk == si.NOISE_LOGISTIC:
                v[t] += -d if base[t] == 1 else d
            elif nk == si.NOISE_UNIFORM_ICDF:
                lg = np.log(v[t]) - np.log1p(-v[t])
                lg += d if base[t] == 1 else -d                      # towards the threshold z
                v[t] = 1 / (1 + np.exp(-lg))
            elif nk == si.NOISE_GUMBEL:
                sc = z[t] + v[t]
                runner = np.argsort(sc)[-2]
                v[t, runner] += d
            else:
                p = np.exp(z[t] - z[t].max())
                cdf = np.cumsum(p) / p.sum()
                k = int(base[t])
                below = v[t] - (cdf[k - 1] if k > 0 else -np.inf)
                above = (cdf[k] if k < cfg.C - 1 else np.inf) - v[t]
                v[t] += (-d if below < above else d) / 2
            out = m.jacobi_step(x, v.astype(np.float32), nk)
            np.testing.assert_array_equal(out[:t], base[:t])
            assert (out[t] != base[t]) == flips, (nk, t, scale, mg[t])


# ---------------------------------- categorical inverse CDF, one uniform number per position
def test_uniform_cat_brute_force_and_numpy_rule():
    """All 3^5 outcomes of a tiny 3-way model: for given uniforms exactly one outcome is a fixed point
    of the parallel update computed by numpy (softmax, cumulative sum, first class whose cumulative
    probability exceeds u), and every solver returns it."""
    nk = si.NOISE_UNIFORM_CAT
    cfg = si.MadeConfig("icdf", 51, D=5, C=3, H=(10,), act=si.ACT_RELU, prec=si.PREC_F32, batch=12,
                        noise_kind=nk, w_var_scale=12.0, b_var=0.5)
    W, b = si.made_weights(cfg)
    m = oracle.from_config(cfg, W, b, si.made_lut(cfg))
    noise = si.draw_noise(cfg)
    allx = np.array(list(itertools.product(range(3), repeat=cfg.D)), dtype=np.uint8)
    Z = np.stack([m.forward_logits(v) for v in allx]).astype(np.float64)              # [243, D, 3]
    P = np.exp(Z - Z.max(2, keepdims=True))
    CDF = np.cumsum(P, 2) / P.sum(2, keepdims=True)
    prob = np.prod(np.take_along_axis(P / P.sum(2, keepdims=True), allx[:, :, None].astype(np.int64), 2)[:, :, 0], 1)
    assert abs(prob.sum() - 1) < 1e-12
    iters = []
    for s_ in range(cfg.batch):
        u = noise[s_].astype(np.float64)
        G = np.minimum((CDF <= u[None, :, None]).sum(2), cfg.C - 1).astype(np.uint8)   # first class with CDF > u
        fixed = np.nonzero(np.all(G == allx, axis=1))[0]
        assert len(fixed) == 1
        xstar = allx[fixed[0]]
        np.testing.assert_array_equal(m.jacobi_step(xstar, noise[s_], nk), xstar)
        np.testing.assert_array_equal(m.sequential(noise[s_], nk), xstar)
        np.testing.assert_array_equal(m.sequential(noise[s_], nk, literal=True), xstar)
        xj, k, conv, _ = m.jacobi(noise[s_], nk)
        np.testing.assert_array_equal(xj, xstar)
        assert conv and k <= cfg.D
        iters.append(k)
        np.testing.assert_array_equal(m.gs_jacobi(noise[s_], nk, 2)[0], xstar)
        np.testing.assert_array_equal(m.jacobi_gs(noise[s_], nk, 2)[0], xstar)
    assert max(iters) > 2          # the couplings are strong enough for the iteration to matter


def test_uniform_cat_boundary_goes_to_the_upper_class():
    """Four equally likely classes: the cumulative probabilities are 1/4, 1/2, 3/4, 1 exactly; a uniform
    number equal to a boundary belongs to the class above it (strict comparison), 0 to class 0 and
    anything up to 1 to the last class."""
    D, C = 3, 4
    m0 = Oracle.made(D, C, [2], si.ACT_RELU, si.PREC_F32,
                     [np.zeros((2, D), np.float32), np.zeros((D * C, 2), np.float32)],
                     [np.zeros(2, np.float32), np.zeros(D * C, np.float32)], np.zeros(C, np.float32))
    x = np.zeros(D, np.uint8)
    for u, want in ((0.0, 0), (0.2499, 0), (0.25, 1), (0.5, 2), (0.7499, 2), (0.75, 3), (1.0, 3)):
        out = m0.jacobi_step(x, np.full(D, u, np.float32), si.NOISE_UNIFORM_CAT)
        np.testing.assert_array_equal(out, np.full(D, want, np.uint8))
