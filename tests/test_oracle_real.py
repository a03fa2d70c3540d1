"""Pins of the oracle's continuous-state sampler (logistic conditionals, stopping tolerance eps > 0)
against closed forms, numpy recomputation, Proposition 1 and the definition of the stopping rule."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from oracle import Oracle
from test_oracle_pins import bf16, made_masks


def real_model(prec=si.PREC_F32, D=10, H=(20, 16), index=81, w_var_scale=3.0, batch=6):
    cfg = si.MadeConfig("real", index, D=D, C=2, H=H, act=si.ACT_RELU, prec=prec, batch=batch,
                        noise_kind=si.NOISE_LOGISTIC, w_var_scale=w_var_scale, b_var=0.05)
    W, b = si.made_weights(cfg)
    W[-1][1::2] *= 0.25                      # log-scales stay moderate
    b[-1][1::2] -= 1.0
    m = Oracle.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, W, b, np.zeros(2, np.float32))
    return cfg, W, b, m, si.draw_noise(cfg)


def numpy_logits_real(cfg, W, b, x):
    masks = made_masks(cfg.D, 2, cfg.H)
    rnd = bf16 if cfg.prec == si.PREC_BF16 else (lambda v: np.asarray(v, dtype=np.float32))
    a = rnd(x).astype(np.float64)
    for l in range(len(cfg.H)):
        pre = (rnd(W[l] * masks[l]).astype(np.float64) @ a + b[l]).astype(np.float32).astype(np.float64)
        a = rnd(np.maximum(pre, 0).astype(np.float32)).astype(np.float64)
    return (rnd(W[-1] * masks[-1]).astype(np.float64) @ a + b[-1]).astype(np.float32).reshape(cfg.D, 2)


@pytest.mark.parametrize("prec", [si.PREC_F32, si.PREC_BF16])
def test_real_forward_matches_numpy_and_is_autoregressive(prec):
    cfg, W, b, m, noise = real_model(prec)
    rng = np.random.default_rng(1)
    x = rng.normal(size=cfg.D).astype(np.float32)
    z = m.forward_logits_real(x)
    np.testing.assert_array_equal(z, numpy_logits_real(cfg, W, b, x))
    for t in range(cfg.D):
        y = x.copy()
        y[t] += 1.5
        zy = m.forward_logits_real(y)
        np.testing.assert_array_equal(zy[: t + 1], z[: t + 1])
    assert np.any(m.forward_logits_real(x + 1)[1:] != z[1:])


def test_real_update_is_location_plus_scale_times_noise():
    """x_t = m_t + exp(l_t) * noise_t, with the logits of a numpy forward pass."""
    cfg, W, b, m, noise = real_model()
    rng = np.random.default_rng(2)
    x = rng.normal(size=cfg.D).astype(np.float32)
    z = numpy_logits_real(cfg, W, b, x).astype(np.float64)
    want = (z[:, 0] + np.exp(z[:, 1]) * noise[0].astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(m.jacobi_step_real(x, noise[0]), want)
    # with all weights zero the positions are independent logistic variables with the biases' location and scale
    Wz = [w * 0 for w in W]
    m0 = Oracle.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, Wz, b, np.zeros(2, np.float32))
    want0 = (b[-1][0::2].astype(np.float64) + np.exp(b[-1][1::2].astype(np.float64)) * noise[1]).astype(np.float32)
    np.testing.assert_array_equal(m0.sequential_real(noise[1]), want0)
    x0, k0, c0 = m0.jacobi_real(noise[1])
    np.testing.assert_array_equal(x0, want0)
    assert k0 == 2 and c0                       # Example 1: one step reaches it, the second confirms


def test_real_first_position_follows_the_logistic_law():
    """Position 0 depends on nothing: x_0 = m + s * logit(u) is logistic(m, s); Kolmogorov-Smirnov against its CDF."""
    cfg, W, b, m, _ = real_model(D=4, H=(8,), index=82)
    N = 4000
    noise = si.draw_noise(cfg, batch=N)
    x0 = np.array([m.sequential_real(noise[i])[0] for i in range(N)], dtype=np.float64)
    loc, scale = float(b[-1][0]), float(np.exp(np.float64(b[-1][1])))
    xs = np.sort(x0)
    cdf = 1 / (1 + np.exp(-(xs - loc) / scale))
    ks = np.max(np.abs(cdf - (np.arange(1, N + 1) - 0.5) / N))
    assert ks < 1.95 / np.sqrt(N), ks            # 0.1 % level


@pytest.mark.parametrize("prec", [si.PREC_F32, si.PREC_BF16])
def test_real_jacobi_is_exact_within_T_iterations(prec):
    """Proposition 1 on continuous states with eps = 0: from any start the exact feedforward result, after k
    iterations the first k states are exact, at most T iterations."""
    cfg, W, b, m, noise = real_model(prec)
    rng = np.random.default_rng(3)
    for s_ in range(cfg.batch):
        ref = m.sequential_real(noise[s_])
        for init in (None, rng.normal(size=cfg.D).astype(np.float32)):
            x, k, conv = m.jacobi_real(noise[s_], 0.0, init)
            np.testing.assert_array_equal(x, ref)
            assert conv and k <= cfg.D
            y = np.zeros(cfg.D, np.float32) if init is None else init.copy()
            for it in range(1, cfg.D + 1):
                y = m.jacobi_step_real(y, noise[s_])
                np.testing.assert_array_equal(y[:it], ref[:it])
        for B in (1, 3, cfg.D):
            xg, kg, cg = m.gs_jacobi_real(noise[s_], B)
            np.testing.assert_array_equal(xg, ref)
            assert cg
        assert m.gs_jacobi_real(noise[s_], 1)[1] == cfg.D          # one-position blocks: the feedforward pass


def test_real_stopping_rule_is_the_first_small_maximum_change():
    """With eps > 0 the iteration stops at the first k whose largest change is <= eps (and not before), a
    larger eps never needs more iterations, and the error of the stopped iterate shrinks with eps."""
    cfg, W, b, m, noise = real_model(D=24, H=(48, 40), index=83, w_var_scale=2.0)
    errs = {}
    for s_ in range(cfg.batch):
        ref = m.sequential_real(noise[s_])
        last_k = None
        for eps in (0.0, 1e-6, 1e-3, 1e-1):
            x, k, conv = m.jacobi_real(noise[s_], eps)
            y, kk = np.zeros(cfg.D, np.float32), 0
            while True:
                prev, y = y, m.jacobi_step_real(y, noise[s_])
                kk += 1
                if np.max(np.abs(y - prev)) <= eps or kk == cfg.D:
                    break
            assert k == kk and conv
            np.testing.assert_array_equal(x, y)
            if last_k is not None:
                assert k <= last_k
            last_k = k
            errs.setdefault(eps, []).append(float(np.max(np.abs(x - ref))))
        x2, k2, conv2 = m.jacobi_real(noise[s_], 0.0, max_iters=2)
        assert k2 == 2 and not conv2
    assert max(errs[0.0]) == 0.0
    assert np.mean(errs[1e-1]) >= np.mean(errs[1e-3]) >= np.mean(errs[1e-6])
    # a change in ONE position beyond eps must keep the iteration going: the maximum norm, not a mean
    assert np.mean(errs[1e-1]) > 0


def test_real_gs_jacobi_follows_algorithm_3_step_by_step():
    """Blocks in order; inside a block only its own states are updated and only its own largest change is
    tested against eps: recomputed here from single parallel updates."""
    cfg, W, b, m, noise = real_model(D=24, H=(48, 40), index=84, w_var_scale=2.0)
    for s_ in range(3):
        for B, eps in ((5, 0.0), (8, 1e-3), (24, 1e-2)):
            x = np.zeros(cfg.D, np.float32)
            total = 0
            for a in range(0, cfg.D, B):
                e = min(a + B, cfg.D)
                k = 0
                while True:
                    nxt = m.jacobi_step_real(x, noise[s_])
                    k += 1
                    d = np.max(np.abs(nxt[a:e] - x[a:e]))
                    x[a:e] = nxt[a:e]
                    if d <= eps or k == e - a:
                        break
                total += k
            got, kk, conv = m.gs_jacobi_real(noise[s_], B, eps)
            np.testing.assert_array_equal(got, x)
            assert kk == total and conv
