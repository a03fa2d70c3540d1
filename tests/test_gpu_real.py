"""Continuous states with logistic conditionals on the device (jacobi_sample_real) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from oracle import Oracle

pytestmark = pytest.mark.gpu


def pkg():
    import __graft_entry__ as ge
    ge.build()
    import paper_2002_03629_b200 as p
    return p


class RealCase:
    def __init__(self, prec, D=40, H=(96, 72), batch=37, index=91, w_var_scale=2.0):
        p = pkg()
        self.p = p
        self.cfg = cfg = si.MadeConfig("real", index, D=D, C=2, H=H, act=si.ACT_RELU, prec=prec, batch=batch,
                                       noise_kind=si.NOISE_LOGISTIC, w_var_scale=w_var_scale, b_var=0.05)
        W, b = si.made_weights(cfg)
        W[-1][1::2] *= 0.25
        b[-1][1::2] -= 1.0
        lut = np.zeros(2, np.float32)
        self.orc = Oracle.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, W, b, lut)
        self.model = p.Model.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, W, b, lut, cfg.batch)
        self.noise = si.draw_noise(cfg)
        self.d_noise = torch.from_numpy(self.noise).cuda()
        # fp32 models: the two sides differ by float rounding only; bf16 models: a hidden unit now and then
        # rounds the other way (see the logit tolerance of the symbol samplers), and states feed back
        self.tol = 5e-4 if prec == si.PREC_F32 else 6e-2

    def run(self, mode, block=0, eps=0.0, max_iters=0, init=None):
        cfg, p = self.cfg, self.p
        out = torch.full((cfg.batch, cfg.D), 7.0, dtype=torch.float32, device="cuda")
        iters = torch.full((cfg.batch,), -1, dtype=torch.int32, device="cuda")
        d_init = None if init is None else torch.from_numpy(init).cuda()
        rc = p.jacobi_sample_real(self.model, self.d_noise, d_init, mode, block, max_iters, eps, out, iters)
        return rc, out.cpu().numpy(), iters.cpu().numpy()

    def close_to(self, got, want):
        scale = np.maximum(1.0, np.abs(want))
        assert np.max(np.abs(got - want) / scale) <= self.tol, float(np.max(np.abs(got - want) / scale))


@pytest.fixture(scope="module", params=[si.PREC_F32, si.PREC_BF16], ids=["f32", "bf16"])
def case(request):
    return RealCase(request.param)


def test_real_network_outputs_match_oracle(case):
    p, cfg = case.p, case.cfg
    x = np.random.default_rng(4).normal(size=(cfg.batch, cfg.D)).astype(np.float32)
    z = torch.empty((cfg.batch, cfg.D, 2), dtype=torch.float32, device="cuda")
    assert p.js_forward_logits_real(case.model, torch.from_numpy(x).cuda(), z) == 0
    ref = np.stack([case.orc.forward_logits_real(x[s]) for s in range(6)])
    got = z[:6].cpu().numpy()
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    err = np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms))
    assert err <= (1e-5 if cfg.prec == si.PREC_F32 else 2e-2), err


def test_real_exact_solvers_agree_with_the_feedforward_pass(case):
    """eps = 0: Jacobi, GS-Jacobi and the strict order return the very same floats on the device (Propositions 1
    and 2: all solve the same triangular system with the same arithmetic), close to the oracle's."""
    p, cfg = case.p, case.cfg
    ref = np.stack([case.orc.sequential_real(case.noise[s]) for s in range(cfg.batch)])
    seq = torch.empty((cfg.batch, cfg.D), dtype=torch.float32, device="cuda")
    assert p.sequential_sample_real(case.model, case.d_noise, seq) == 0
    seq = seq.cpu().numpy()
    case.close_to(seq, ref)
    init = np.random.default_rng(5).normal(size=(cfg.batch, cfg.D)).astype(np.float32)
    for mode, B, i0 in ((p.JS_JACOBI, 0, None), (p.JS_JACOBI, 0, init), (p.JS_GS_JACOBI, 7, None),
                        (p.JS_GS_JACOBI, 40, init), (p.JS_GAUSS_SEIDEL, 0, init)):
        rc, x, it = case.run(mode, B, 0.0, init=i0)
        assert rc == 0
        np.testing.assert_array_equal(x, seq)
        if mode == p.JS_JACOBI:
            assert it.max() <= cfg.D
            want = np.array([case.orc.jacobi_real(case.noise[s], 0.0, None if i0 is None else i0[s])[1]
                             for s in range(cfg.batch)])
            # with eps = 0 the count is the iteration at which the floats stop moving in their last bit; the
            # oracle evaluates the update in double and the kernel in float, so that moment may come an
            # iteration or two apart (the counts for eps > 0 are compared sharply in the next test)
            assert np.abs(it - want).max() <= 2, (it, want)
        elif mode == p.JS_GAUSS_SEIDEL:
            assert np.all(it == 1)
    with pytest.raises(p.JsError) as e:
        case.run(p.JS_JACOBI_GS, 8)
    assert e.value.code == p.JS_ERR_UNSUPPORTED


@pytest.mark.parametrize("eps", [1e-4, 1e-2, 0.3])
def test_real_stopping_tolerance(case, eps):
    """eps > 0: per-sample stopping at the first iteration whose largest change is <= eps: iteration counts beside
    the oracle's (equal unless the oracle's deciding change lies within a few percent of eps), states close to
    the oracle's stopped iterate, and the device's own stopped iterate obeys the rule."""
    p, cfg = case.p, case.cfg
    rc, x, it = case.run(p.JS_JACOBI, 0, eps)
    assert rc == 0
    n_same = 0
    for s in range(cfg.batch):
        xo, ko, conv = case.orc.jacobi_real(case.noise[s], eps)
        assert conv
        if it[s] == ko:
            n_same += 1
            case.close_to(x[s], xo)
        else:
            # the change that decided the oracle's stop (or non-stop) must be a near-tie with eps
            y = np.zeros(cfg.D, np.float32)
            deltas = []
            for _ in range(max(ko, int(it[s]))):
                prev, y = y, case.orc.jacobi_step_real(y, case.noise[s])
                deltas.append(float(np.max(np.abs(y - prev))))
            k_lo = min(ko, int(it[s]))
            assert abs(deltas[k_lo - 1] - eps) <= max(case.tol, 0.05) * max(eps, deltas[k_lo - 1]), (s, ko, it[s], deltas)
    assert n_same >= cfg.batch - 3
    # a larger tolerance never needs more iterations
    rc2, x2, it2 = case.run(p.JS_JACOBI, 0, eps * 10)
    assert np.all(it2 <= it)
    # truncated run
    rc3, x3, it3 = case.run(p.JS_JACOBI, 0, 0.0, max_iters=3)
    assert rc3 == p.JS_NOT_CONVERGED and np.all(it3 == 3)
    xo3 = np.stack([case.orc.jacobi_real(case.noise[s], 0.0, max_iters=3)[0] for s in range(cfg.batch)])
    case.close_to(x3, xo3)


def test_real_entry_points_reject_symbol_models():
    p = pkg()
    cfg = si.CONFIGS["made_tiny"]
    W, b = si.made_weights(cfg)
    m = p.Model.from_config(cfg, W, b, si.made_lut(cfg))
    noise = torch.zeros((cfg.batch, cfg.D), device="cuda")
    out = torch.empty((cfg.batch, cfg.D), dtype=torch.float32, device="cuda")
    with pytest.raises(p.JsError) as e:
        p.jacobi_sample_real(m, noise, None, p.JS_JACOBI, 0, 0, 0.0, out)
    assert e.value.code == p.JS_ERR_UNSUPPORTED
    m.close()
