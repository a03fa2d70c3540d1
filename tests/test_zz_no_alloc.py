"""jacobi_sample_noalloc, the entry point for callers that may not allocate device
memory, against jacobi_sample on the same fp32 model.

Collected last on purpose (file name): a run that stops at the first failure has
then already gone through every other test.  The entry point keeps its scratch in
one array inside the library that survives from call to call, so the test calls it
twice in a row, with different noise, and expects both results to match: leftovers
of the first call must not leak into the second."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _pkg():
    import __graft_entry__ as ge
    ge.build()
    import paper_2002_03629_b200 as p
    return p


CASES = [
    si.CONFIGS["made_tiny"],
    si.MadeConfig("na_bin", 51, D=48, C=1, H=(96, 80), act=si.ACT_RELU, prec=si.PREC_F32, batch=20,
                  noise_kind=si.NOISE_LOGISTIC, w_var_scale=8.0, b_var=0.1),
    si.MadeConfig("na_cat", 52, D=12, C=16, H=(40,), act=si.ACT_RELU, prec=si.PREC_F32, batch=7,
                  noise_kind=si.NOISE_GUMBEL, w_var_scale=10.0),
]


@pytest.mark.parametrize("cfg", CASES, ids=[c.name for c in CASES])
def test_noalloc_matches_jacobi_sample_twice_in_a_row(cfg):
    p = _pkg()
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    model = p.Model.from_config(cfg, W, b, lut)
    dW = [torch.from_numpy(w).cuda() for w in W]
    db = [torch.from_numpy(v).cuda() for v in b]
    dlut = torch.from_numpy(lut).cuda()
    assert p.noalloc_scratch_needed(cfg.D, cfg.C, cfg.H, cfg.batch) <= p.noalloc_scratch_limit()
    for call, (salt, init) in enumerate([(0, None), (1, si.random_init(cfg, salt=1))]):
        noise = torch.from_numpy(si.draw_noise(cfg, salt=salt)).cuda()
        d_init = None if init is None else torch.from_numpy(init).cuda()
        ref = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
        ref_it = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")
        rc_ref = p.jacobi_sample(model, noise, cfg.noise_kind, d_init, p.JS_JACOBI, 0, 0, ref, ref_it)
        got = torch.full_like(ref, 255)
        got_it = torch.full_like(ref_it, -1)
        rc = p.jacobi_sample_noalloc(cfg.D, cfg.C, cfg.H, cfg.act, dW, db, dlut, noise, cfg.noise_kind, d_init, 0,
                                     got, got_it)
        assert rc == rc_ref == 0, (call, rc, rc_ref)
        # integer outputs: bit-exact, like every other sample comparison in this suite
        assert torch.equal(got, ref), f"call {call}: samples differ"
        assert torch.equal(got_it, ref_it), f"call {call}: iteration counts differ"
    # a truncated run reports non-convergence the same way
    noise = torch.from_numpy(si.draw_noise(cfg, salt=0)).cuda()
    a, b2 = torch.empty_like(ref), torch.empty_like(ref)
    rc_ref = p.jacobi_sample(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 1, a, None)
    rc = p.jacobi_sample_noalloc(cfg.D, cfg.C, cfg.H, cfg.act, dW, db, dlut, noise, cfg.noise_kind, None, 1, b2, None)
    assert rc == rc_ref == p.JS_NOT_CONVERGED and torch.equal(a, b2)
    model.close()


def test_noalloc_rejects_shapes_beyond_its_scratch():
    p = _pkg()
    cfg = si.MadeConfig("na_big", 53, D=64, C=1, H=(4096,), act=si.ACT_RELU, prec=si.PREC_F32, batch=512,
                        noise_kind=si.NOISE_LOGISTIC)
    assert p.noalloc_scratch_needed(cfg.D, cfg.C, cfg.H, cfg.batch) > p.noalloc_scratch_limit()
    W = [torch.zeros((4096, 64), device="cuda"), torch.zeros((64, 4096), device="cuda")]
    b = [torch.zeros(4096, device="cuda"), torch.zeros(64, device="cuda")]
    lut = torch.tensor([0.0, 1.0], device="cuda")
    noise = torch.zeros((cfg.batch, cfg.D), device="cuda")
    out = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
    with pytest.raises(p.JsError) as e:
        p.jacobi_sample_noalloc(cfg.D, cfg.C, cfg.H, cfg.act, W, b, lut, noise, cfg.noise_kind, None, 0, out, None)
    assert e.value.code == p.JS_ERR_ARG and "scratch" in str(e.value)


def test_noalloc_row_without_a_finite_score_gets_class_zero():
    """Weights or noise from the caller may hold NaN: a position whose scores are all NaN has no
    largest one.  The call must come back cleanly with class 0 there, like jacobi_sample."""
    p = _pkg()
    cfg = CASES[2]
    W, b = si.made_weights(cfg)
    bad = 3
    b[-1][bad * cfg.C:(bad + 1) * cfg.C] = np.nan
    dW = [torch.from_numpy(w).cuda() for w in W]
    db = [torch.from_numpy(v).cuda() for v in b]
    dlut = torch.from_numpy(si.made_lut(cfg)).cuda()
    noise = torch.from_numpy(si.draw_noise(cfg)).cuda()
    got = torch.full((cfg.batch, cfg.D), 255, dtype=torch.uint8, device="cuda")
    rc = p.jacobi_sample_noalloc(cfg.D, cfg.C, cfg.H, cfg.act, dW, db, dlut, noise, cfg.noise_kind, None, 0, got, None)
    assert rc == 0
    x = got.cpu().numpy()
    assert np.all(x[:, bad] == 0) and x.max() < cfg.C
