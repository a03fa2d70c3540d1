"""JS_OPT_TRACE / js_get_trace: the device timeline of a call, for both tensor-core kernels.

The stamps of a phase must be ordered in time (producer start <= first operands <= last MMA issued,
last accumulator <= epilogues done <= barrier passed), phases must follow one another, and tracing must
not change the samples.  The second traced CTA can be chosen."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _model(cfg):
    import paper_2002_03629_b200 as p
    if cfg.kind == "made":
        W, b = si.made_weights(cfg)
        lut = si.made_lut(cfg)
    else:
        W, b = si.conv_weights(cfg)
        lut = si.conv_lut(cfg)
    return p, p.Model.from_config(cfg, W, b, lut)


@pytest.mark.parametrize("name", ["made", "conv"])
def test_timeline_is_ordered_and_tracing_changes_nothing(name):
    cfg = (si.scaled(si.CONFIGS["made_784"], D=256, H=(256, 256), batch=130) if name == "made"
           else si.scaled(si.CONFIGS["conv_32"], height=8, width=8, ch=64, layers=2, batch=3))
    p, model = _model(cfg)
    try:
        noise = torch.from_numpy(si.draw_noise(cfg)).cuda()
        ref = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
        assert p.jacobi_sample(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, ref) == 0
        passes = model.stats().iterations
        model.set_option(p.JS_OPT_TRACE, 1)
        out = torch.empty_like(ref)
        assert p.jacobi_sample(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, out) == 0
        assert torch.equal(out, ref)
        tr = model.trace().astype(np.int64)[0]                  # first CTA: [phase][slot]
        layers = (len(cfg.H) if cfg.kind == "made" else cfg.layers) + 1
        phases = [ph for ph in range(1, tr.shape[0]) if tr[ph, 5] > 0]
        assert len(phases) == passes * layers                   # every layer of every pass left a barrier stamp
        last_barrier = 0
        for ph in phases:
            row = tr[ph]
            assert row[0] >= last_barrier > -1                  # a phase starts after the previous barrier
            worked = row[1] > 0                                 # this CTA had a tile in the phase
            if worked:
                assert row[0] <= row[1] <= row[2] <= row[5]
                assert row[3] <= row[4] <= row[5]
            last_barrier = row[5]
        # a chosen CTA in the second slot (option value n >= 2 traces CTA n - 2 beside the first one): CTA 1
        # has a tile in the first phase of both cases, so its row carries a start stamp and a barrier stamp
        # that lie inside the first CTA's call
        model.set_option(p.JS_OPT_TRACE, 2 + 1)
        assert p.jacobi_sample(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, out) == 0
        assert torch.equal(out, ref)
        both = model.trace().astype(np.int64)
        first, chosen = both[0], both[1]
        ph1 = [ph for ph in range(1, first.shape[0]) if first[ph, 5] > 0][0]
        assert chosen[ph1, 0] > 0 and chosen[ph1, 5] >= chosen[ph1, 0]
        assert abs(chosen[ph1, 5] - first[ph1, 5]) < 1_000_000          # the same barrier, within a millisecond
        model.set_option(p.JS_OPT_TRACE, 0)
    finally:
        model.close()
