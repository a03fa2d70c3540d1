"""jacobi_sample_host: host buffers in and out, the noise upload overlapped with the first hidden layers.

Checked against jacobi_sample (device buffers) bit for bit, on every kernel path, twice in a row, from
pinned and from pageable memory."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _cases():
    made = si.CONFIGS["made_784"]
    return {
        # tensor-core kernel, binary outputs: the kernel itself waits for the noise
        "bin_tc": (si.scaled(made, D=256, H=(256, 256), batch=150), 0),
        # tensor-core kernel, 256-way outputs
        "cat_tc": (si.scaled(si.CONFIGS["made_cat"], D=24, H=(128, 96), batch=9), 0),
        # CUDA-core kernels: the launch waits for the upload
        "bin_cc": (si.scaled(made, D=64, H=(64,), batch=20), 1),
        "tiny": (si.CONFIGS["made_tiny"], 1),
        "conv": (si.scaled(si.CONFIGS["conv_32"], height=8, width=8, ch=64, layers=2, batch=3), 0),
    }


@pytest.mark.parametrize("name", list(_cases()))
@pytest.mark.parametrize("pinned", [True, False])
def test_host_call_equals_device_call(name, pinned):
    import paper_2002_03629_b200 as p
    cfg, path = _cases()[name]
    if cfg.kind == "made":
        W, b = si.made_weights(cfg)
        lut = si.made_lut(cfg)
    else:
        W, b = si.conv_weights(cfg)
        lut = si.conv_lut(cfg)
    noise = si.draw_noise(cfg)
    model = p.Model.from_config(cfg, W, b, lut)
    if cfg.kind == "made":
        model.set_option(p.JS_OPT_PATH, path)
    try:
        d_noise = torch.from_numpy(noise).cuda()
        for init in (None, si.random_init(cfg, salt=2)):
            for mode, block in ((p.JS_JACOBI, 0), (p.JS_GS_JACOBI, max(2, cfg.D // 3))):
                ref = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
                ref_it = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")
                d_init = None if init is None else torch.from_numpy(init).cuda()
                rc_ref = p.jacobi_sample(model, d_noise, cfg.noise_kind, d_init, mode, block, 0, ref, ref_it)
                h_noise = torch.from_numpy(noise.copy())
                h_init = None if init is None else torch.from_numpy(init.copy())
                h_out = torch.full((cfg.batch, cfg.D), 255, dtype=torch.uint8)
                h_it = torch.full((cfg.batch,), -1, dtype=torch.int32)
                if pinned:
                    h_noise, h_out, h_it = h_noise.pin_memory(), h_out.pin_memory(), h_it.pin_memory()
                    h_init = None if h_init is None else h_init.pin_memory()
                for _ in range(2):          # the staging buffers and the arrival word are reused
                    h_out.fill_(255)
                    rc = p.jacobi_sample_host(model, h_noise, cfg.noise_kind, h_init, mode, block, 0, h_out, h_it)
                    assert rc == rc_ref
                    assert torch.equal(h_out, ref.cpu())
                    assert torch.equal(h_it, ref_it.cpu())
        assert model.stats().path == (0 if cfg.kind == "conv" else path)
    finally:
        model.close()


def test_host_call_argument_errors():
    import paper_2002_03629_b200 as p
    cfg = si.CONFIGS["made_tiny"]
    W, b = si.made_weights(cfg)
    model = p.Model.from_config(cfg, W, b, si.made_lut(cfg))
    try:
        noise = torch.from_numpy(si.draw_noise(cfg))
        out = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8)
        with pytest.raises(p.JsError):        # a device tensor where host memory is expected
            p.jacobi_sample_host(model, noise.cuda(), cfg.noise_kind, None, p.JS_JACOBI, 0, 0, out)
        with pytest.raises(p.JsError):        # batch beyond the model's max_batch
            big = torch.empty((cfg.batch + 1, cfg.D), dtype=torch.uint8)
            p.jacobi_sample_host(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, big)
        with pytest.raises(p.JsError):        # hybrid without a block size
            p.jacobi_sample_host(model, noise, cfg.noise_kind, None, p.JS_GS_JACOBI, 0, 0, out)
    finally:
        model.close()
