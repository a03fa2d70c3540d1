"""Parity of the CUDA masked-MLP sampler with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from parity import check_samples, logits_close

pytestmark = pytest.mark.gpu


def pkg():
    import __graft_entry__ as ge
    ge.build()
    import paper_2002_03629_b200 as p
    return p


class Case:
    """Arrays, oracle model and CUDA model of one workload."""

    def __init__(self, cfg, salt=0, path=None):
        p = pkg()
        self.p, self.cfg = p, cfg
        self.W, self.b = si.made_weights(cfg, salt)
        self.lut = si.made_lut(cfg)
        self.noise = si.draw_noise(cfg, salt=salt)
        self.orc = oracle.from_config(cfg, self.W, self.b, self.lut)
        self.model = p.Model.from_config(cfg, self.W, self.b, self.lut)
        if path is not None:
            self.model.set_option(p.JS_OPT_PATH, path)
        self.d_noise = torch.from_numpy(self.noise).cuda()
        self.nk = cfg.noise_kind
        self._xstar = None

    @property
    def xstar(self):
        if self._xstar is None:
            self._xstar = self.orc.sequential_batch(self.noise, self.nk, threads=8)
        return self._xstar

    def run(self, mode, block=0, max_iters=0, init=None):
        cfg, p = self.cfg, self.p
        out = torch.full((cfg.batch, cfg.D), 255, dtype=torch.uint8, device="cuda")
        iters = torch.full((cfg.batch,), -1, dtype=torch.int32, device="cuda")
        d_init = None if init is None else torch.from_numpy(init).cuda()
        rc = p.jacobi_sample(self.model, self.d_noise, self.nk, d_init, mode, block, max_iters, out, iters)
        return rc, out.cpu().numpy(), iters.cpu().numpy()

    def oracle_counts(self, mode, block=0, max_iters=0, init=None, samples=None):
        p, o = self.p, self.orc
        samples = range(self.cfg.batch) if samples is None else samples
        xs, its = [], []
        for s in samples:
            i0 = None if init is None else init[s]
            if mode == p.JS_JACOBI:
                x, it, _, _ = o.jacobi(self.noise[s], self.nk, i0, max_iters)
            elif mode == p.JS_GS_JACOBI:
                x, it, _ = o.gs_jacobi(self.noise[s], self.nk, block, i0, max_iters)
            elif mode == p.JS_JACOBI_GS:
                x, it, _ = o.jacobi_gs(self.noise[s], self.nk, block, i0, max_iters)
            else:
                x, it = o.gauss_seidel(self.noise[s], self.nk, i0), 1
            xs.append(x)
            its.append(it)
        return np.stack(xs), np.array(its, dtype=np.int32)

    def check(self, mode, block=0, init=None, expect_rc=0):
        rc, x, it = self.run(mode, block, 0, init)
        assert rc == expect_rc
        audit = check_samples(self.orc, x, self.xstar, self.noise, self.nk)
        _, it_ref = self.oracle_counts(mode, block, 0, init)
        clean = np.setdiff1d(np.arange(self.cfg.batch), audit["excused_samples"])
        np.testing.assert_array_equal(it[clean], it_ref[clean])
        return audit, it, it_ref


TINY = si.CONFIGS["made_tiny"]
BIN = si.scaled(si.CONFIGS["made_784"], D=200, H=(192, 160), batch=70)        # ragged tiles
CAT = si.scaled(si.CONFIGS["made_cat"], D=24, H=(128, 96), batch=9)
CHAIN = si.scaled(si.CONFIGS["made_4096"], D=256, H=(256, 256, 256, 256), batch=130, w_var_scale=4.0)

# long K ranges with few tiles: the tensor-core kernels cut every tile's K loop into several work units
SPLIT = si.scaled(si.CONFIGS["made_784"], D=512, H=(2688, 2688), batch=130, w_var_scale=3.0)

# four row tiles (the last one ragged) and enough 128-wide tiles per hidden layer to go without split K;
# compaction takes the working batch through every number of row tiles
ROWS4 = si.scaled(si.CONFIGS["made_784"], D=256, H=(1280, 1280), batch=400, w_var_scale=3.0, index=11)

# more rows than the 256-way epilogue keeps in shared memory: rows beyond load their noise directly
CAT_ROWS = si.scaled(si.CONFIGS["made_cat"], D=16, H=(64, 64), batch=100)

# uniform noise with the inverse-CDF rule on a bf16 model (the tensor-core epilogue has one instance per noise kind)
BIN_ICDF = si.scaled(si.CONFIGS["made_784"], D=144, H=(128,), batch=40, noise_kind=si.NOISE_UNIFORM_ICDF)

# 256-way positions sampled by the inverse CDF of the softmax from one uniform number each; the second
# case has long K ranges, so the tensor-core kernels cut its output tiles into several work units
CAT_ICDF = si.scaled(si.CONFIGS["made_cat"], D=24, H=(128, 96), batch=70, noise_kind=si.NOISE_UNIFORM_CAT, index=7)
CAT_ICDF_SPLIT = si.scaled(si.CONFIGS["made_cat"], D=16, H=(2688,), batch=20, noise_kind=si.NOISE_UNIFORM_CAT,
                           index=8, w_var_scale=2.0)
# 7-way positions: CUDA-core kernels only
CAT7_ICDF = si.MadeConfig("cat7", 9, D=20, C=7, H=(48,), act=si.ACT_RELU, prec=si.PREC_F32, batch=11,
                          noise_kind=si.NOISE_UNIFORM_CAT, w_var_scale=8.0, b_var=0.2)

CASES = {"tiny": TINY, "bin": BIN, "cat": CAT, "chain": CHAIN, "split": SPLIT, "rows4": ROWS4, "cat_rows": CAT_ROWS,
         "bin_icdf": BIN_ICDF, "cat_icdf": CAT_ICDF, "cat_icdf_split": CAT_ICDF_SPLIT, "cat7_icdf": CAT7_ICDF}
# kernel path: 1 = CUDA-core kernels, 0 = tensor-core kernels (bf16 models only)
COMBOS = [(n, 1) for n in CASES] + [(n, 0) for n in CASES if n != "tiny"]
COMBO_IDS = [f"{n}-{'tc' if p == 0 else 'cc'}" for n, p in COMBOS]
_cache = {}
_path = {"v": 1}


def case(name, path=None):
    path = _path["v"] if path is None else path
    key = (name, path)
    if key not in _cache:
        _cache[key] = Case(CASES[name], path=path)
    return _cache[key]


@pytest.fixture(params=[1, 0], ids=["cc", "tc"], autouse=True)
def kernel_path(request):
    """Every test runs once per kernel path; fp32-only cases skip the tensor-core pass."""
    _path["v"] = request.param
    yield request.param
    _path["v"] = 1


def _skip_if_not_applicable(name):
    if _path["v"] == 0 and CASES[name].prec != si.PREC_BF16:
        pytest.skip("tensor-core kernels serve bf16 models only")


@pytest.mark.parametrize("name", list(CASES))
def test_logits_match_oracle(name):
    _skip_if_not_applicable(name)
    c = case(name)
    cfg, p = c.cfg, c.p
    x = si.random_init(cfg, salt=5)
    logits = torch.empty((cfg.batch, cfg.D, cfg.C), dtype=torch.float32, device="cuda")
    assert p.js_forward_logits(c.model, torch.from_numpy(x).cuda(), logits) == 0
    got = logits.cpu().numpy()
    n = min(cfg.batch, 6)
    ref = np.stack([c.orc.forward_logits(x[s]) for s in range(n)])
    rel = 1e-5 if cfg.prec == si.PREC_F32 else 2e-2
    err, ok = logits_close(got[:n], ref, rel)
    assert ok, err


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("skip", [1, 0])
def test_jacobi_matches_sequential_and_counts(name, skip):
    _skip_if_not_applicable(name)
    c = case(name)
    c.model.set_option(c.p.JS_OPT_FRONTIER_SKIP, skip)
    try:
        c.check(c.p.JS_JACOBI)
        assert c.model.stats().path == _path["v"]          # the requested kernels really ran
        c.check(c.p.JS_JACOBI, init=si.random_init(c.cfg, salt=1))
    finally:
        c.model.set_option(c.p.JS_OPT_FRONTIER_SKIP, 1)


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("seq_skip", [0, 1, 2])
def test_sequential_and_gauss_seidel(name, seq_skip):
    """The strict order three ways: a full forward pass per position, the band that changed, and the
    cached sweep (every hidden unit evaluated once; binary bf16 models on the tensor cores)."""
    _skip_if_not_applicable(name)
    c = case(name)
    p, cfg = c.p, c.cfg
    c.model.set_option(p.JS_OPT_SEQ_SKIP, seq_skip)
    try:
        out = torch.full((cfg.batch, cfg.D), 7, dtype=torch.uint8, device="cuda")
        assert p.sequential_sample(c.model, c.d_noise, c.nk, out) == 0
        check_samples(c.orc, out.cpu().numpy(), c.xstar, c.noise, c.nk)
        if seq_skip == 2 and _path["v"] == 0 and cfg.C == 1:
            st = c.model.stats()
            assert st.path == 0 and st.iterations == 1 and st.mma_flops > 0, "the cached sweep must have served this call"
        rc, x, it = c.run(p.JS_GAUSS_SEIDEL, init=si.random_init(cfg, salt=2))
        assert rc == 0 and np.all(it == 1)
        check_samples(c.orc, x, c.xstar, c.noise, c.nk)
    finally:
        c.model.set_option(p.JS_OPT_SEQ_SKIP, 2)


@pytest.mark.parametrize("name,blocks", [("tiny", (1, 4, 5, 16)), ("bin", (64, 30, 1, 200)), ("cat", (8, 5)),
                                         ("chain", (32, 64, 100)), ("split", (256,)), ("bin_icdf", (48,)),
                                         ("cat_icdf", (8,)), ("cat7_icdf", (6,))])
@pytest.mark.parametrize("skip", [1, 0])
def test_hybrids(name, blocks, skip):
    _skip_if_not_applicable(name)
    c = case(name)
    p = c.p
    c.model.set_option(p.JS_OPT_FRONTIER_SKIP, skip)
    try:
        for B in blocks:
            for init in (None, si.random_init(c.cfg, salt=3)):
                c.check(p.JS_GS_JACOBI, B, init)
                c.check(p.JS_JACOBI_GS, B, init)
                # Algorithm 2 runs on the tensor cores for binary bf16 models, else on the CUDA cores
                assert c.model.stats().path == (0 if (_path["v"] == 0 and c.cfg.C == 1) else 1)
    finally:
        c.model.set_option(p.JS_OPT_FRONTIER_SKIP, 1)


@pytest.mark.parametrize("name", ["bin", "chain"])
def test_max_iters_returns_last_iterate(name):
    _skip_if_not_applicable(name)
    c = case(name)
    p = c.p
    _, it_full = c.oracle_counts(p.JS_JACOBI)
    k = max(2, int(it_full.max()) // 2)
    rc, x, it = c.run(p.JS_JACOBI, max_iters=k)
    x_ref, it_ref = c.oracle_counts(p.JS_JACOBI, max_iters=k)
    assert rc == (p.JS_NOT_CONVERGED if it_full.max() > k else 0)
    # after k iterations the first k positions are final (proof of Proposition 1): that prefix goes
    # through the ordinary sample check; the rest is the oracle's k-th iterate, bit for bit, for
    # every sample that needed no near-tie excuse
    audit = check_samples(c.orc, x, c.xstar, c.noise, c.nk, hi=k)
    clean = np.setdiff1d(np.arange(c.cfg.batch), audit["excused_samples"])
    np.testing.assert_array_equal(x[clean], x_ref[clean])
    np.testing.assert_array_equal(it[clean], it_ref[clean])
    assert len(clean) >= c.cfg.batch - 2


def test_compaction_changes_nothing_but_the_work():
    """Finished samples leave the working batch (tensor-core kernels): same samples, same
    per-sample counts, fewer tiles."""
    if _path["v"] != 0:
        pytest.skip("compaction lives in the tensor-core kernels")
    c = case("chain")
    p = c.p
    res = {}
    for on in (1, 0):
        c.model.set_option(p.JS_OPT_COMPACT, on)
        rc, x, it = c.run(p.JS_JACOBI)
        st = c.model.stats()
        res[on] = (x, it, st.compactions, st.tiles_issued)
        assert rc == 0
    c.model.set_option(p.JS_OPT_COMPACT, 1)
    np.testing.assert_array_equal(res[1][0], res[0][0])
    np.testing.assert_array_equal(res[1][1], res[0][1])
    assert res[0][2] == 0 and res[1][2] >= 1, "the 130-sample case must drop to one row tile at some point"
    assert res[1][3] < res[0][3]
    check_samples(c.orc, res[1][0], c.xstar, c.noise, c.nk)


def test_tiny_model_brute_force_on_device():
    """Config 1 on the device alone: logits of all 2^16 outcomes from js_forward_logits, the parallel
    update of every outcome under each sample's noise, and exactly one fixed point - the sample that
    jacobi_sample and sequential_sample return."""
    if _path["v"] != 1:
        pytest.skip("fp32 model: CUDA-core kernels")
    p = pkg()
    cfg = TINY
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    noise = si.draw_noise(cfg)
    D = cfg.D
    big = p.Model.from_config(cfg, W, b, lut, max_batch=4096)
    allx = ((np.arange(2 ** D)[:, None] >> np.arange(D)[None, :]) & 1).astype(np.uint8)
    Z = np.empty((2 ** D, D), np.float32)
    for s0 in range(0, 2 ** D, 4096):
        logits = torch.empty((4096, D, 1), dtype=torch.float32, device="cuda")
        assert p.js_forward_logits(big, torch.from_numpy(allx[s0:s0 + 4096]).cuda(), logits) == 0
        Z[s0:s0 + 4096] = logits[:, :, 0].cpu().numpy()
    P1 = (1.0 / (1.0 + np.exp(-Z.astype(np.float32)))).astype(np.float32)
    d_noise = torch.from_numpy(noise).cuda()
    out = torch.empty((cfg.batch, D), dtype=torch.uint8, device="cuda")
    seq = torch.empty_like(out)
    assert p.jacobi_sample(big, d_noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, out, None) == 0
    assert p.sequential_sample(big, d_noise, cfg.noise_kind, seq) == 0
    got = out.cpu().numpy()
    np.testing.assert_array_equal(got, seq.cpu().numpy())
    for s in range(cfg.batch):
        G = (noise[s][None, :] < P1).astype(np.uint8)
        fixed = np.nonzero(np.all(G == allx, axis=1))[0]
        assert len(fixed) == 1
        np.testing.assert_array_equal(allx[fixed[0]], got[s])
    big.close()


def test_examples_of_section_4_on_device():
    """Markov chain (Example 3): T iterations; independent chain (Example 1): one plus the confirmation."""
    p = pkg()
    T, c0 = 40, 64.0
    H = T - 1
    W0 = np.zeros((H, T), np.float32)
    W1 = np.zeros((T, H), np.float32)
    for j in range(H):
        W0[j, j] = 1.0
        W1[j + 1, j] = c0
    b1 = np.full(T, -c0 / 2, np.float32)
    b1[0] = c0
    cfg = si.MadeConfig("ex3", 41, D=T, C=1, H=(H,), act=si.ACT_RELU, prec=si.PREC_F32, batch=5,
                        noise_kind=si.NOISE_LOGISTIC)
    noise = si.draw_noise(cfg)
    lut = np.array([0, 1], np.float32)
    for W, expect in (([W0, W1], T), ([W0 * 0, W1 * 0], 2)):
        m = p.Model.made(T, 1, [H], p.JS_ACT_RELU, p.JS_F32, W, [np.zeros(H, np.float32), b1], lut, cfg.batch)
        out = torch.empty((cfg.batch, T), dtype=torch.uint8, device="cuda")
        iters = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")
        assert p.jacobi_sample(m, torch.from_numpy(noise).cuda(), si.NOISE_LOGISTIC, None, p.JS_JACOBI, 0, 0, out,
                               iters) == 0
        assert np.all(iters.cpu().numpy() == expect)
        if expect == T:
            assert np.all(out.cpu().numpy() == 1)
        m.close()


def test_argument_errors():
    c = case("tiny")
    p, cfg = c.p, c.cfg
    out = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
    lib = p.load_library()
    h = c.model._h
    s = torch.cuda.current_stream().cuda_stream
    assert lib.jacobi_sample(h, cfg.batch, None, c.nk, None, 0, 0, 0, out.data_ptr(), None, s) == p.JS_ERR_ARG
    assert lib.jacobi_sample(h, cfg.batch + 1, c.d_noise.data_ptr(), c.nk, None, 0, 0, 0, out.data_ptr(), None,
                             s) == p.JS_ERR_ARG
    assert lib.jacobi_sample(h, cfg.batch, c.d_noise.data_ptr(), c.nk, None, 7, 0, 0, out.data_ptr(), None,
                             s) == p.JS_ERR_ARG
    assert lib.jacobi_sample(h, cfg.batch, c.d_noise.data_ptr(), p.JS_NOISE_GUMBEL, None, 0, 0, 0, out.data_ptr(),
                             None, s) == p.JS_ERR_ARG
    assert lib.jacobi_sample(h, cfg.batch, c.d_noise.data_ptr(), c.nk, None, p.JS_GS_JACOBI, 0, 0, out.data_ptr(),
                             None, s) == p.JS_ERR_ARG
    assert lib.jacobi_sample(None, cfg.batch, c.d_noise.data_ptr(), c.nk, None, 0, 0, 0, out.data_ptr(), None,
                             s) == p.JS_ERR_ARG


def test_bounded_wait_reports_timeout_and_model_stays_usable():
    """With a spin limit of zero the first grid barrier gives up: the call returns
    JS_ERR_TIMEOUT instead of hanging, and the next call works again."""
    c = case("bin")
    p = c.p
    c.model.set_option(p.JS_OPT_SPIN_LIMIT, 0)
    try:
        with pytest.raises(p.JsError) as e:
            c.run(p.JS_JACOBI)
        assert e.value.code == p.JS_ERR_TIMEOUT
    finally:
        c.model.set_option(p.JS_OPT_SPIN_LIMIT, 1 << 22)
    c.check(p.JS_JACOBI)


def test_batch_of_one_and_aliasing_init():
    c = case("bin")
    p, cfg = c.p, c.cfg
    init = si.random_init(cfg, salt=4)
    buf = torch.from_numpy(init[:1].copy()).cuda()
    rc = p.jacobi_sample(c.model, c.d_noise[:1].contiguous(), c.nk, buf, p.JS_JACOBI, 0, 0, buf, None)
    assert rc == 0
    check_samples(c.orc, buf.cpu().numpy(), c.xstar[:1], c.noise[:1], c.nk)


def _shuffled_degrees(cfg, seed=5):
    rng = np.random.default_rng(seed)
    return [rng.permutation(1 + (np.arange(h) * (cfg.D - 1)) // h).astype(np.int32) for h in cfg.H]


@pytest.mark.parametrize("prec", [si.PREC_F32, si.PREC_BF16])
def test_custom_unsorted_hidden_degrees(prec):
    """Degrees given by the caller, in random order: the CUDA-core kernels serve the model (the
    tensor-core kernels need tile-monotone degrees and must decline it even when asked for), and
    logits, samples and counts equal the oracle's with the same degrees."""
    if _path["v"] != 1:
        pytest.skip("one pass is enough: the request for the tensor-core kernels is part of the test")
    p = pkg()
    cfg = si.MadeConfig("deg", 13, D=72, C=1, H=(136, 120), act=si.ACT_RELU, prec=prec, batch=33,
                        noise_kind=si.NOISE_LOGISTIC, w_var_scale=6.0, b_var=0.1)
    W, b = si.made_weights(cfg)
    lut = si.made_lut(cfg)
    hd = _shuffled_degrees(cfg)
    orc = oracle.Oracle.made(cfg.D, cfg.C, list(cfg.H), cfg.act, cfg.prec, W, b, lut, hidden_deg=hd)
    model = p.Model.made(cfg.D, cfg.C, list(cfg.H), cfg.act, cfg.prec, W, b, lut, cfg.batch, hidden_deg=hd)
    model.set_option(p.JS_OPT_PATH, 0)                     # ask for the tensor-core kernels
    noise = si.draw_noise(cfg)
    d_noise = torch.from_numpy(noise).cuda()
    x0 = si.random_init(cfg, salt=5)
    logits = torch.empty((cfg.batch, cfg.D, 1), dtype=torch.float32, device="cuda")
    assert p.js_forward_logits(model, torch.from_numpy(x0).cuda(), logits) == 0
    assert model.stats().path == 1, "unsorted degrees: the CUDA-core kernels must have run"
    ref = np.stack([orc.forward_logits(x0[s_]) for s_ in range(6)])
    err, ok = logits_close(logits[:6].cpu().numpy(), ref, 1e-5 if prec == si.PREC_F32 else 2e-2)
    assert ok, err
    xstar = orc.sequential_batch(noise, cfg.noise_kind, threads=8)
    for mode, B in ((p.JS_JACOBI, 0), (p.JS_GS_JACOBI, 16), (p.JS_JACOBI_GS, 16), (p.JS_GAUSS_SEIDEL, 0)):
        out = torch.full((cfg.batch, cfg.D), 255, dtype=torch.uint8, device="cuda")
        iters = torch.full((cfg.batch,), -1, dtype=torch.int32, device="cuda")
        assert p.jacobi_sample(model, d_noise, cfg.noise_kind, None, mode, B, 0, out, iters) == 0
        assert model.stats().path == 1
        audit = check_samples(orc, out.cpu().numpy(), xstar, noise, cfg.noise_kind)
        clean = np.setdiff1d(np.arange(cfg.batch), audit["excused_samples"])
        if mode == p.JS_JACOBI:
            want = np.array([orc.jacobi(noise[s_], cfg.noise_kind)[1] for s_ in range(cfg.batch)])
        elif mode == p.JS_GS_JACOBI:
            want = np.array([orc.gs_jacobi(noise[s_], cfg.noise_kind, B)[1] for s_ in range(cfg.batch)])
        elif mode == p.JS_JACOBI_GS:
            want = np.array([orc.jacobi_gs(noise[s_], cfg.noise_kind, B)[1] for s_ in range(cfg.batch)])
        else:
            want = np.ones(cfg.batch, np.int32)
        np.testing.assert_array_equal(iters.cpu().numpy()[clean], want[clean])
    model.close()


def test_row_without_a_finite_score_gets_class_zero():
    """A position whose logits are all NaN (a NaN bias here) has no largest score: the call returns
    cleanly and the position gets class 0 (CUDA-core kernels; the tensor-core epilogue starts its
    running argmax from class 0 as well)."""
    p = pkg()
    cfg = si.MadeConfig("nan", 14, D=10, C=12, H=(24,), act=si.ACT_RELU, prec=si.PREC_F32 if _path["v"] == 1 else si.PREC_BF16,
                        batch=5, noise_kind=si.NOISE_GUMBEL, w_var_scale=4.0)
    if _path["v"] == 0:
        pytest.skip("12-way outputs are served by the CUDA-core kernels only")
    W, b = si.made_weights(cfg)
    bad = 4
    b[-1][bad * cfg.C:(bad + 1) * cfg.C] = np.nan
    model = p.Model.from_config(cfg, W, b, si.made_lut(cfg))
    noise = torch.from_numpy(si.draw_noise(cfg)).cuda()
    out = torch.full((cfg.batch, cfg.D), 255, dtype=torch.uint8, device="cuda")
    rc = p.jacobi_sample(model, noise, cfg.noise_kind, None, p.JS_JACOBI, 0, 0, out, None)
    assert rc == 0
    x = out.cpu().numpy()
    assert np.all(x[:, bad] == 0) and x.max() < cfg.C
    model.close()


def test_jacobi_gs_on_tensor_cores_truncated_and_aliased():
    """Algorithm 2 on the tensor-core path: a lowered cap reports non-convergence with the oracle's
    iterate of that outer iteration, and init may alias the output buffer."""
    if _path["v"] != 0:
        pytest.skip("tensor-core path only")
    c = case("chain")
    p, cfg = c.p, c.cfg
    B = 32
    _, it_full = c.oracle_counts(p.JS_JACOBI_GS, B)
    assert it_full.max() >= 3
    rc, x, it = c.run(p.JS_JACOBI_GS, B, max_iters=2)
    x_ref, it_ref = c.oracle_counts(p.JS_JACOBI_GS, B, max_iters=2)
    assert rc == p.JS_NOT_CONVERGED
    # after two outer iterations the first two blocks are final (proof of Proposition 2)
    audit = check_samples(c.orc, x, c.xstar, c.noise, c.nk, hi=2 * B)
    clean = np.setdiff1d(np.arange(cfg.batch), audit["excused_samples"])
    np.testing.assert_array_equal(x[clean], x_ref[clean])
    np.testing.assert_array_equal(it[clean], it_ref[clean])
    init = si.random_init(cfg, salt=6)
    buf = torch.from_numpy(init.copy()).cuda()
    iters = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")
    assert p.jacobi_sample(c.model, c.d_noise, c.nk, buf, p.JS_JACOBI_GS, B, 0, buf, iters) == 0
    check_samples(c.orc, buf.cpu().numpy(), c.xstar, c.noise, c.nk)
    _, want = c.oracle_counts(p.JS_JACOBI_GS, B, init=init)
    np.testing.assert_array_equal(iters.cpu().numpy(), want)
