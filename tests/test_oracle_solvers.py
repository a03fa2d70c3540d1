"""Pins of the oracle's iterative solvers: Propositions 1 and 2, the remark that
one Gauss-Seidel iteration is the feedforward pass (Section 3.2), the worked
Examples 1-3 and the critical-path bound (Section 4.1), and agreement of the
fast sweeps with the literal definitions."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from oracle import Oracle
from test_oracle_pins import small_conv, small_made


def _models():
    out = []
    cfg, W, b, lut, m = small_made(prec=si.PREC_BF16, D=14, H=(28, 28), w_var_scale=10.0)
    out.append(("made_bin", cfg, m))
    cfg, W, b, lut, m = small_made(prec=si.PREC_BF16, D=9, C=6, H=(18,), act=si.ACT_GELU_TANH,
                                   nk=si.NOISE_GUMBEL, index=12, w_var_scale=12.0)
    out.append(("made_cat", cfg, m))
    cfg, W, b, lut, m = small_conv()
    out.append(("conv", cfg, m))
    return out


MODELS = _models()
IDS = [m[0] for m in MODELS]


@pytest.mark.parametrize("name,cfg,m", MODELS, ids=IDS)
def test_sequential_sweep_equals_literal_definition(name, cfg, m):
    noise = si.draw_noise(cfg)
    for s in range(cfg.batch):
        np.testing.assert_array_equal(m.sequential(noise[s], cfg.noise_kind),
                                      m.sequential(noise[s], cfg.noise_kind, literal=True))


@pytest.mark.parametrize("name,cfg,m", MODELS, ids=IDS)
def test_prop1_jacobi_any_init_prefix_invariant(name, cfg, m):
    """Proposition 1 and the induction in its proof: from any start, after k
    parallel iterations the first k positions are final, and the result after at
    most T iterations is the feedforward one.  Also the sharper frontier: if
    iteration k left positions < j unchanged then positions <= j are final."""
    noise = si.draw_noise(cfg)
    T, nk = m.T, cfg.noise_kind
    inits = [si.zero_init(cfg), si.random_init(cfg), si.random_init(cfg, salt=1)]
    some_slow = False
    for s in range(cfg.batch):
        xstar = m.sequential(noise[s], nk)
        for init in inits:
            x = init[s].copy()
            for k in range(1, T + 1):
                nxt = m.jacobi_step(x, noise[s], nk)
                np.testing.assert_array_equal(nxt[:k], xstar[:k])
                diff = np.nonzero(nxt != x)[0]
                j = T if len(diff) == 0 else diff[0]
                np.testing.assert_array_equal(nxt[: min(j + 1, T)], xstar[: min(j + 1, T)])
                x = nxt
            np.testing.assert_array_equal(x, xstar)
            got, iters, conv, kc = m.jacobi(noise[s], nk, init[s], x_star=xstar)
            np.testing.assert_array_equal(got, xstar)
            assert conv and 1 <= iters <= T and 0 <= kc <= iters
            # the stop test fires one iteration after the iterate became exact, or at the cap
            assert iters == min(kc + 1, T) or (kc == 0 and iters == 1)
            some_slow |= kc > 2
    assert some_slow, "test model converges trivially; couple it more strongly"


@pytest.mark.parametrize("name,cfg,m", MODELS, ids=IDS)
def test_gauss_seidel_one_sweep_is_feedforward(name, cfg, m):
    noise = si.draw_noise(cfg)
    init = si.random_init(cfg)
    for s in range(cfg.batch):
        np.testing.assert_array_equal(m.gauss_seidel(noise[s], cfg.noise_kind, init[s]),
                                      m.sequential(noise[s], cfg.noise_kind))


@pytest.mark.parametrize("name,cfg,m", MODELS, ids=IDS)
def test_prop2_hybrids_exact_and_bounded(name, cfg, m):
    noise = si.draw_noise(cfg)
    T, nk = m.T, cfg.noise_kind
    init = si.random_init(cfg, salt=2)
    for s in range(min(cfg.batch, 3)):
        xstar = m.sequential(noise[s], nk)
        for B in (1, 3, 4, T):
            M = -(-T // B)
            x, it, conv = m.gs_jacobi(noise[s], nk, B, init[s])
            np.testing.assert_array_equal(x, xstar)
            assert conv and M <= it <= T           # at least one and at most |B_i| per block
            x, it, conv = m.jacobi_gs(noise[s], nk, B, init[s])
            np.testing.assert_array_equal(x, xstar)
            assert conv and 1 <= it <= M
            x2, it2, conv2 = m.jacobi_gs(noise[s], nk, B, init[s], literal=True)
            np.testing.assert_array_equal(x2, xstar)
            assert it2 == it
        # block size 1: GS-Jacobi is the feedforward pass, one inner iteration per position
        assert m.gs_jacobi(noise[s], nk, 1, init[s])[1] == T
        # one block of size T: both hybrids reduce to Jacobi / to one sequential sweep
        assert m.gs_jacobi(noise[s], nk, T, init[s])[1] == m.jacobi(noise[s], nk, init[s])[1]
        assert m.jacobi_gs(noise[s], nk, T, init[s])[1] == 1


@pytest.mark.parametrize("name,cfg,m", MODELS, ids=IDS)
def test_jacobi_gs_block_invariant(name, cfg, m):
    """Proof of Proposition 2: after outer iteration k the first k blocks are final."""
    noise = si.draw_noise(cfg)
    T, nk, B = m.T, cfg.noise_kind, 4
    init = si.random_init(cfg, salt=3)
    for s in range(min(cfg.batch, 2)):
        xstar = m.sequential(noise[s], nk)
        for k in range(1, -(-T // B) + 1):
            x, it, conv = m.jacobi_gs(noise[s], nk, B, init[s], max_iters=k)
            np.testing.assert_array_equal(x[: min(k * B, T)], xstar[: min(k * B, T)])


def test_max_iters_reports_non_convergence():
    name, cfg, m = MODELS[0]
    noise = si.draw_noise(cfg)
    nk = cfg.noise_kind
    found = False
    for s in range(cfg.batch):
        xstar = m.sequential(noise[s], nk)
        _, iters, _, kc = m.jacobi(noise[s], nk, x_star=xstar)
        if iters >= 4:
            x, it, conv, _ = m.jacobi(noise[s], nk, max_iters=2)
            assert it == 2 and not conv
            found = True
    assert found


# ------------------------------------------------ worked examples, Section 4.1
def _chain_model(T, kind, c=64.0):
    """Hand-built binary networks realising Examples 1-3 (one hidden layer of T-1
    ReLU units, hidden unit j has degree j+1 under the default rule)."""
    H = T - 1
    W0 = np.zeros((H, T), np.float32)
    W1 = np.zeros((T, H), np.float32)
    b0 = np.zeros(H, np.float32)
    b1 = np.full(T, -c / 2, np.float32)
    b1[0] = c
    if kind == "independent":          # Example 1: s_t = h_t(u)
        b1[:] = np.where(np.arange(T) % 2 == 0, c, -c)
    elif kind == "skip":               # Example 2: s_t = h_t(u, s_1)
        W0[0, 0] = 1.0                 # hidden unit 0 copies x_0
        W1[1:, 0] = c                  # every later position reads it
    elif kind == "markov":             # Example 3: s_t = h_t(s_{t-1})
        for j in range(H):
            W0[j, j] = 1.0             # hidden unit j copies x_j
            W1[j + 1, j] = c           # position j+1 reads it
    return Oracle.made(T, 1, [H], si.ACT_RELU, si.PREC_F32, [W0, W1], [b0, b1], np.array([0, 1], np.float32))


@pytest.mark.parametrize("kind,expected", [("independent", 1), ("skip", 2), ("markov", None)])
def test_worked_examples_iteration_counts(kind, expected):
    T = 20
    m = _chain_model(T, kind)
    cfg = si.MadeConfig("ex", 41, D=T, C=1, H=(T - 1,), act=si.ACT_RELU, prec=si.PREC_F32, batch=4,
                        noise_kind=si.NOISE_LOGISTIC)
    noise = si.draw_noise(cfg)
    assert np.abs(noise).max() < 30          # the constants dominate the noise
    want = T if expected is None else expected
    for s in range(cfg.batch):
        xstar = m.sequential(noise[s], si.NOISE_LOGISTIC)
        if kind != "independent":
            np.testing.assert_array_equal(xstar, np.ones(T, np.uint8))
        x, iters, conv, kc = m.jacobi(noise[s], si.NOISE_LOGISTIC, x_star=xstar)
        np.testing.assert_array_equal(x, xstar)
        assert kc == want                                 # the paper's counts: 1, 2, T
        assert iters == min(want + 1, T) and conv         # plus the confirming iteration
        # GS-Jacobi on the Markov chain needs |B| iterations in every block
        if kind == "markov":
            assert m.gs_jacobi(noise[s], si.NOISE_LOGISTIC, 5)[1] == T
            assert m.jacobi_gs(noise[s], si.NOISE_LOGISTIC, 5)[1] == 4
        if kind == "independent":
            assert m.jacobi_gs(noise[s], si.NOISE_LOGISTIC, 5)[1] == 2
            # Algorithm 3 starts every block from the initial guess: from a start that is wrong
            # everywhere each of the M blocks needs one iteration to fix itself and one to confirm
            # (an implementation that also updated later blocks early would need fewer)
            wrong = (1 - xstar).astype(np.uint8)
            assert m.gs_jacobi(noise[s], si.NOISE_LOGISTIC, 5, wrong)[1] == 2 * (T // 5)


def test_critical_path_bound():
    """Iterations to exactness never exceed the longest dependency path; a model
    whose positions only read positions at least `gap` earlier has a path of
    about T/gap."""
    T, gap = 24, 6
    cfg = si.MadeConfig("cp", 43, D=T, C=1, H=(T - 1,), act=si.ACT_RELU, prec=si.PREC_F32, batch=6,
                        noise_kind=si.NOISE_LOGISTIC, w_var_scale=40.0)
    W, b = si.made_weights(cfg)
    # hidden unit j (degree j+1) reads position j only; output d reads hidden units <= d-gap
    W0 = np.diag(np.ones(T - 1, np.float32))
    W0 = np.concatenate([W0, np.zeros((T - 1, 1), np.float32)], axis=1)
    W1 = W[1] * (np.arange(T - 1)[None, :] <= (np.arange(T)[:, None] - gap))
    m = Oracle.made(T, 1, [T - 1], si.ACT_RELU, si.PREC_F32, [W0, W1], b, np.array([0, 1], np.float32))
    noise = si.draw_noise(cfg)
    path = -(-T // gap)            # ceil(T / gap) positions can lie on one dependency chain
    worst = 0
    for s in range(cfg.batch):
        xstar = m.sequential(noise[s], si.NOISE_LOGISTIC)
        _, _, _, kc = m.jacobi(noise[s], si.NOISE_LOGISTIC, si.random_init(cfg)[s], x_star=xstar)
        assert kc <= path
        worst = max(worst, kc)
    assert worst >= 2
