"""Seeded synthetic inputs for the autoregressive samplers.

This module only draws random arrays (unmasked weights, biases, noise, initial
iterates) and names the workload shapes.  It holds none of the sampler's
arithmetic: no masks, no rounding to bf16, no forward pass, no sampling rule.
Both the CPU oracle's tests and the CUDA library's tests and benchmark take
their inputs from here, so the two sides always see identical arrays.

Recipe (all draws from ``numpy.random.Generator(PCG64(seed))``):

* seed of a stream = ``1000 * config_index + stream`` with stream 0 = weights,
  1 = biases, 2 = noise, 3 = random initial iterates;
* weights of a layer ``~ N(0, w_var_scale / fan_in)`` with ``fan_in`` the dense
  input width of the layer, stored unmasked as ``float32 [out, in]``;
* biases ``~ N(0, b_var)`` (zeros when ``b_var == 0``);
* noise from 32 random bits ``r``: ``u = (r + 0.5) * 2**-32`` in float64, then
  logistic ``log(u) - log(1 - u)`` or Gumbel ``-log(-log(u))`` rounded to
  float32; uniform noise (one number per position, for binary and for C-way
  inverse-CDF sampling alike) uses 23 bits, ``(k + 0.5) * 2**-23``, which
  float32 holds exactly and which can never reach 0 or 1.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np

NOISE_UNIFORM_ICDF = 0
NOISE_LOGISTIC = 1
NOISE_GUMBEL = 2
NOISE_UNIFORM_CAT = 3      # one uniform number per C-way position (inverse CDF of the softmax)

ACT_RELU = 0
ACT_GELU_TANH = 1

PREC_F32 = 0
PREC_BF16 = 1


@dataclass(frozen=True)
class MadeConfig:
    """Shape of a masked-MLP workload (one row of the benchmark's config list)."""
    name: str
    index: int                 # position in the config list; fixes the seeds
    D: int                     # number of positions T
    C: int                     # classes per position: 1 = binary, 256 = categorical
    H: tuple                   # hidden widths
    act: int
    prec: int
    batch: int
    noise_kind: int
    w_var_scale: float = 1.0   # weights ~ N(0, w_var_scale / fan_in)
    b_var: float = 0.0         # biases  ~ N(0, b_var)
    blocks: tuple = ()         # block sizes the workload asks the hybrids to use
    kind: str = "made"

    @property
    def n_symbols(self) -> int:
        return 2 if self.C == 1 else self.C


@dataclass(frozen=True)
class ConvConfig:
    """Shape of a masked-convolution workload (PixelCNN-style stack)."""
    name: str
    index: int
    height: int
    width: int
    in_ch: int                 # image channels (3)
    ch: int                    # hidden channels
    layers: int                # number of 3x3 masked convolutions
    C: int                     # classes per sub-pixel
    batch: int
    noise_kind: int = NOISE_GUMBEL
    prec: int = PREC_BF16
    blocks: tuple = ()
    kind: str = "conv"

    @property
    def D(self) -> int:
        return self.height * self.width * self.in_ch


CONFIGS: Dict[str, object] = {
    # config 1: tiny fp32 model, small enough to enumerate all 2^16 outcomes
    "made_tiny": MadeConfig("made_tiny", 0, D=16, C=1, H=(64,), act=ACT_RELU, prec=PREC_F32,
                            batch=8, noise_kind=NOISE_UNIFORM_ICDF),
    # config 2: binary 28x28 raster
    "made_784": MadeConfig("made_784", 1, D=784, C=1, H=(1024, 1024), act=ACT_RELU, prec=PREC_BF16,
                           batch=256, noise_kind=NOISE_LOGISTIC, b_var=0.1),
    # config 3: 256-way categorical
    "made_cat": MadeConfig("made_cat", 2, D=1024, C=256, H=(2048, 2048), act=ACT_GELU_TANH,
                           prec=PREC_BF16, batch=64, noise_kind=NOISE_GUMBEL, blocks=(64,)),
    # config 4: large chain with weakened long-range dependencies
    "made_4096": MadeConfig("made_4096", 3, D=4096, C=1, H=(4096, 4096, 4096, 4096), act=ACT_RELU,
                            prec=PREC_BF16, batch=512, noise_kind=NOISE_LOGISTIC, w_var_scale=0.5,
                            blocks=(128, 512)),
    # config 5: masked-convolution sampler
    "conv_32": ConvConfig("conv_32", 4, height=32, width=32, in_ch=3, ch=128, layers=8, C=256, batch=16),
}
# extension: config 3's model sampled by the categorical inverse CDF, one uniform number per position
# (same weights: same index; 1/256 of the noise)
CONFIGS["made_cat_icdf"] = replace(CONFIGS["made_cat"], name="made_cat_icdf", noise_kind=NOISE_UNIFORM_CAT)


# continuous states (logistic conditionals: a location and a log-scale per position, C = 2): config 2's shape
# with fp32 weights; stopping tolerance of the solvers in REAL_EPS
REAL_CONFIGS: Dict[str, MadeConfig] = {
    "made_784_real": MadeConfig("made_784_real", 7, D=784, C=2, H=(1024, 1024), act=ACT_RELU, prec=PREC_F32,
                                batch=256, noise_kind=NOISE_LOGISTIC, w_var_scale=2.0, b_var=0.05),
}
REAL_EPS = 0.01


def made_real_weights(cfg: MadeConfig, salt: int = 0):
    """Weights of a network with continuous states: the rows of the output layer that produce log-scales are
    damped (a quarter of the weight, bias shifted by -1), so that the conditionals stay narrow enough for the
    fixed-point iteration to settle in a few dozen steps."""
    W, b = made_weights(cfg, salt)
    W[-1][1::2] *= np.float32(0.25)
    b[-1][1::2] -= np.float32(1.0)
    return W, b


def scaled(cfg, **changes):
    """A smaller workload with the same structure (used by parity tests)."""
    return replace(cfg, **changes)


def _rng(cfg, stream: int, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(1000 * cfg.index + stream + 7919 * salt))


def _normal(rng, shape, var) -> np.ndarray:
    out = rng.standard_normal(shape, dtype=np.float32)
    out *= np.float32(np.sqrt(var))
    return out


def made_lut(cfg: MadeConfig) -> np.ndarray:
    """Input encoding table: network input for each symbol value.

    Binary positions feed 0/1; a 256-way position feeds the scalar
    ``x / 127.5 - 1`` (model data: both sides receive this very table).
    """
    if cfg.C == 1:
        return np.array([0.0, 1.0], dtype=np.float32)
    n = cfg.C
    return (np.arange(n, dtype=np.float64) / ((n - 1) / 2.0) - 1.0).astype(np.float32)


def made_weights(cfg: MadeConfig, salt: int = 0):
    """Unmasked weights ``W[l]`` (float32 ``[out, in]``) and biases ``b[l]`` for l = 0..L."""
    widths = [cfg.D, *cfg.H, cfg.D * cfg.C]
    rw, rb = _rng(cfg, 0, salt), _rng(cfg, 1, salt)
    W: List[np.ndarray] = []
    b: List[np.ndarray] = []
    for l in range(len(widths) - 1):
        fan_in, out = widths[l], widths[l + 1]
        W.append(_normal(rw, (out, fan_in), cfg.w_var_scale / fan_in))
        if cfg.b_var > 0:
            b.append(_normal(rb, (out,), cfg.b_var))
        else:
            b.append(np.zeros((out,), dtype=np.float32))
    return W, b


def noise_shape(cfg, batch: Optional[int] = None):
    bt = cfg.batch if batch is None else batch
    if cfg.noise_kind == NOISE_GUMBEL:
        return (bt, cfg.D, cfg.C)
    return (bt, cfg.D)


def draw_noise(cfg, batch: Optional[int] = None, salt: int = 0) -> np.ndarray:
    """Per-position noise, drawn once and reused by every iteration of every solver."""
    rng = _rng(cfg, 2, salt)
    shape = noise_shape(cfg, batch)
    r = rng.integers(0, 2 ** 32, size=shape, dtype=np.uint32)
    if cfg.noise_kind in (NOISE_UNIFORM_ICDF, NOISE_UNIFORM_CAT):
        k = (r >> np.uint32(9)).astype(np.float64)
        return ((k + 0.5) * 2.0 ** -23).astype(np.float32)
    u = (r.astype(np.float64) + 0.5) * 2.0 ** -32
    if cfg.noise_kind == NOISE_LOGISTIC:
        return (np.log(u) - np.log1p(-u)).astype(np.float32)
    if cfg.noise_kind == NOISE_GUMBEL:
        return (-np.log(-np.log(u))).astype(np.float32)
    raise ValueError("unknown noise kind")


def zero_init(cfg, batch: Optional[int] = None) -> np.ndarray:
    bt = cfg.batch if batch is None else batch
    return np.zeros((bt, cfg.D), dtype=np.uint8)


def random_init(cfg, batch: Optional[int] = None, salt: int = 0) -> np.ndarray:
    bt = cfg.batch if batch is None else batch
    n = 2 if cfg.C == 1 else cfg.C
    return _rng(cfg, 3, salt).integers(0, n, size=(bt, cfg.D), dtype=np.uint8)


def conv_weights(cfg: ConvConfig, salt: int = 0):
    """Unmasked convolution weights and zero biases.

    ``W[0]``: ``[ch, 3, 3, in_ch]``; ``W[1..layers-1]``: ``[ch, 3, 3, ch]``;
    ``W[layers]`` (1x1 head): ``[in_ch * C, ch]``.  He-style variance
    ``2 / fan_in`` with a nominal fan-in that needs no mask logic here: a causal
    3x3 kernel keeps four full taps plus about half of the centre tap, so
    ``fan_in = 4.5 * c_in``; the head sees about two thirds of its inputs and
    uses ``fan_in = (2/3) * ch``, without the ReLU factor (variance ``1/fan_in``).
    """
    rw = _rng(cfg, 0, salt)
    W, b = [], []
    c_in = cfg.in_ch
    for _ in range(cfg.layers):
        W.append(_normal(rw, (cfg.ch, 3, 3, c_in), 2.0 / (4.5 * c_in)))
        b.append(np.zeros((cfg.ch,), dtype=np.float32))
        c_in = cfg.ch
    W.append(_normal(rw, (cfg.in_ch * cfg.C, cfg.ch), 1.0 / (cfg.ch * 2.0 / 3.0)))
    b.append(np.zeros((cfg.in_ch * cfg.C,), dtype=np.float32))
    return W, b


def conv_lut(cfg: ConvConfig) -> np.ndarray:
    n = cfg.C
    return (np.arange(n, dtype=np.float64) / ((n - 1) / 2.0) - 1.0).astype(np.float32)


# ---------------------------------------------------------------- recurrent-network workload
@dataclass(frozen=True)
class RnnConfig:
    """Shape of the recurrent-network workload (back-propagation through time, Section 5.1)."""
    name: str
    index: int                 # fixes the seeds
    T: int = 100               # sequence length: a 10x10 image, one pixel per step
    H: int = 128               # hidden units
    d_in: int = 1
    d_out: int = 1
    batch: int = 1             # independent sequences
    w_std: float = 0.1         # weights ~ N(0, w_std^2), biases zero
    kind: str = "rnn"


# The paper trains on MNIST digits resized to 10x10 and fed pixel by pixel; seeded images of a few
# soft strokes on a 10x10 grid stand in for them (same length, same value range, same smoothness).
RNN_CONFIGS: Dict[str, RnnConfig] = {
    "rnn_small": RnnConfig("rnn_small", 10, T=12, H=16, batch=3),
    "rnn_100": RnnConfig("rnn_100", 11, T=100, H=128, batch=1),
    "rnn_100_batch": RnnConfig("rnn_100_batch", 12, T=100, H=128, batch=592),
}


def rnn_weights(cfg: RnnConfig):
    """(W_h [H,H], W_x [H,d_in], b [H], W_o [d_out,H], b_o [d_out]) as float32."""
    rng = _rng(cfg, 0)
    var = cfg.w_std * cfg.w_std
    Wh = _normal(rng, (cfg.H, cfg.H), var)
    Wx = _normal(rng, (cfg.H, cfg.d_in), var)
    Wo = _normal(rng, (cfg.d_out, cfg.H), var)
    return Wh, Wx, np.zeros(cfg.H, np.float32), Wo, np.zeros(cfg.d_out, np.float32)


def rnn_sequences(cfg: RnnConfig):
    """Inputs x [batch, T, d_in] in [0, 1] and targets r [batch, T, d_out] (the next input, zero after
    the last step), float32."""
    rng = _rng(cfg, 2)
    side = int(np.ceil(np.sqrt(cfg.T)))
    yy, xx = np.mgrid[0:side, 0:side].astype(np.float64)
    x = np.zeros((cfg.batch, cfg.T, cfg.d_in), np.float32)
    for b in range(cfg.batch):
        for c in range(cfg.d_in):
            img = np.zeros((side, side))
            for _ in range(3):                       # three soft strokes
                cy, cx = rng.uniform(min(1.0, side - 1.0), max(side - 2.0, min(1.0, side - 1.0)), size=2)
                sy, sx = rng.uniform(0.6, 2.0, size=2)
                img += np.exp(-0.5 * (((yy - cy) / sy) ** 2 + ((xx - cx) / sx) ** 2))
            img = np.clip(img, 0.0, 1.0)
            x[b, :, c] = img.reshape(-1)[:cfg.T].astype(np.float32)
    r = np.zeros((cfg.batch, cfg.T, cfg.d_out), np.float32)
    n = min(cfg.d_in, cfg.d_out)
    r[:, :-1, :n] = x[:, 1:, :n]
    return x, r
