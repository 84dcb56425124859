"""Seeded synthetic workloads shaped like the paper's WSJ1 / AMI hybrid DNNs.

This module only *draws numbers*: it holds none of the method's arithmetic (no Sign, no
packing of activations, no dot products) so that the CPU oracle and the CUDA path can both
be fed from it without sharing any code of the method.

The paper (Section 3) uses feed-forward nets with 6 hidden layers of 1024 or 2048 units on
11-frame splices of 40-dim filterbank features, with 3307 (WSJ1) / 3972 (AMI) tied-state
outputs.  The corpora and trained weights are not available, so the shapes below stand in
for them with iid values.

Draw order for a model (one ``numpy.random.Generator(PCG64(seed))``):
  for each hidden layer l = 1..L:  W_l, scale_l, shift_l   then   Wout, bout.
Frames use an independent generator ``PCG64([seed, 0x5eed])`` so that any number of frames
can be drawn without touching the model stream.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# Activation kinds of a hidden layer (values mirror include/bnn.h).
ACT_SIGN = 1       # h = Sign(affine(.)), 1-bit output
ACT_HARDTANH = 2   # h = clamp(affine(.), -1, 1), fp32 output


@dataclass(frozen=True)
class Config:
    name: str
    seed: int
    frames: int          # M
    in_dim: int          # K0: spliced feature dimension
    hidden: int          # H
    n_hidden: int        # number of hidden layers (first one reads real input)
    classes: int         # C
    act: int = ACT_SIGN  # hidden activation
    per_layer_alpha: bool = False  # binary-weights-only variant: scale = alpha_l, shift = 0
    mixed: bool = False  # the paper's most accurate topology (Table 2): real-valued Sigmoid first layer,
                         # binary layers with Sign units in between, binary last hidden layer with Sigmoid units


CONFIGS = {
    # tiny: 440 -> 1024 -> 1024 -> 1024 -> 2000
    "tiny": Config("tiny", 0, 256, 440, 1024, 3, 2000),
    # WSJ-scale: 440 -> 6 x 2048 -> 3400
    "wsj": Config("wsj", 1, 8192, 440, 2048, 6, 3400),
    # binary weights only, real activations (hardtanh), same shape
    "wsj_bw": Config("wsj_bw", 2, 8192, 440, 2048, 6, 3400, ACT_HARDTANH, True),
    # AMI-scale: 600 -> 6 x 3072 -> 4000
    "ami": Config("ami", 3, 65536, 600, 3072, 6, 4000),
    # mixed topology at the WSJ shape (sigma, b, b, b, b, sigma, softmax); first-layer weights ~ N(0, 1/K)
    "wsj_mixed": Config("wsj_mixed", 5, 8192, 440, 2048, 6, 3400, mixed=True),
}

# Isolated XNOR GEMM sweep.
SWEEP_SEED = 4
SWEEP_M = (256, 4096, 65536)
SWEEP_K = (1024, 2048, 4096, 8192)
SWEEP_N = (1024, 2048, 4096, 8192)
SWEEP_P = (0.5, 0.1)


@dataclass
class Model:
    cfg: Config
    W: list = field(default_factory=list)      # fp32 [N_l][K_l], real-valued, sign iid +-1
    scale: list = field(default_factory=list)  # fp32 [N_l]
    shift: list = field(default_factory=list)  # fp32 [N_l]
    Wout: np.ndarray = None                    # fp32 [C][H]
    bout: np.ndarray = None                    # fp32 [C]


def _signed_weights(rng: np.random.Generator, n: int, k: int) -> np.ndarray:
    """Real-valued weights whose sign is iid +-1 with p = 0.5 and |w| in [0.1, 1)."""
    mag = rng.uniform(0.1, 1.0, size=(n, k)).astype(np.float32)
    neg = rng.integers(0, 2, size=(n, k), dtype=np.uint8).astype(bool)
    np.negative(mag, where=neg, out=mag)
    return mag


def make_model(cfg: Config, seed: int | None = None) -> Model:
    rng = np.random.Generator(np.random.PCG64(cfg.seed if seed is None else seed))
    m = Model(cfg)
    k = cfg.in_dim
    for l in range(cfg.n_hidden):
        if cfg.mixed and l == 0:   # real-valued layer: weights and a bias (Eq. 1), no scale
            m.W.append(rng.normal(0.0, 1.0 / np.sqrt(k), size=(cfg.hidden, k)).astype(np.float32))
            m.scale.append(None)
            m.shift.append(rng.normal(0.0, 0.1, size=cfg.hidden).astype(np.float32))
            k = cfg.hidden
            continue
        m.W.append(_signed_weights(rng, cfg.hidden, k))
        if cfg.per_layer_alpha:
            alpha = np.float32(rng.uniform(0.01, 0.1))
            m.scale.append(np.full(cfg.hidden, alpha, dtype=np.float32))
            m.shift.append(np.zeros(cfg.hidden, dtype=np.float32))
        else:
            m.scale.append(rng.uniform(0.5, 1.5, size=cfg.hidden).astype(np.float32))
            m.shift.append(rng.normal(0.0, 0.1, size=cfg.hidden).astype(np.float32))
        k = cfg.hidden
    m.Wout = rng.normal(0.0, 1.0 / np.sqrt(cfg.hidden),
                        size=(cfg.classes, cfg.hidden)).astype(np.float32)
    m.bout = rng.normal(0.0, 0.1, size=cfg.classes).astype(np.float32)
    return m


def make_frames(cfg: Config, frames: int | None = None, seed: int | None = None) -> np.ndarray:
    """fp32 [frames][in_dim], iid N(0,1): stands in for spliced filterbank features."""
    s = cfg.seed if seed is None else seed
    rng = np.random.Generator(np.random.PCG64([s, 0x5EED]))
    n = cfg.frames if frames is None else frames
    return rng.standard_normal(size=(n, cfg.in_dim), dtype=np.float32)


def sweep_point_seed(m: int, k: int, n: int, p: float) -> list:
    return [SWEEP_SEED, m, k, n, int(round(p * 1000))]


def make_bit_matrix(rows: int, k: int, p: float, seed) -> np.ndarray:
    """uint8 [rows][k] of iid Bernoulli(p) bits (1 stands for +1, 0 for -1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if p == 0.5:
        return rng.integers(0, 2, size=(rows, k), dtype=np.uint8)
    return (rng.random(size=(rows, k), dtype=np.float32) < np.float32(p)).astype(np.uint8)


def make_bit_planes(rows: int, k: int, p: float, seed, pitch_words: int | None = None) -> np.ndarray:
    """Packed uint32 bit-planes [rows][pitch_words] of iid Bernoulli(p) bits.

    The sweep's inputs are *defined* as packed planes: element k of a row is bit k%32 of
    word k//32; bits at positions >= k and pitch words beyond ceil(k/32) are zero.
    For p = 0.5 whole random words are drawn (fast enough for 65536 x 8192).
    """
    kw = (k + 31) // 32
    pw = kw if pitch_words is None else pitch_words
    rng = np.random.Generator(np.random.PCG64(seed))
    out = np.zeros((rows, pw), dtype=np.uint32)
    if p == 0.5:
        out[:, :kw] = rng.integers(0, 2**32, size=(rows, kw), dtype=np.uint32)
    else:
        acc = np.zeros((rows, kw), dtype=np.uint32)
        for b in range(32):
            hit = rng.random(size=(rows, kw), dtype=np.float32) < np.float32(p)
            acc |= hit.astype(np.uint32) << np.uint32(b)
        out[:, :kw] = acc
    tail = k % 32
    if tail:
        out[:, kw - 1] &= np.uint32((1 << tail) - 1)
    return out
