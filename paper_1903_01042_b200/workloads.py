"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers (weights, inputs, targets, labels, generator
coefficients) and names the five benchmark configurations; it holds none of the method's
arithmetic, so both the CUDA path and the CPU checker can be fed from it.

The paper trains a 784-10^4-10^4-10 network on MNIST (Section "Experimental Results"); the
dataset is not available here, so inputs of the same shape and range stand in for it.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


def _rng(seed, stream):
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def bf16_round(a):
    """Round float32 values to the nearest bfloat16 (ties to even), returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def weights(n_out, n_in, seed=0, layer=0, bf16=False):
    """W ~ N(0, 1/n_in), float32 (optionally already bfloat16-representable)."""
    w = (_rng(seed, 100 + layer).standard_normal((n_out, n_in), dtype=np.float32)
         / np.float32(np.sqrt(n_in))).astype(np.float32)
    return bf16_round(w) if bf16 else w


def gaussian_inputs(batch, dim, seed=0, iteration=0):
    """x ~ N(0, 1)."""
    return _rng(seed, 1000 + iteration).standard_normal((batch, dim), dtype=np.float32)


def gaussian_targets(batch, dim, seed=0, iteration=0):
    """regression target ~ N(0, 1)."""
    return _rng(seed, 500000 + iteration).standard_normal((batch, dim), dtype=np.float32)


def uniform_inputs(batch, dim, seed=0, iteration=0):
    """Pixel-like inputs, uniform on [0, 1)."""
    return _rng(seed, 1000 + iteration).random((batch, dim), dtype=np.float32)


def labels(batch, n_classes, seed=0, iteration=0):
    return _rng(seed, 900000 + iteration).integers(0, n_classes, size=(batch,), dtype=np.int32)


COND_LIMIT = 1e3   # a drawn generator is kept when every erasure sub-system is better conditioned than this


def worst_condition(P):
    """Largest ||A||_inf ||A^-1||_inf over the square sub-systems A = P[F, Q]^T of a parity part P (k x r): the
    systems erasure decoding solves when the data outputs F are located and the parities Q are used."""
    import itertools
    P = np.asarray(P, np.float64)
    k, r = P.shape
    worst = 0.0
    for s in range(1, min(k, r) + 1):
        for F in itertools.combinations(range(k), s):
            for Q in itertools.combinations(range(r), s):
                A = P[np.ix_(F, Q)].T
                if abs(np.linalg.det(A)) == 0.0:
                    return float("inf")
                worst = max(worst, float(np.abs(A).sum(1).max() * np.abs(np.linalg.inv(A)).sum(1).max()))
    return worst


def gaussian_parity(k, r, seed=0, which=0):
    """Parity part P (k x r) of a systematic real generator [I | P], entries N(0, 1).  A draw with an erasure
    sub-system worse conditioned than COND_LIMIT is thrown away and the next stream of the same seed is drawn
    (a Gaussian matrix is MDS with probability one, but a draw can come arbitrarily close to a singular minor)."""
    for attempt in range(64):
        P = _rng(seed, 7000 + which + 100000 * attempt).standard_normal((k, r)).astype(np.float32)
        if r == 0 or worst_condition(P) <= COND_LIMIT:
            return P
    raise RuntimeError("no well-conditioned generator found")


def check_slice(length, slices=8):
    """Slice length for the inner checksums: the block side is cut into at most ``slices`` equal
    slices, so that a corrupted block output is tested by several independent sums."""
    for ns in range(min(slices, length), 0, -1):
        if length % ns == 0:
            return length // ns
    return length


@dataclass
class LayerSpec:
    n_out: int
    n_in: int
    m: int
    n: int
    r_row: int
    r_col: int
    gaussian_code: bool = False
    slices: int = 8       # inner-check slices per block side; slices x batch statistics test each node

    @property
    def check_rows(self):
        return check_slice(-(-self.n_out // self.m), self.slices)

    @property
    def check_cols(self):
        return check_slice(-(-self.n_in // self.n), self.slices)


@dataclass
class Config:
    name: str
    layers: List[LayerSpec]
    batch: int
    lr: float
    iterations: int
    bf16: bool = False
    activation: str = "identity"      # hidden-layer activation
    loss: str = "mse"                 # "mse" | "softmax_ce"
    inputs: str = "gaussian"          # "gaussian" | "uniform"
    fault_mode: str = "bernoulli"     # "bernoulli" | "exactly_one" | "none"
    p: float = 0.0
    sigma: float = 10.0
    seed: int = 0
    p_sweep: List[float] = field(default_factory=list)
    note: Optional[str] = None


def config(name, scale=1):
    """The five benchmark configurations and the paper's own network; ``scale`` divides every layer width (for checks that
    must finish quickly) while keeping the grid, the code and the batch."""
    s = int(scale)
    if name == "c1":
        return Config("c1", [LayerSpec(1024 // s, 1024 // s, 2, 2, 1, 1)], 1, 0.01, 100,
                      fault_mode="exactly_one")
    if name == "c2":
        return Config("c2", [LayerSpec(1000 // s, 784 // s, 4, 4, 1, 1),
                             LayerSpec(1000 // s, 1000 // s, 4, 4, 1, 1),
                             LayerSpec(10, 1000 // s, 4, 4, 1, 1)], 1, 0.01, 10000,
                      activation="relu", loss="softmax_ce", inputs="uniform", p=1e-3)
    if name == "c3":
        return Config("c3", [LayerSpec(8192 // s, 8192 // s, 8, 8, 1, 1)], 1, 0.01, 1000,
                      p=1e-3, p_sweep=[0.0, 1e-3, 1e-2])
    if name == "c4":
        # batch 128 already gives every node 128 independent inner-check statistics: one slice per side
        return Config("c4", [LayerSpec(16384 // s, 16384 // s, 8, 8, 2, 2, gaussian_code=True, slices=1)], 128,
                      0.01, 200, bf16=True, p=5e-3)
    if name == "c5":
        layers = [LayerSpec(4096 // s, 4096 // s, 4, 4, 1, 1, slices=1) for _ in range(8)]
        layers.append(LayerSpec(10, 4096 // s, 4, 4, 1, 1, slices=1))
        return Config("c5", layers, 64, 0.01, 2000, activation="relu", loss="softmax_ce", p=1e-3,
                      p_sweep=[0.0, 1e-4, 1e-3, 1e-2])
    if name == "paper":
        # The network of the paper's own experiment (Section "Experimental Results"): 784-10^4-10^4-10, SGD with
        # batch 1, every layer on a 5 x 4 data grid with 2 parity block-rows and 2 parity block-columns (the
        # non-square grid, 2000 x 196 / 2000 x 2500 / 2 x 2500 blocks), soft-error probability 3e-4 per node
        # and phase.  Two parities need a code beyond the checksum column: seeded Gaussian generators.
        # Inputs of MNIST's shape and range stand in for the dataset.
        return Config("paper", [LayerSpec(10000 // s, 784, 5, 4, 2, 2, gaussian_code=True),
                                LayerSpec(10000 // s, 10000 // s, 5, 4, 2, 2, gaussian_code=True),
                                LayerSpec(10, 10000 // s, 5, 4, 2, 2, gaussian_code=True)], 1, 0.01, 2000,
                      activation="relu", loss="softmax_ce", inputs="uniform", p=3e-4)
    raise KeyError(name)


def layer_inputs(cfg, iteration):
    """(X, target) for one iteration of ``cfg``."""
    n_in = cfg.layers[0].n_in
    n_last = cfg.layers[-1].n_out
    if cfg.inputs == "uniform":
        x = uniform_inputs(cfg.batch, n_in, cfg.seed, iteration)
    else:
        x = gaussian_inputs(cfg.batch, n_in, cfg.seed, iteration)
    if cfg.loss == "softmax_ce":
        t = labels(cfg.batch, n_last, cfg.seed, iteration)
    else:
        t = gaussian_targets(cfg.batch, n_last, cfg.seed, iteration)
    return x, t


def layer_codes(spec, seed=0, layer=0):
    """(P_row, P_col) for a layer: all-ones checksum columns, or seeded Gaussian ones."""
    if spec.gaussian_code:
        return (gaussian_parity(spec.m, spec.r_row, seed, 2 * layer),
                gaussian_parity(spec.n, spec.r_col, seed, 2 * layer + 1))
    return (np.ones((spec.m, spec.r_row), np.float32), np.ones((spec.n, spec.r_col), np.float32))
