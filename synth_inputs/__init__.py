"""Seeded synthetic inputs for Parle rounds.

This module produces *data only*: initial replica parameters, minibatches,
teacher labels and the named workload configurations.  It holds none of the
method's arithmetic (no gradient, no update rule) and imports neither the CPU
oracle nor the CUDA library; both of those consume the arrays made here.

Random numbers come from a counter-based generator: a 64-bit mixing function
(the SplitMix64 finaliser) applied to ``key + counter * odd_constant``, mapped
to uniforms on (0,1) with 53 random bits and to normals by the Box-Muller
transform.  Every tensor is addressed by (seed, tensor tag, integer words...)
so any tensor of any round/step/replica can be regenerated on its own.

The paper trains on MNIST, CIFAR-10/100 and SVHN (Section 4); those datasets
are not reproduced here.  The generators below only borrow their *shapes*
(28x28 pixels in [0,1], 32x32x3 standardised inputs, 10/100 classes) and draw
every value at random; labels come from a fixed seeded random teacher.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Sequence, Tuple

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)
_MASK = (1 << 64) - 1


def _mix64_int(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def _mix64(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        return z ^ (z >> _U64(31))


# tensor tags (first word of every stream key)
TAG_PARAM_W = 1
TAG_INPUT = 2
TAG_TEACHER = 3
TAG_GRAD = 4
TAG_STATE = 5
TAG_QUAD = 6
TAG_DATASET = 7
TAG_INDEX = 8


def stream_key(seed: int, *words: int) -> int:
    """Fold (seed, words...) into one 64-bit key."""
    k = _mix64_int(seed ^ 0x5851F42D4C957F2D)
    for w in words:
        k = _mix64_int(k ^ _mix64_int((int(w) + 0x632BE59BD9B4E019) & _MASK))
    return k


def raw_u64(key: int, count: int, start: int = 0) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=_U64)
    with np.errstate(over="ignore"):
        return _mix64(_U64(key) + (idx + _U64(1)) * _GOLDEN)


def uniform01(key: int, count: int, start: int = 0) -> np.ndarray:
    """fp64 uniforms strictly inside (0,1)."""
    r = raw_u64(key, count, start)
    return ((r >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal01(key: int, count: int) -> np.ndarray:
    """fp64 standard normals (Box-Muller on consecutive counter pairs)."""
    pairs = (count + 1) // 2
    out = np.empty(2 * pairs, dtype=np.float64)
    chunk = 1 << 22
    for p0 in range(0, pairs, chunk):
        p1 = min(pairs, p0 + chunk)
        u = uniform01(key, 2 * (p1 - p0), 2 * p0)
        r = np.sqrt(-2.0 * np.log(u[0::2]))
        t = (2.0 * np.pi) * u[1::2]
        out[2 * p0:2 * p1:2] = r * np.cos(t)
        out[2 * p0 + 1:2 * p1:2] = r * np.sin(t)
    return out[:count]


def normal_f32(key: int, shape: Sequence[int], std: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape)) if len(shape) else 1
    return (normal01(key, n) * std).astype(np.float32).reshape(shape)


def uniform_f32(key: int, shape: Sequence[int]) -> np.ndarray:
    n = int(np.prod(shape)) if len(shape) else 1
    return uniform01(key, n).astype(np.float32).reshape(shape)


# --------------------------------------------------------------------------
# Workload configurations
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class ParleConfig:
    name: str
    n: int                      # replicas
    dims: Tuple[int, ...]       # d_0 ... d_last
    batch: int
    L: int                      # inner steps per round
    rounds: int
    gemm_dtype: int = 0         # 0: fp32 operands, 1: bf16 operands / fp32 accumulate
    eta: float = 0.1
    eta_prime: float = 0.1
    alpha: float = 0.75
    gamma: float = 1.0
    rho: float = 1.0
    input_dist: str = "normal"  # "normal": N(0,1); "uniform": U[0,1]
    teacher: Tuple[int, ...] = ()   # hidden widths of the teacher (empty: linear)
    seed: int = 1707_00424

    @property
    def n_layers(self) -> int:
        return len(self.dims) - 1

    @property
    def n_params(self) -> int:
        return sum(self.dims[l + 1] * self.dims[l] + self.dims[l + 1] for l in range(self.n_layers))

    def scaled(self, **kw) -> "ParleConfig":
        return replace(self, **kw)


# The five workloads, in the order they are usually quoted (C1..C5; C4 is the
# update-kernel sweep and has its own helper below).
C1 = ParleConfig("C1", n=3, dims=(64, 32, 10), batch=16, L=5, rounds=2)
C2 = ParleConfig("C2", n=8, dims=(784, 1024, 1024, 10), batch=128, L=25, rounds=4,
                 input_dist="uniform", teacher=(256,))
C3 = ParleConfig("C3", n=8, dims=(3072, 2048, 2048, 2048, 100), batch=128, L=25, rounds=4,
                 gemm_dtype=1)
C5 = ParleConfig("C5", n=16, dims=(4096, 8192, 8192, 8192, 8192, 1000), batch=256, L=25,
                 rounds=2, gemm_dtype=1)
CONFIGS = {"C1": C1, "C2": C2, "C3": C3, "C5": C5}

SWEEP_D = (1 << 20, 1 << 24, 1 << 26, 1 << 28)
SWEEP_N = (3, 8, 16)


# --------------------------------------------------------------------------
# Parameters, minibatches, labels
# --------------------------------------------------------------------------

def init_layer(cfg: ParleConfig, replica: int, layer: int, fast: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Initial W_l ~ N(0, 1/fan_in) as [d_l, d_{l-1}] fp32 and b_l = 0.

    fast=True draws the same distribution from numpy's Philox bit generator keyed by the
    same stream key (about 20x quicker; for the 243 M-parameter workload)."""
    d_in, d_out = cfg.dims[layer], cfg.dims[layer + 1]
    key = stream_key(cfg.seed, TAG_PARAM_W, replica, layer)
    if fast:
        rng = np.random.Generator(np.random.Philox(key=key))
        W = rng.standard_normal((d_out, d_in), dtype=np.float32)
        W *= np.float32(d_in ** -0.5)
    else:
        W = normal_f32(key, (d_out, d_in), std=d_in ** -0.5)
    b = np.zeros(d_out, dtype=np.float32)
    return W, b


def init_replica(cfg: ParleConfig, replica: int, fast: bool = False) -> List[Tuple[np.ndarray, np.ndarray]]:
    return [init_layer(cfg, replica, l, fast) for l in range(cfg.n_layers)]


def _teacher_weights(cfg: ParleConfig) -> List[np.ndarray]:
    widths = (cfg.dims[0],) + tuple(cfg.teacher) + (cfg.dims[-1],)
    Ws = []
    for l in range(len(widths) - 1):
        key = stream_key(cfg.seed, TAG_TEACHER, l)
        std = 1.0 if not cfg.teacher else widths[l] ** -0.5
        Ws.append(normal01(key, widths[l] * widths[l + 1]).reshape(widths[l], widths[l + 1]) * std)
    return Ws


def teacher_labels(cfg: ParleConfig, X: np.ndarray) -> np.ndarray:
    """Labels = argmax of the fixed seeded teacher on X (ties: lowest index)."""
    h = X.astype(np.float64)
    if cfg.input_dist == "uniform":
        h = h - 0.5        # centre the pixels so that the classes are not degenerate
    Ws = _teacher_weights(cfg)
    for i, W in enumerate(Ws):
        h = h @ W
        if i + 1 < len(Ws):
            h = np.maximum(h, 0.0)
    return np.argmax(h, axis=-1).astype(np.int32)


def minibatch(cfg: ParleConfig, replica: int, rnd: int, step: int,
              shared: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Minibatch of replica `replica` at inner step `step` of round `rnd`.

    Returns X [batch, d_0] fp32 and labels [batch] int32.  With shared=True
    every replica gets replica 0's batch.
    """
    a = 0 if shared else replica
    key = stream_key(cfg.seed, TAG_INPUT, a, rnd, step)
    shape = (cfg.batch, cfg.dims[0])
    X = uniform_f32(key, shape) if cfg.input_dist == "uniform" else normal_f32(key, shape)
    return X, teacher_labels(cfg, X)


def round_batches(cfg: ParleConfig, rnd: int, shared: bool = False, pool: int = 0):
    """X [L, n, batch, d_0] fp32 and labels [L, n, batch] int32 for one round.

    pool > 0: only `pool` distinct inner steps are drawn and cycled through the L steps
    (for the largest workload, where a round of fresh minibatches is gigabytes)."""
    X = np.empty((cfg.L, cfg.n, cfg.batch, cfg.dims[0]), dtype=np.float32)
    c = np.empty((cfg.L, cfg.n, cfg.batch), dtype=np.int32)
    for l in range(cfg.L):
        if pool and l >= pool:
            X[l], c[l] = X[l % pool], c[l % pool]
            continue
        for a in range(cfg.n):
            X[l, a], c[l, a] = minibatch(cfg, a, rnd, l, shared)
    return X, c


# --------------------------------------------------------------------------
# Update-kernel sweep inputs (flat parameter vectors, no network)
# --------------------------------------------------------------------------

def sweep_state(seed: int, n: int, d: int):
    """x, y, z [n, d] ~ N(0,1) and g [n, d] ~ N(0, 1e-2) (variance; std 0.1), fp32."""
    def one(tag, std):
        out = np.empty((n, d), dtype=np.float32)
        for a in range(n):
            out[a] = normal_f32(stream_key(seed, TAG_STATE, tag, a), (d,), std)
        return out
    x = one(0, 1.0)
    y = one(1, 1.0)
    z = one(2, 1.0)
    g = np.empty((n, d), dtype=np.float32)
    for a in range(n):
        g[a] = normal_f32(stream_key(seed, TAG_GRAD, a), (d,), 0.1)
    return x, y, z, g


def quadratic_spectrum(seed: int, d: int, lo: float = 0.05, hi: float = 2.0) -> np.ndarray:
    """Eigenvalues of a diagonal positive quadratic loss, uniform on [lo, hi]."""
    u = uniform01(stream_key(seed, TAG_QUAD), d)
    return lo + (hi - lo) * u


# --------------------------------------------------------------------------
# A finite synthetic dataset and its split between replicas (Section 5 of the paper:
# the dataset xi is the union of shards xi^a and replica a samples minibatches from xi^a only)
# --------------------------------------------------------------------------

def dataset_sample(cfg: ParleConfig, index: int) -> np.ndarray:
    """Sample `index` of the dataset: d_0 values drawn from the config's input distribution."""
    key = stream_key(cfg.seed, TAG_DATASET, index)
    d = cfg.dims[0]
    return uniform_f32(key, (d,)) if cfg.input_dist == "uniform" else normal_f32(key, (d,))


def shard_bounds(dataset_size: int, n: int, replica: int) -> Tuple[int, int]:
    """Half-open index range of shard `replica` when the dataset is cut into n contiguous shards."""
    return replica * dataset_size // n, (replica + 1) * dataset_size // n


def dataset_minibatch_indices(cfg: ParleConfig, replica: int, rnd: int, step: int,
                              dataset_size: int, split: bool) -> np.ndarray:
    """Indices (with replacement) of the minibatch of `replica` at (rnd, step): from its own shard when
    `split`, from the whole dataset otherwise."""
    lo, hi = shard_bounds(dataset_size, cfg.n, replica) if split else (0, dataset_size)
    u = uniform01(stream_key(cfg.seed, TAG_INDEX, replica, rnd, step), cfg.batch)
    return lo + np.minimum((u * (hi - lo)).astype(np.int64), hi - lo - 1)


def dataset_round_batches(cfg: ParleConfig, rnd: int, dataset_size: int, split: bool):
    """X [L, n, batch, d_0], labels [L, n, batch] and the sample indices [L, n, batch] of one round."""
    X = np.empty((cfg.L, cfg.n, cfg.batch, cfg.dims[0]), dtype=np.float32)
    idx = np.empty((cfg.L, cfg.n, cfg.batch), dtype=np.int64)
    cache = {}
    for l in range(cfg.L):
        for a in range(cfg.n):
            idx[l, a] = dataset_minibatch_indices(cfg, a, rnd, l, dataset_size, split)
            for i, k in enumerate(idx[l, a]):
                if k not in cache:
                    cache[k] = dataset_sample(cfg, int(k))
                X[l, a, i] = cache[k]
    c = teacher_labels(cfg, X.reshape(-1, cfg.dims[0])).reshape(cfg.L, cfg.n, cfg.batch)
    return X, c, idx
