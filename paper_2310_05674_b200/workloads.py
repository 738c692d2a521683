"""Seeded synthetic workloads for the SAMA meta-gradient step.

This module only draws random inputs. It holds none of the method's arithmetic
(no Adam Jacobian, no norm, no perturbation, no forward pass), so both the CUDA
path and the CPU checker can consume exactly the same bytes from it.

Every value is a pure function of ``(seed, stream, index)``: a 64-bit mixing
hash (the SplitMix64 finaliser) of the counter gives two 32-bit uniforms, and a
Box-Muller transform turns them into one standard normal.  Any slice of any
array can therefore be regenerated without storing or generating the rest.

Distribution notation: a scalar second argument of N(., .) is a standard
deviation (``theta ~ N(0, 0.02)`` is the usual 0.02-std initialiser);
``N(0, 4 I)`` is a covariance, i.e. std 2 per coordinate.

The workloads take the shapes of the settings the paper runs on (noisy-label
data reweighting with an MLP / classifier head, and flat parameter vectors of
BERT-base and RoBERTa-large size); they stand in for the paper's datasets and
pretrained weights, none of which is used.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)
_CHUNK = 1 << 21

# stream ids: one per logical array, so arrays never share counters
STREAM_THETA = 1
STREAM_M = 2
STREAM_S = 3
STREAM_GBASE = 4
STREAM_GMETA = 5
STREAM_X = 6
STREAM_LABEL = 7
STREAM_FLIP = 8
STREAM_FLIP_TO = 9
STREAM_LAMBDA = 10
STREAM_MEANS = 11
STREAM_REG_X = 12
STREAM_REG_XV = 13
STREAM_REG_W = 14
STREAM_REG_NOISE = 15
STREAM_REG_NOISE_V = 16
STREAM_REG_LAMBDA = 17


def _mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on a uint64 array (wraps modulo 2**64)."""
    z = (z ^ (z >> _U64(30))) * _M1
    z = (z ^ (z >> _U64(27))) * _M2
    return z ^ (z >> _U64(31))


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix64(np.array([(seed * 0x632BE59BD9B4E019 + stream * 0xD1342543DE82EF95 + 0x1234567) % (1 << 64)],
                            dtype=_U64))
    return k[0]


def _bits(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=_U64)
        return _mix64(_mix64(idx * _GOLDEN + _key(seed, stream)) + _GOLDEN)


def _uniform_chunk(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    b = _bits(seed, stream, start, count)
    return ((b >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_chunk(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    b = _bits(seed, stream, start, count)
    u1 = ((b >> _U64(32)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    u2 = ((b & _U64(0xFFFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * np.pi) * u2)


def _chunked(fn, seed: int, stream: int, n: int, offset: int, dtype) -> np.ndarray:
    out = np.empty(n, dtype=dtype)
    if n == 0:
        return out
    spans = [(s, min(_CHUNK, n - s)) for s in range(0, n, _CHUNK)]

    def work(span):
        s, c = span
        out[s:s + c] = fn(seed, stream, offset + s, c)

    if len(spans) == 1:
        work(spans[0])
    else:
        with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 8)) as ex:
            list(ex.map(work, spans))
    return out


def normal(seed: int, stream: int, n: int, offset: int = 0, dtype=np.float64) -> np.ndarray:
    """n standard normals: elements offset..offset+n-1 of stream ``stream``."""
    return _chunked(_normal_chunk, seed, stream, n, offset, dtype)


def uniform(seed: int, stream: int, n: int, offset: int = 0, dtype=np.float64) -> np.ndarray:
    """n uniforms in (0, 1)."""
    return _chunked(_uniform_chunk, seed, stream, n, offset, dtype)


# --------------------------------------------------------------------------
# Adam state and direct gradient (all fp32, length n)
# --------------------------------------------------------------------------

@dataclass
class AdamHyper:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    step: int = 100


def adam_state(n: int, seed: int) -> Dict[str, np.ndarray]:
    """m ~ N(0, std 1e-3); s = m^2 + 1e-6 |z|; g_meta ~ N(0, std 1e-2).

    g_base is a draw whose first two moments agree with (m, s):
    g_base = m + sqrt(s - m^2) z'.
    """
    m = (1e-3 * normal(seed, STREAM_M, n)).astype(np.float32)
    z = normal(seed, STREAM_S, n)
    spread = 1e-6 * np.abs(z)
    s = (m.astype(np.float64) ** 2 + spread).astype(np.float32)
    g_base = (m.astype(np.float64) + np.sqrt(spread) * normal(seed, STREAM_GBASE, n)).astype(np.float32)
    del z, spread
    g_meta = (1e-2 * normal(seed, STREAM_GMETA, n)).astype(np.float32)
    return {"m": m, "s": s, "g_base": g_base, "g_meta": g_meta}


# --------------------------------------------------------------------------
# Flat-vector workload (adapt + perturb sweep, no forward)
# --------------------------------------------------------------------------

def flat_vector(n: int, seed: int = 0) -> Dict[str, np.ndarray]:
    """theta ~ N(0, std 0.02) plus Adam state, all of length n."""
    out = adam_state(n, seed)
    out["theta"] = (0.02 * normal(seed, STREAM_THETA, n)).astype(np.float32)
    return out


# --------------------------------------------------------------------------
# MLP data-reweighting workloads
# --------------------------------------------------------------------------

@dataclass
class MLPConfig:
    name: str
    dims: Tuple[int, ...]
    batch: int
    noise_rate: float
    priors: Optional[Tuple[float, ...]] = None
    adam: AdamHyper = field(default_factory=AdamHyper)
    alpha: float = 1e-2

    @property
    def n_params(self) -> int:
        return sum(self.dims[l] * self.dims[l + 1] + self.dims[l + 1] for l in range(len(self.dims) - 1))

    @property
    def n_classes(self) -> int:
        return self.dims[-1]

    @property
    def forward_flops(self) -> int:
        """Multiply-adds of both branches counted as 2 flops each."""
        return 2 * 2 * self.batch * sum(self.dims[l] * self.dims[l + 1] for l in range(len(self.dims) - 1))


CONFIGS: Dict[str, MLPConfig] = {
    "tiny": MLPConfig("tiny", (784, 256, 10), 128, 0.40),
    "mlp3072": MLPConfig("mlp3072", (3072, 1024, 1024, 10), 512, 0.40),
    "head1024": MLPConfig("head1024", (1024, 1024, 4), 4096, 0.20, priors=(0.55, 0.25, 0.15, 0.05)),
    "wide4096": MLPConfig("wide4096", (4096, 4096, 4096, 1000), 2048, 0.40),
}

FLAT_SIZES: Dict[str, int] = {"flat110m": 110_000_000, "flat355m": 355_000_000}


def layer_offsets(dims: Sequence[int]) -> List[Tuple[int, int]]:
    """(weight offset, bias offset) of every layer in the flat vector.

    The flat vector is W1, b1, W2, b2, ... with W_l stored [d_l][d_{l-1}] row-major.
    """
    offs, o = [], 0
    for l in range(len(dims) - 1):
        w = o
        o += dims[l] * dims[l + 1]
        b = o
        o += dims[l + 1]
        offs.append((w, b))
    return offs


def kaiming_theta(dims: Sequence[int], seed: int) -> np.ndarray:
    """Kaiming-normal weights W ~ N(0, 2/fan_in), zero biases, flattened."""
    n = sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))
    theta = np.zeros(n, dtype=np.float32)
    for l, (w, b) in enumerate(layer_offsets(dims)):
        cnt = dims[l] * dims[l + 1]
        std = np.sqrt(2.0 / dims[l])
        theta[w:w + cnt] = (std * normal(seed, STREAM_THETA, cnt, offset=w)).astype(np.float32)
    return theta


def cluster_batch(d_in: int, n_classes: int, batch: int, noise_rate: float,
                  priors: Optional[Sequence[float]], seed: int) -> Dict[str, np.ndarray]:
    """Gaussian-cluster inputs with symmetric label noise.

    class means ~ N(0, 4 I); clean label from ``priors`` (uniform if None);
    x ~ N(mean[clean], I); with probability ``noise_rate`` the observed label is
    replaced by one drawn uniformly from the other n_classes-1 classes.
    """
    means = 2.0 * normal(seed, STREAM_MEANS, n_classes * d_in).reshape(n_classes, d_in)
    u = uniform(seed, STREAM_LABEL, batch)
    if priors is None:
        clean = np.minimum((u * n_classes).astype(np.int64), n_classes - 1)
    else:
        cdf = np.cumsum(np.asarray(priors, dtype=np.float64))
        cdf[-1] = 1.0
        clean = np.searchsorted(cdf, u, side="right").astype(np.int64)
        clean = np.minimum(clean, n_classes - 1)
    x = (means[clean] + normal(seed, STREAM_X, batch * d_in).reshape(batch, d_in)).astype(np.float32)
    flip = uniform(seed, STREAM_FLIP, batch) < noise_rate
    if n_classes > 1:
        shift = 1 + np.minimum((uniform(seed, STREAM_FLIP_TO, batch) * (n_classes - 1)).astype(np.int64),
                               n_classes - 2)
        noisy = np.where(flip, (clean + shift) % n_classes, clean)
    else:
        noisy = clean
    return {"X": np.ascontiguousarray(x), "y": noisy.astype(np.int32), "y_clean": clean.astype(np.int32)}


def mlp_workload(cfg: MLPConfig, seed: int = 0) -> Dict[str, np.ndarray]:
    """All inputs of one SAMA meta-gradient step for an MLP config."""
    n = cfg.n_params
    out = adam_state(n, seed)
    out["theta"] = kaiming_theta(cfg.dims, seed)
    out.update(cluster_batch(cfg.dims[0], cfg.n_classes, cfg.batch, cfg.noise_rate, cfg.priors, seed))
    out["lam"] = normal(seed, STREAM_LAMBDA, cfg.batch).astype(np.float32)
    return out


def custom_mlp(dims: Sequence[int], batch: int, seed: int, noise_rate: float = 0.4,
               name: str = "custom") -> Tuple[MLPConfig, Dict[str, np.ndarray]]:
    """A workload of arbitrary (e.g. ragged) shape with the same recipe."""
    cfg = MLPConfig(name, tuple(int(d) for d in dims), int(batch), noise_rate)
    return cfg, mlp_workload(cfg, seed)


# --------------------------------------------------------------------------
# Biased regression (the setting of the paper's Appendix E; its sizes are not stated there)
# --------------------------------------------------------------------------

@dataclass
class BiasRegConfig:
    name: str
    d: int          # features = dim(w) = dim(lambda)
    n: int          # base (training) samples
    n_val: int      # meta (validation) samples
    beta: float = 0.1
    noise: float = 0.1
    meta_updates: int = 100


BIASREG: Dict[str, BiasRegConfig] = {
    "biasreg256": BiasRegConfig("biasreg256", 256, 512, 512),
    "biasreg4096": BiasRegConfig("biasreg4096", 4096, 8192, 8192),
}


def biased_regression(cfg: BiasRegConfig, seed: int = 0) -> Dict[str, np.ndarray]:
    """X, X' ~ N(0, 1) entrywise scaled by 1/sqrt(d); y = X w_true + noise z, y' = X' w_true + noise z';
    w_true ~ N(0, 1); lambda_0 ~ N(0, 1).  All fp32."""
    d, n, nv = cfg.d, cfg.n, cfg.n_val
    sc = 1.0 / np.sqrt(d)
    X = (sc * normal(seed, STREAM_REG_X, n * d)).astype(np.float32).reshape(n, d)
    Xv = (sc * normal(seed, STREAM_REG_XV, nv * d)).astype(np.float32).reshape(nv, d)
    w_true = normal(seed, STREAM_REG_W, d)
    y = (X.astype(np.float64) @ w_true + cfg.noise * normal(seed, STREAM_REG_NOISE, n)).astype(np.float32)
    yv = (Xv.astype(np.float64) @ w_true + cfg.noise * normal(seed, STREAM_REG_NOISE_V, nv)).astype(np.float32)
    lam0 = normal(seed, STREAM_REG_LAMBDA, d).astype(np.float32)
    return {"X": X, "y": y, "Xv": Xv, "yv": yv, "lam0": lam0, "w_true": w_true.astype(np.float32)}
