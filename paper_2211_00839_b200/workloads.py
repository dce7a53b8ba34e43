"""Seeded synthetic inputs for the resource-constrained submodular partition.

This module only draws random feature matrices, labels and capacity vectors.
It holds none of the method's arithmetic (no similarity, no objective, no
greedy step), so both the CUDA library's tests and the CPU oracle's tests can
take their inputs from it without sharing any code of the method itself.

The paper evaluates on CIFAR-10 / CIFAR-100 features taken from an
auto-encoder bottleneck (Section 4, item 1).  Those datasets are not used
here: every workload below is a synthetic stand-in with the same shape
(classes x samples per class x feature width), drawn from a per-class
Gaussian mixture so that the similarity matrix has the block structure that
real clustered features give (dense same-component blocks, near-zero and
negative cross-component entries, dominant diagonal).

Feature storage
---------------
``int8``  : ``numpy.int8``  array ``[N, d]``.
``bf16``  : ``numpy.uint16`` array ``[N, d]`` holding bfloat16 bit patterns
            (rows L2-normalised in fp32, then rounded to nearest-even).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

__all__ = ["Workload", "CONFIGS", "make_workload", "make_mixture", "fp32_to_bf16_bits",
           "bf16_bits_to_fp32"]


def fp32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bfloat16 (round-to-nearest-even); return the 16-bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return u.astype(np.uint16)


def bf16_bits_to_fp32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to fp32 (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    name: str
    dtype: str                 # "int8" or "bf16"
    features: np.ndarray       # [N, d] int8, or uint16 bf16 bit patterns
    labels: np.ndarray         # [N] int32, values in [0, L)
    capacities: np.ndarray     # [W] float64, > 0
    L: int
    W: int

    @property
    def N(self) -> int:
        return int(self.features.shape[0])

    @property
    def d(self) -> int:
        return int(self.features.shape[1])


# name -> recipe.  ``law``: "gauss" draws x = mu_k + eps ; "relu" draws x = |mu_k + eps|.
CONFIGS: Dict[str, dict] = {
    # 2 classes x 200, int8 d=64, 3 equal-weight components, W=4 capacities 1:1:2:4
    "C1": dict(seed=0, L=2, M=200, d=64, dtype="int8", K=3, weights="equal", law="gauss",
               mean_std=4.0, caps="list", caps_list=[1, 1, 2, 4]),
    # CIFAR-10-shaped exact
    "C2": dict(seed=1, L=10, M=5000, d=512, dtype="int8", K=8, weights="dirichlet", law="gauss",
               mean_std=4.0, caps="list", caps_list=[1, 1, 1, 1, 2, 2, 4, 4]),
    # CIFAR-10-shaped float
    "C3": dict(seed=2, L=10, M=5000, d=512, dtype="bf16", K=8, weights="dirichlet", law="gauss",
               mean_std=4.0, caps="uniform_half", W=16),
    # CIFAR-100-shaped
    "C4": dict(seed=3, L=100, M=500, d=2048, dtype="bf16", K=4, weights="dirichlet", law="relu",
               mean_std=1.0, caps="loguniform8", W=32),
    # ImageNet-shaped
    "C5": dict(seed=4, L=1000, M=1300, d=2048, dtype="int8", K=16, weights="dirichlet", law="gauss",
               mean_std=4.0, caps="tiers", W=64),
}


def make_mixture(rng: np.random.Generator, M: int, d: int, K: int, weights: str, law: str,
                 mean_std: float) -> np.ndarray:
    """One class: ``M`` fp32 samples from a ``K``-component mixture in ``d`` dimensions."""
    mu = (rng.standard_normal((K, d), dtype=np.float32) * np.float32(mean_std))
    if weights == "equal":
        w = np.full(K, 1.0 / K)
    elif weights == "dirichlet":
        w = rng.dirichlet(np.ones(K))
    else:
        raise ValueError(weights)
    comp = rng.choice(K, size=M, p=w)
    x = mu[comp] + rng.standard_normal((M, d), dtype=np.float32)
    if law == "relu":
        x = np.abs(x)
    elif law != "gauss":
        raise ValueError(law)
    return x


def _capacities(rng: np.random.Generator, spec: dict) -> np.ndarray:
    kind = spec["caps"]
    if kind == "list":
        return np.asarray(spec["caps_list"], dtype=np.float64)
    W = spec["W"]
    if kind == "uniform_half":       # uniform on [1,4], rounded to the nearest 0.5
        return np.round(rng.uniform(1.0, 4.0, size=W) * 2.0) / 2.0
    if kind == "loguniform8":        # log-uniform over [1,8]
        return np.exp(rng.uniform(0.0, 1.0, size=W) * np.log(8.0))
    if kind == "tiers":              # four equal tiers 1:2:4:8
        return np.asarray([2.0 ** (j // (W // 4)) for j in range(W)], dtype=np.float64)
    raise ValueError(kind)


def make_workload(name: str, L: Optional[int] = None, M: Optional[int] = None,
                  d: Optional[int] = None, seed: Optional[int] = None,
                  shuffle: bool = True) -> Workload:
    """Build a named workload; ``L``/``M``/``d``/``seed`` override the recipe (reduced cases).

    Samples are generated class by class, then (with ``shuffle``) the sample
    order is permuted by the same generator so labels arrive interleaved, as a
    dataset's would.
    """
    spec = dict(CONFIGS[name])
    L = spec["L"] if L is None else int(L)
    M = spec["M"] if M is None else int(M)
    d = spec["d"] if d is None else int(d)
    seed = spec["seed"] if seed is None else int(seed)
    rng = np.random.default_rng(seed)
    caps = _capacities(rng, spec)
    W = len(caps)
    N = L * M
    if spec["dtype"] == "int8":
        feats = np.empty((N, d), dtype=np.int8)
    else:
        feats = np.empty((N, d), dtype=np.uint16)
    labels = np.repeat(np.arange(L, dtype=np.int32), M)
    for l in range(L):
        x = make_mixture(rng, M, d, spec["K"], spec["weights"], spec["law"], spec["mean_std"])
        if spec["dtype"] == "int8":
            feats[l * M:(l + 1) * M] = np.clip(np.rint(x), -127, 127).astype(np.int8)
        else:
            nrm = np.sqrt((x.astype(np.float32) ** 2).sum(axis=1, keepdims=True, dtype=np.float32))
            x = (x / np.maximum(nrm, np.float32(1e-30))).astype(np.float32)
            feats[l * M:(l + 1) * M] = fp32_to_bf16_bits(x)
    if shuffle:
        perm = rng.permutation(N)
        feats = np.ascontiguousarray(feats[perm])
        labels = np.ascontiguousarray(labels[perm])
    return Workload(name=name, dtype=spec["dtype"], features=feats, labels=labels,
                    capacities=caps, L=L, W=W)
