"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers: it holds none of the method's arithmetic, so both
the CUDA path and the CPU oracle can be fed from it without sharing any code that
matters.  The paper measures on LongBench prompts through ChatGLM2-6B-32k
(n = 32768) and on a synthetic single-layer benchmark (Sec. 4.2, d = 64,
n = 4096 .. 131072, b = m = 256, causal recursion down to 4096); neither dataset nor
weights are available, so i.i.d. / clustered / heavy-tailed stand-ins of the same
shapes are used.

bf16 tensors are carried as uint16 bit patterns so both sides read identical values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One configuration of the forward pass (paper notation: b block, m samples, r bits)."""
    name: str
    B: int
    H: int
    n: int
    d: int
    dtype: str          # "bf16" or "fp32"
    b: int
    m: int
    r: int
    causal: bool
    n0: int
    kind: str           # "gaussian" | "clustered" | "student_t" | "ramp"
    gen_seed: int
    seed: int = 0       # the library's seed (hash directions and sampled columns)
    n_k: int = 0        # rows of K and V when they differ from n (0: n)

    @property
    def G(self) -> int:
        return self.B * self.H

    @property
    def nk(self) -> int:
        return self.n_k or self.n

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (index = position in the baseline's config list).
CONFIGS = [
    Workload("c1_n1024_fp32", 1, 1, 1024, 64, "fp32", 128, 128, 7, False, 0, "gaussian", 1000),
    Workload("c2_n32k_d128", 1, 32, 32768, 128, "bf16", 256, 256, 7, False, 0, "gaussian", 1001),
    Workload("c3_n131k_causal", 1, 32, 131072, 64, "bf16", 256, 256, 7, True, 4096, "gaussian", 1002),
    Workload("c4_clustered", 1, 32, 131072, 64, "bf16", 256, 256, 7, False, 0, "clustered", 1003),
    Workload("c5_heavy_tail_causal", 4, 32, 16384, 128, "bf16", 128, 512, 8, True, 2048, "student_t", 1004),
]


def _gaussian(rng, G, n, d):
    return [rng.standard_normal((G, n, d), dtype=np.float32) for _ in range(3)]


def _clustered(rng, G, n, d, centres=64, noise=0.1, q_gain=3.0):
    """Per segment: 64 Gaussian centres; key = its centre + noise, query = 3 x its centre
    + noise (cluster assignment i.i.d. uniform), values i.i.d. N(0,1).  Plants large
    attention entries for the LSH to find and many equal bucket ids for the sort."""
    Q = np.empty((G, n, d), dtype=np.float32)
    K = np.empty((G, n, d), dtype=np.float32)
    for g in range(G):
        c = rng.standard_normal((centres, d), dtype=np.float32)
        aq = rng.integers(0, centres, size=n)
        ak = rng.integers(0, centres, size=n)
        Q[g] = q_gain * c[aq] + noise * rng.standard_normal((n, d), dtype=np.float32)
        K[g] = c[ak] + noise * rng.standard_normal((n, d), dtype=np.float32)
    V = rng.standard_normal((G, n, d), dtype=np.float32)
    return [Q, K, V]


def _student_t(rng, G, n, d, dof=3.0, clip=20.0):
    return [np.clip(rng.standard_t(dof, size=(G, n, d)), -clip, clip).astype(np.float32) for _ in range(3)]


def _ramp(rng, G, n, d):
    """Logits that keep growing along the key index: every query is close to one direction u,
    key j is (j / n) * 24 * sqrt(d) * u plus noise, so the row maxima found while walking the
    keys in index order rise by hundreds of octaves - a stress case for running-maximum bookkeeping.  Test input
    only; not one of the paper's workloads."""
    u = rng.standard_normal((G, 1, d)).astype(np.float32)
    u /= np.linalg.norm(u, axis=2, keepdims=True)
    q = (u * np.sqrt(d) * 3.0 + 0.3 * rng.standard_normal((G, n, d))).astype(np.float32)
    ramp = (np.arange(n, dtype=np.float32) / n)[None, :, None]
    k = (u * ramp * 24.0 * np.sqrt(d) + 0.3 * rng.standard_normal((G, n, d))).astype(np.float32)
    v = rng.standard_normal((G, n, d)).astype(np.float32)
    return [q, k, v]


def make_inputs(w: Workload):
    """Returns Q (G, n, d) and K, V (G, n_k, d) as numpy arrays: float32 for "fp32" workloads,
    uint16 bf16 bit patterns for "bf16" workloads."""
    rng = np.random.Generator(np.random.PCG64(w.gen_seed))
    gen = {"gaussian": _gaussian, "clustered": _clustered, "student_t": _student_t, "ramp": _ramp}[w.kind]
    if w.nk != w.n:
        # unequal sides: draw max(n, n_k) rows of everything and keep the first n / n_k of each
        big = gen(rng, w.G, max(w.n, w.nk), w.d)
        qkv = [np.ascontiguousarray(big[0][:, :w.n]), np.ascontiguousarray(big[1][:, :w.nk]), np.ascontiguousarray(big[2][:, :w.nk])]
    else:
        qkv = gen(rng, w.G, w.n, w.d)
    if w.dtype == "bf16":
        return [f32_to_bf16_bits(x) for x in qkv]
    return qkv


def as_f64(x: np.ndarray) -> np.ndarray:
    """The exact real values of an input array, widened to fp64."""
    if x.dtype == np.uint16:
        return bf16_bits_to_f32(x).astype(np.float64)
    return x.astype(np.float64)
