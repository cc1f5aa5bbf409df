"""Seeded synthetic inputs for the thresholded all-pairs similarity join.

This module only *draws inputs*: point sets P (n x d) and Q (m x d), planted
near pairs and cluster labels.  It holds none of the join's arithmetic (no
scores, no thresholds applied, no norms used for a decision) so that both the
CUDA library and the CPU oracle can be fed from it without sharing any of the
method's code.

The paper (Section 4) evaluates on no dataset; the five workloads below are
synthetic stand-ins with the structure its analysis assumes (Theorem 3's proof
splits candidate pairs into near pairs and a far background): a far background
of iid points plus a known set of planted near pairs, or a Gaussian mixture
whose same-cluster pairs are the dense output.

Element types
    "i8"    numpy int8, values as drawn.
    "bf16"  numpy uint16 holding bfloat16 bit patterns (round-to-nearest-even
            of the fp32 value).  Those bits are *the* inputs for every consumer.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

KINDS = ("ip", "cos", "l2")
DTYPES = ("i8", "bf16")


@dataclasses.dataclass
class Workload:
    cfg_id: int
    name: str
    kind: str            # "ip" | "cos" | "l2"
    dtype: str           # "i8" | "bf16"
    n: int
    m: int
    d: int
    threshold: float     # t for ip/cos (score >= t), r for l2 (distance <= r)
    P: np.ndarray        # (n, d) int8 or uint16 (bf16 bits), C-contiguous
    Q: np.ndarray        # (m, d)
    planted: np.ndarray  # (k, 2) int64: (row in P, row in Q) of planted pairs
    labels_p: Optional[np.ndarray] = None  # cluster id per P row (mixture only)
    labels_q: Optional[np.ndarray] = None
    seed: int = 0
    note: str = ""

    @property
    def ops(self) -> int:
        """2*n*m*d, the operation count the throughput metric is defined on."""
        return 2 * self.n * self.m * self.d


# Full-size parameters of the five benchmark configurations.
CONFIGS = {
    1: dict(name="cfg1_ip_i8_pm1_2048_d64", kind="ip", dtype="i8", n=2048, m=2048, d=64,
            threshold=40.0, planted=32, flips=4),
    2: dict(name="cfg2_cos_bf16_65536_d128", kind="cos", dtype="bf16", n=65536, m=65536, d=128,
            threshold=0.9, planted=1000, noise=0.3),
    3: dict(name="cfg3_ip_i8_u8_262144_d256", kind="ip", dtype="i8", n=262144, m=262144, d=256,
            threshold=3000.0, planted=10000, lo=-8, hi=8),
    4: dict(name="cfg4_ip_i8_pm1_1048576_d128", kind="ip", dtype="i8", n=1048576, m=1048576, d=128,
            threshold=100.0, planted=100000, flips=8),
    5: dict(name="cfg5_l2_bf16_mixture_524288_d64", kind="l2", dtype="bf16", n=524288, m=524288,
            d=64, threshold=0.25, centers=1024, sigma=0.05),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _distinct_coords(rng: np.random.Generator, k: int, d: int, c: int) -> np.ndarray:
    """For each of k rows, c distinct coordinates out of d, uniformly."""
    if k == 0:
        return np.zeros((0, c), dtype=np.int64)
    return np.argsort(rng.random((k, d)), axis=1)[:, :c].astype(np.int64)


def _planted_indices(rng, n, m, k):
    if k > min(n, m):
        raise ValueError("more planted pairs than rows")
    ip = rng.choice(n, size=k, replace=False).astype(np.int64)
    jp = rng.choice(m, size=k, replace=False).astype(np.int64)
    return ip, jp


def make_workload(cfg_id: int, *, n: Optional[int] = None, m: Optional[int] = None,
                  d: Optional[int] = None, planted: Optional[int] = None,
                  centers: Optional[int] = None, seed: int = 0,
                  sigma_reading: str = "radial", threshold: Optional[float] = None) -> Workload:
    """Build configuration `cfg_id` (1..5); size arguments override the full-size
    defaults so that tests can use small and ragged shapes of the same recipe.

    Draw order is fixed: P body, Q body, planted P rows, planted Q rows, noise.
    `sigma_reading` applies to configuration 5 only: "radial" scales the cluster
    noise so that its total (radial) standard deviation is sigma, which makes all
    same-cluster pairs fall inside r (dense output); "percoord" uses sigma per
    coordinate, which makes the join empty at full size.
    """
    if cfg_id not in CONFIGS:
        raise ValueError(f"unknown configuration {cfg_id}")
    c = dict(CONFIGS[cfg_id])
    n = c["n"] if n is None else int(n)
    m = c["m"] if m is None else int(m)
    d = c["d"] if d is None else int(d)
    thr = c["threshold"] if threshold is None else float(threshold)
    rng = np.random.default_rng([seed, cfg_id])
    labels_p = labels_q = None
    note = ""

    if cfg_id in (1, 4):
        k = c["planted"] if planted is None else int(planted)
        P = (rng.integers(0, 2, size=(n, d), dtype=np.int8) * 2 - 1).astype(np.int8)
        Q = (rng.integers(0, 2, size=(m, d), dtype=np.int8) * 2 - 1).astype(np.int8)
        ip, jp = _planted_indices(rng, n, m, k)
        flips = _distinct_coords(rng, k, d, c["flips"])
        Y = P[ip].copy()
        rows = np.repeat(np.arange(k), c["flips"])
        Y[rows, flips.ravel()] = -Y[rows, flips.ravel()]
        Q[jp] = Y
    elif cfg_id == 3:
        k = c["planted"] if planted is None else int(planted)
        P = rng.integers(c["lo"], c["hi"] + 1, size=(n, d), dtype=np.int8)
        Q = rng.integers(c["lo"], c["hi"] + 1, size=(m, d), dtype=np.int8)
        ip, jp = _planted_indices(rng, n, m, k)
        e = rng.integers(-1, 2, size=(k, d), dtype=np.int8)
        Q[jp] = (P[ip] + e).astype(np.int8)          # values reach +-9: no clipping
    elif cfg_id == 2:
        k = c["planted"] if planted is None else int(planted)
        Pf = rng.standard_normal((n, d), dtype=np.float32)
        Pf /= np.linalg.norm(Pf, axis=1, keepdims=True)
        Qf = rng.standard_normal((m, d), dtype=np.float32)
        Qf /= np.linalg.norm(Qf, axis=1, keepdims=True)
        ip, jp = _planted_indices(rng, n, m, k)
        Y = Pf[ip] + np.float32(c["noise"]) * rng.standard_normal((k, d), dtype=np.float32) \
            / np.float32(np.sqrt(d))
        if k:
            Y /= np.linalg.norm(Y, axis=1, keepdims=True)
            Qf[jp] = Y
        P = f32_to_bf16_bits(Pf)
        Q = f32_to_bf16_bits(Qf)
    else:  # cfg 5: Gaussian mixture, no planted pairs; the clusters are the structure
        ncent = c["centers"] if centers is None else int(centers)
        cent = rng.standard_normal((ncent, d), dtype=np.float32)
        labels_p = rng.integers(0, ncent, size=n, dtype=np.int64)
        labels_q = rng.integers(0, ncent, size=m, dtype=np.int64)
        if sigma_reading == "radial":
            s = np.float32(c["sigma"] / np.sqrt(d))
        elif sigma_reading == "percoord":
            s = np.float32(c["sigma"])
        else:
            raise ValueError("sigma_reading must be 'radial' or 'percoord'")
        Pf = cent[labels_p] + s * rng.standard_normal((n, d), dtype=np.float32)
        Qf = cent[labels_q] + s * rng.standard_normal((m, d), dtype=np.float32)
        P = f32_to_bf16_bits(Pf)
        Q = f32_to_bf16_bits(Qf)
        ip = jp = np.zeros(0, dtype=np.int64)
        note = f"sigma_reading={sigma_reading}, centers={ncent}"

    plant = np.stack([ip, jp], axis=1).astype(np.int64) if len(ip) else np.zeros((0, 2), np.int64)
    return Workload(cfg_id=cfg_id, name=c["name"], kind=c["kind"], dtype=c["dtype"], n=n, m=m, d=d,
                    threshold=thr, P=np.ascontiguousarray(P), Q=np.ascontiguousarray(Q),
                    planted=plant, labels_p=labels_p, labels_q=labels_q, seed=seed, note=note)


def random_points(dtype: str, rows: int, d: int, seed: int, lo: int = -3, hi: int = 3,
                  scale: float = 1.0) -> np.ndarray:
    """Unstructured iid points for shape/edge-case tests: integers in [lo,hi] as
    int8, or scale*N(0,1) rounded to bf16 bits."""
    rng = np.random.default_rng([seed, rows, d, 77])
    if dtype == "i8":
        return rng.integers(lo, hi + 1, size=(rows, d), dtype=np.int8)
    if dtype == "bf16":
        return f32_to_bf16_bits(np.float32(scale) * rng.standard_normal((rows, d), dtype=np.float32))
    raise ValueError(dtype)


def random_bits(rows: int, d: int, seed: int, planted_from=None, flips: int = 0):
    """Bit-packed points in {0,1}^d: uint8 array (rows, d/8), coordinate k = bit k%8 of byte k/8.
    With `planted_from` (another packed array) the first len(planted_from) rows are copies of it with
    `flips` distinct coordinates flipped each (near pairs at Hamming distance `flips`)."""
    if d % 8:
        raise ValueError("d must be a multiple of 8")
    rng = np.random.default_rng([seed, rows, d, 99])
    bits = rng.integers(0, 2, size=(rows, d), dtype=np.uint8)
    if planted_from is not None:
        src = np.unpackbits(planted_from, axis=1, bitorder="little")[:, :d]
        k = len(src)
        cols = _distinct_coords(rng, k, d, flips)
        src = src.copy()
        if flips:
            rr = np.repeat(np.arange(k), flips)
            src[rr, cols.ravel()] ^= 1
        bits[:k] = src
    return np.packbits(bits, axis=1, bitorder="little")
