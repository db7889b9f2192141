"""Seeded synthetic inputs for range-filtering k-ANN search (numpy only).

This module produces the raw inputs of the search problem -- base vectors, one integer
attribute per object, query vectors and query attribute ranges -- for the five workloads the
benchmarks and tests run on.  It contains none of the method's arithmetic (no ranks, no
distances, no graph, no index): both the CPU oracle and the CUDA path consume its arrays, and
neither of them is imported here.

The workloads stand in for the datasets of the paper's Table 1 (Deep10M 10M x 96, SIFT / Audio
1M x 128, text embeddings of several hundred dimensions), which are not available offline; the
shapes, value ranges and attribute rules follow them:

* ``tiny``   n=10,000  d=32   16-cluster isotropic Gaussian mixture; attribute = a seeded
  permutation of 0..n-1 (the paper's rule for its synthetic attributes, Sec. 8.1.2).
* ``sift``   n=1,000,000 d=128 integer-valued components in [0,255] stored as fp32
  (64-cluster mixture of low-rank Gaussians, marginals ~ |N(0,40)|); attribute uniform int32
  in [0, 1e6) (duplicates occur).
* ``deep1m`` n=1,000,000 d=96 unit-normalised 256-cluster low-rank mixture; attribute = insertion
  timestamp, correlated with the cluster (clusters arrive in seeded contiguous blocks).
* ``deep10m`` n=10,000,000 d=96 as above, attribute uniform int32 with 1% duplicated values.
* ``text``   n=1,000,000 d=768 anisotropic Gaussian (variance of component i ~ i^-0.8),
  unit-normalised; attribute uniform int32.

Query ranges: a width fraction f is drawn (log-uniform in [2^-a, 1], or from a fixed list), the
range covers w = max(1, round(f n)) consecutive objects in attribute order starting at a uniform
position, and [lo, hi] are the attribute values of its two end objects.  With duplicated
attribute values the realised number of objects in [lo, hi] can exceed w; consumers recompute it.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import numpy as np

__all__ = ["Workload", "WORKLOADS", "make_workload", "make_ranges", "scaled"]


@dataclasses.dataclass
class Workload:
    """Raw inputs of one workload (all arrays C-contiguous)."""

    name: str
    vectors: np.ndarray      # [n, d] float32, object i in row i
    attrs: np.ndarray        # [n] int32, attribute of object i
    queries: np.ndarray      # [nq, d] float32
    lo: np.ndarray           # [nq] int32 inclusive lower attribute bound
    hi: np.ndarray           # [nq] int32 inclusive upper attribute bound
    k: int
    # index parameters the paper prescribes for this dimensionality (Sec. 8.1.4)
    m: int
    ef_c: int
    n_inv: int
    seed: int

    @property
    def n(self) -> int:
        return int(self.vectors.shape[0])

    @property
    def d(self) -> int:
        return int(self.vectors.shape[1])

    @property
    def nq(self) -> int:
        return int(self.queries.shape[0])


# name -> (n, d, nq, log2 of the smallest width fraction, seed)
WORKLOADS = {
    "tiny": dict(n=10_000, d=32, nq=200, min_log2=8, seed=0x5EED0001),
    "sift": dict(n=1_000_000, d=128, nq=10_000, min_log2=10, seed=0x5EED0002),
    "deep1m": dict(n=1_000_000, d=96, nq=10_000, min_log2=10, seed=0x5EED0003),
    "deep10m": dict(n=10_000_000, d=96, nq=10_000, min_log2=12, seed=0x5EED0004),
    "text": dict(n=1_000_000, d=768, nq=10_000, min_log2=10, seed=0x5EED0005),
}


def _paper_params(d: int):
    """Default index parameters by dimensionality (paper Sec. 8.1.4)."""
    if d <= 300:
        return dict(m=16, ef_c=128, n_inv=7)
    return dict(m=32, ef_c=256, n_inv=6)


def _mixture(rng, n, d, n_clusters, center_sigma, noise_sigma, labels=None, chunk=1 << 18):
    centers = (rng.standard_normal((n_clusters, d)) * center_sigma).astype(np.float32)
    if labels is None:
        labels = rng.integers(0, n_clusters, size=n, dtype=np.int64)
    out = np.empty((n, d), dtype=np.float32)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        noise = rng.standard_normal((e - s, d), dtype=np.float32) * np.float32(noise_sigma)
        out[s:e] = centers[labels[s:e]] + noise
    return out, centers, labels


def _normalise_rows(x: np.ndarray, chunk=1 << 18) -> None:
    for s in range(0, x.shape[0], chunk):
        blk = x[s:s + chunk]
        nrm = np.sqrt((blk.astype(np.float64) ** 2).sum(axis=1))
        nrm[nrm == 0] = 1.0
        blk /= nrm[:, None].astype(np.float32)


class _FactorMixture:
    """Mixture of K low-rank Gaussians: x = c_k + z A_k + e, z ~ N(0, I_r), e ~ N(0, s_e^2 I_d).

    Centers c_k ~ N(0, s_c^2 I_d); loadings A_k (r x d) with entries N(0, s_l^2 / r), so a
    component has variance s_c^2 + s_l^2 + s_e^2 overall.  A small latent dimension r gives the
    data the low local intrinsic dimensionality (about 10-20) reported for descriptor and
    embedding datasets such as SIFT and Deep, which an isotropic Gaussian in d dimensions lacks.
    """

    def __init__(self, rng, d, n_clusters, r, s_c, s_l, s_e):
        self.d, self.K, self.r, self.s_e = d, n_clusters, r, s_e
        self.centers = (rng.standard_normal((n_clusters, d)) * s_c).astype(np.float32)
        self.load = (rng.standard_normal((n_clusters, r, d)) * (s_l / np.sqrt(r))).astype(np.float32)

    def sample(self, rng, n, labels=None, chunk=1 << 18):
        if labels is None:
            labels = rng.integers(0, self.K, size=n, dtype=np.int64)
        out = np.empty((n, self.d), dtype=np.float32)
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            lab = labels[s:e]
            z = rng.standard_normal((e - s, self.r), dtype=np.float32)
            blk = rng.standard_normal((e - s, self.d), dtype=np.float32) * np.float32(self.s_e)
            order = np.argsort(lab, kind="stable")
            bounds = np.searchsorted(lab[order], np.arange(self.K + 1))
            for c in range(self.K):
                idx = order[bounds[c]:bounds[c + 1]]
                if idx.size:
                    blk[idx] += self.centers[c] + z[idx] @ self.load[c]
            out[s:e] = blk
        return out


def _to_sift_range(x: np.ndarray) -> np.ndarray:
    """Integer-valued components in [0, 255]: clip(round(|x|)), in place."""
    np.abs(x, out=x)
    np.rint(x, out=x)
    np.clip(x, 0, 255, out=x)
    return x


def make_ranges(attrs: np.ndarray, nq: int, rng, min_log2: Optional[int] = None,
                fractions: Optional[Sequence[float]] = None):
    """Draw nq attribute ranges.

    ``min_log2``: width fraction f = 2^(-min_log2 * U), U ~ U[0,1] (log-uniform).
    ``fractions``: instead, pick f uniformly from this list per query (the paper's mixed
    setting uses 2^-i, i in 0..9, each with equal probability, Sec. 8.1.2).
    Returns (lo, hi, f).
    """
    n = attrs.shape[0]
    srt = np.sort(attrs, kind="stable")
    if fractions is not None:
        f = np.asarray(fractions, dtype=np.float64)[rng.integers(0, len(fractions), size=nq)]
    else:
        f = np.exp2(-float(min_log2) * rng.random(nq))
    w = np.maximum(1, np.rint(f * n).astype(np.int64))
    w = np.minimum(w, n)
    start = (rng.random(nq) * (n - w + 1)).astype(np.int64)
    start = np.minimum(start, n - w)
    lo = srt[start].astype(np.int32)
    hi = srt[start + w - 1].astype(np.int32)
    return np.ascontiguousarray(lo), np.ascontiguousarray(hi), f


def make_workload(name: str, n: Optional[int] = None, nq: Optional[int] = None,
                  seed: Optional[int] = None, fractions: Optional[Sequence[float]] = None,
                  k: int = 10) -> Workload:
    """Generate workload ``name``; ``n``/``nq`` override the size (same recipe, same seed)."""
    spec = dict(WORKLOADS[name])
    n = int(spec["n"] if n is None else n)
    nq = int(spec["nq"] if nq is None else nq)
    seed = int(spec["seed"] if seed is None else seed)
    d = spec["d"]
    rng = np.random.Generator(np.random.PCG64(seed))
    qrng = np.random.Generator(np.random.PCG64(seed ^ 0xA5A5A5A5))

    if name == "tiny":
        vectors, centers, _ = _mixture(rng, n, d, 16, 1.0, 0.3)
        attrs = rng.permutation(n).astype(np.int32)
        ql = qrng.integers(0, 16, size=nq)
        queries = centers[ql] + qrng.standard_normal((nq, d), dtype=np.float32) * np.float32(0.3)
    elif name == "sift":
        # components ~ |N(0, 40)| overall: 20^2 (centers) + 34.4^2 (12 latent factors) + 4^2
        mix = _FactorMixture(rng, d, 64, 12, 20.0, 34.4, 4.0)
        vectors = _to_sift_range(mix.sample(rng, n))
        attrs = rng.integers(0, 1_000_000, size=n, dtype=np.int64).astype(np.int32)
        queries = _to_sift_range(mix.sample(qrng, nq))
    elif name in ("deep1m", "deep10m"):
        n_clusters = 256
        mix = _FactorMixture(rng, d, n_clusters, 12, 0.5, 1.0, 0.12)
        if name == "deep1m":
            # clusters arrive in contiguous blocks of the insertion timeline
            n_blocks = 2048
            block_cluster = rng.integers(0, n_clusters, size=n_blocks)
            t = np.arange(n, dtype=np.int64)
            labels_by_time = block_cluster[(t * n_blocks) // n]
            perm = rng.permutation(n)           # object i was inserted at time perm[i]
            labels = labels_by_time[perm]
            vectors = mix.sample(rng, n, labels=labels)
            attrs = perm.astype(np.int32)
        else:
            vectors = mix.sample(rng, n)
            attrs = rng.integers(0, 2**31 - 1, size=n, dtype=np.int64).astype(np.int32)
            n_dup = n // 100                     # 1% of the objects copy another's attribute
            dst = rng.choice(n, size=n_dup, replace=False)
            src = rng.integers(0, n, size=n_dup)
            attrs[dst] = attrs[src]
        _normalise_rows(vectors)
        queries = mix.sample(qrng, nq)
        _normalise_rows(queries)
    elif name == "text":
        lam = np.arange(1, d + 1, dtype=np.float64) ** -0.8
        sd = np.sqrt(lam).astype(np.float32)
        vectors = np.empty((n, d), dtype=np.float32)
        chunk = 1 << 16
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            vectors[s:e] = rng.standard_normal((e - s, d), dtype=np.float32) * sd
        _normalise_rows(vectors)
        attrs = rng.integers(0, 2**31 - 1, size=n, dtype=np.int64).astype(np.int32)
        queries = qrng.standard_normal((nq, d), dtype=np.float32) * sd
        _normalise_rows(queries)
    else:
        raise KeyError(name)

    queries = np.ascontiguousarray(queries, dtype=np.float32)
    lo, hi, _ = make_ranges(attrs, nq, qrng, min_log2=spec["min_log2"], fractions=fractions)
    p = _paper_params(d)
    return Workload(name=name, vectors=np.ascontiguousarray(vectors), attrs=np.ascontiguousarray(attrs),
                    queries=queries, lo=lo, hi=hi, k=k, seed=seed, **p)


def scaled(name: str, n: int, nq: int, **kw) -> Workload:
    """The recipe of ``name`` at a reduced size (for tests the oracle finishes in seconds)."""
    return make_workload(name, n=n, nq=nq, **kw)
