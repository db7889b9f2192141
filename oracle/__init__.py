"""Python access to the CPU oracle (test infrastructure; not part of the product).

The arithmetic lives in ``frog_oracle.cpp`` (plain sequential C++, one function per step of the
paper's Alg. 2-4 plus exact filtered kNN by the definition of Sec. 2.1).  This file only
compiles it with g++, reads an index file with numpy and marshals arrays through ctypes.  It
imports nothing from the CUDA package.  Allowed callers: the tests, the smoke check and the
benchmark's CPU-baseline leg.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
import struct
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "frog_oracle.cpp")
_LIB = os.path.join(_HERE, "libfrog_oracle.so")

ST_EMPTY, ST_EXACT, ST_ITER_CAP, ST_SHORT = 1, 2, 4, 8


def build(force: bool = False) -> str:
    """Compile the oracle (no fast-math, no contraction: fused multiply-adds are explicit)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.check_call(cmd)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.frog_oracle_dist2.restype = C.c_float
        _lib.frog_oracle_entry_point.restype = C.c_int64
    return _lib


def _p(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ctype))


# ------------------------------------------------------------------------------------------
# index file (format: 256-byte little-endian header, then four 128-byte-aligned arrays)
# ------------------------------------------------------------------------------------------
@dataclasses.dataclass
class OracleIndex:
    n: int
    d: int
    d_pad: int
    H: int
    m: int
    n_inv: int
    ef_c: int
    patience: int
    beta: float
    gamma: float
    seed: int
    sorted_attr: np.ndarray   # [n] int32
    rank2id: np.ndarray       # [n] int32
    vectors: np.ndarray       # [n, d_pad] float32, row r = vector of rank r
    enc: np.ndarray           # [n, H, m] uint32 ranks, 0xFFFFFFFF = empty


def load_index(path: str) -> OracleIndex:
    with open(path, "rb") as f:
        hdr = f.read(256)
    if hdr[:8] != b"FROGIDX1":
        raise ValueError("bad magic")
    (version, d, d_pad, H, m, n_inv, ef_c, patience) = struct.unpack_from("<8I", hdr, 8)
    beta, gamma = struct.unpack_from("<2f", hdr, 40)
    n, seed = struct.unpack_from("<2Q", hdr, 48)
    bot, _ = struct.unpack_from("<2I", hdr, 64)
    o_attr, o_r2i, o_vec, o_enc, fbytes = struct.unpack_from("<5Q", hdr, 72)
    if version != 1 or bot != 0xFFFFFFFF:
        raise ValueError("bad version")
    if os.path.getsize(path) != fbytes:
        raise ValueError("size mismatch")
    mm = np.memmap(path, dtype=np.uint8, mode="r")
    def arr(off, count, dt):
        return np.frombuffer(mm, dtype=dt, count=count, offset=off)
    return OracleIndex(
        n=n, d=d, d_pad=d_pad, H=H, m=m, n_inv=n_inv, ef_c=ef_c, patience=patience,
        beta=beta, gamma=gamma, seed=seed,
        sorted_attr=arr(o_attr, n, np.int32), rank2id=arr(o_r2i, n, np.int32),
        vectors=arr(o_vec, n * d_pad, np.float32).reshape(n, d_pad),
        enc=arr(o_enc, n * H * m, np.uint32).reshape(n, H, m))


def rounded_to_f16(ix: OracleIndex) -> OracleIndex:
    """The same index with every vector component rounded to the nearest fp16 value (ties to even)
    and widened back to fp32: what a search over half-precision storage sees.  Arithmetic is
    unchanged (fp32, same order), only the stored values differ."""
    v = np.asarray(ix.vectors).astype(np.float16).astype(np.float32)
    return dataclasses.replace(ix, vectors=np.ascontiguousarray(v))


def pad_queries(queries: np.ndarray, d_pad: int) -> np.ndarray:
    q = np.ascontiguousarray(queries, dtype=np.float32)
    if q.shape[1] == d_pad:
        return q
    out = np.zeros((q.shape[0], d_pad), dtype=np.float32)
    out[:, : q.shape[1]] = q
    return out


# ------------------------------------------------------------------------------------------
# step functions
# ------------------------------------------------------------------------------------------
def rank_interval(sorted_attr: np.ndarray, lo: int, hi: int):
    l, r = C.c_int64(), C.c_int64()
    lib().frog_oracle_rank_interval(_p(np.ascontiguousarray(sorted_attr), C.c_int32),
                                    C.c_int64(len(sorted_attr)), C.c_int32(lo), C.c_int32(hi),
                                    C.byref(l), C.byref(r))
    return l.value, r.value


def segment_at(N: int, h: int, x: int):
    L, R = C.c_int64(), C.c_int64()
    lib().frog_oracle_segment_at(C.c_int64(N), C.c_int(h), C.c_int64(x), C.byref(L), C.byref(R))
    return L.value, R.value


def hotspot(l_q: int, r_q: int, H: int, N: int):
    a, b = C.c_int(), C.c_int()
    lib().frog_oracle_hotspot(C.c_int64(l_q), C.c_int64(r_q), C.c_int(H), C.c_int64(N),
                              C.byref(a), C.byref(b))
    return a.value, b.value


def en_identification(enc_u: np.ndarray, l_q: int, r_q: int, L_start: int, L_end: int, B: int,
                      warp: int = 32):
    enc_u = np.ascontiguousarray(enc_u, dtype=np.uint32)
    m = enc_u.shape[1]
    out = np.zeros(max(B, 1), dtype=np.uint32)
    rows = C.c_int()
    cnt = lib().frog_oracle_en_identification(_p(enc_u, C.c_uint32), C.c_int(m), C.c_int64(l_q),
                                              C.c_int64(r_q), C.c_int(L_start), C.c_int(L_end),
                                              C.c_int(B), C.c_int(warp), _p(out, C.c_uint32),
                                              C.byref(rows))
    return out[:cnt].copy(), rows.value


def dist2(q: np.ndarray, x: np.ndarray) -> float:
    q = np.ascontiguousarray(q, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert q.shape == x.shape and q.shape[0] % 4 == 0
    return float(lib().frog_oracle_dist2(_p(q, C.c_float), _p(x, C.c_float), C.c_int(q.shape[0])))


def entry_point(seed: int, l_q: int, r_q: int, j: int) -> int:
    return int(lib().frog_oracle_entry_point(C.c_uint64(seed), C.c_int64(l_q), C.c_int64(r_q), C.c_int(j)))


@dataclasses.dataclass
class SearchResult:
    ids: np.ndarray       # [nq, k] int32 original ids, -1 pad
    dists: np.ndarray     # [nq, k] float32 ascending, +inf pad
    status: np.ndarray    # [nq] uint32
    stats: np.ndarray     # [nq, 4] uint32: expansions, ENC rows read, ENs admitted, distances
    trace: Optional[np.ndarray]
    threads: int


def default_max_iters(ef_s: int) -> int:
    return 16 * ef_s


def search(ix: OracleIndex, queries: np.ndarray, lo: np.ndarray, hi: np.ndarray, k: int, ef_s: int,
           epn: int = 16, B: int = 16, max_iters: int = 0, seed: int = 0, warp: int = 32,
           no_hotspot: bool = False, trace_cap: int = 0, threads: int = 0,
           exact_below: int = 0, eager_hash: bool = False) -> SearchResult:
    """Alg. 2 over the whole batch (parallel over queries only).  Ranges holding at most
    max(ef_s, exact_below) objects are answered by the exact slab scan.  eager_hash: ablation with
    the visited test inside the predicate of Alg. 4."""
    q = pad_queries(queries, ix.d_pad)
    nq = q.shape[0]
    lo = np.ascontiguousarray(lo, dtype=np.int32)
    hi = np.ascontiguousarray(hi, dtype=np.int32)
    ids = np.empty((nq, k), dtype=np.int32)
    dists = np.empty((nq, k), dtype=np.float32)
    status = np.zeros(nq, dtype=np.uint32)
    stats = np.zeros((nq, 4), dtype=np.uint32)
    trace = np.zeros((nq, trace_cap), dtype=np.uint32) if trace_cap > 0 else None
    if max_iters <= 0:
        max_iters = default_max_iters(ef_s)
    used = lib().frog_oracle_search(
        _p(ix.sorted_attr, C.c_int32), _p(ix.rank2id, C.c_int32), _p(ix.vectors, C.c_float),
        _p(ix.enc, C.c_uint32), C.c_int64(ix.n), C.c_int(ix.d_pad), C.c_int(ix.H), C.c_int(ix.m),
        _p(q, C.c_float), _p(lo, C.c_int32), _p(hi, C.c_int32), C.c_int64(nq),
        C.c_int(k), C.c_int(ef_s), C.c_int(epn), C.c_int(B), C.c_int(max_iters), C.c_uint64(seed),
        C.c_int(warp), C.c_int(1 if no_hotspot else 0), C.c_int(exact_below), C.c_int(1 if eager_hash else 0),
        _p(ids, C.c_int32), _p(dists, C.c_float), _p(status, C.c_uint32), _p(stats, C.c_uint32),
        _p(trace, C.c_uint32), C.c_int64(trace_cap), C.c_int(threads))
    return SearchResult(ids, dists, status, stats, trace, int(used))


def exact_scan(vectors: np.ndarray, attrs: np.ndarray, queries: np.ndarray, lo, hi, k: int,
               mode: int = 0, threads: int = 0):
    """Exact filtered kNN by the definition: scan all objects in original order."""
    v = np.ascontiguousarray(vectors, dtype=np.float32)
    a = np.ascontiguousarray(attrs, dtype=np.int32)
    q = np.ascontiguousarray(queries, dtype=np.float32)
    if mode == 1:
        assert v.shape[1] % 4 == 0
    nq = q.shape[0]
    lo = np.ascontiguousarray(lo, dtype=np.int32)
    hi = np.ascontiguousarray(hi, dtype=np.int32)
    ids = np.empty((nq, k), dtype=np.int32)
    dists = np.empty((nq, k), dtype=np.float32)
    lib().frog_oracle_exact_scan(_p(v, C.c_float), _p(a, C.c_int32), C.c_int64(v.shape[0]),
                                 C.c_int(v.shape[1]), _p(q, C.c_float), _p(lo, C.c_int32),
                                 _p(hi, C.c_int32), C.c_int64(nq), C.c_int(k), C.c_int(mode),
                                 _p(ids, C.c_int32), _p(dists, C.c_float), C.c_int(threads))
    return ids, dists


def exact_slab(ix: OracleIndex, queries: np.ndarray, lo, hi, k: int, mode: int = 0, threads: int = 0):
    """Exact filtered kNN through the index: scan the contiguous rank slab of each query."""
    q = pad_queries(queries, ix.d_pad)
    nq = q.shape[0]
    lo = np.ascontiguousarray(lo, dtype=np.int32)
    hi = np.ascontiguousarray(hi, dtype=np.int32)
    ids = np.empty((nq, k), dtype=np.int32)
    dists = np.empty((nq, k), dtype=np.float32)
    used = lib().frog_oracle_exact_slab(
        _p(ix.sorted_attr, C.c_int32), _p(ix.rank2id, C.c_int32), _p(ix.vectors, C.c_float),
        C.c_int64(ix.n), C.c_int(ix.d_pad), _p(q, C.c_float), _p(lo, C.c_int32), _p(hi, C.c_int32),
        C.c_int64(nq), C.c_int(k), C.c_int(mode), _p(ids, C.c_int32), _p(dists, C.c_float),
        C.c_int(threads))
    return ids, dists, int(used)


def recall(ids: np.ndarray, gt_ids: np.ndarray) -> float:
    """Recall@k (paper Sec. 8.1.3): |R ∩ GT| / |GT| averaged over queries with a non-empty GT."""
    tot, cnt = 0.0, 0
    for r, g in zip(ids, gt_ids):
        g = g[g >= 0]
        if g.size == 0:
            continue
        tot += np.intersect1d(r[r >= 0], g).size / g.size
        cnt += 1
    return tot / max(cnt, 1)


def recall_tie_aware(dists: np.ndarray, gt_dists: np.ndarray, rel: float = 1e-6) -> float:
    """Recall counting a result as a hit when its distance does not exceed the k-th true one."""
    tot, cnt = 0.0, 0
    for r, g in zip(dists, gt_dists):
        g = g[np.isfinite(g)]
        if g.size == 0:
            continue
        thr = g[-1] * (1.0 + rel)
        tot += min(int((r[np.isfinite(r)] <= thr).sum()), g.size) / g.size
        cnt += 1
    return tot / max(cnt, 1)


def num_threads() -> int:
    return int(lib().frog_oracle_num_threads())
