"""Python binding of the FROG search library (argument marshalling only).

``libfrog.so`` (CUDA, sm_100a) does all of the work; this module loads it with ctypes, passes raw
device pointers taken from torch tensors (torch is used for device memory and streams only) and
converts error codes into exceptions.  There is no fallback: if the shared library is missing
the import fails.

    build_index(vectors, attrs, path)                -> writes an index file (host builder)
    ix = Index.load(path, device=0)
    ids, dists = ix.search(queries, lo, hi, k, beam_width)      # device tensors in and out
    ids, dists = ix.exact_search(queries, lo, hi, k)
    ids, dists = ix.search_host(queries_np, lo_np, hi_np, k, beam_width)   # host in and out
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_SEARCH = os.environ.get("FROG_LIBFROG", os.path.join(_HERE, "libfrog.so"))   # override: A/B builds
_LIB_BUILD = os.path.join(_HERE, "libfrog_build.so")

FROG_MAX_BEAM_WIDTH = 512
ST_EMPTY, ST_EXACT, ST_ITER_CAP, ST_SHORT, ST_FORGOT = 1, 2, 4, 8, 16
VISITED_AUTO, VISITED_BITMAP, VISITED_HASH = 0, 1, 2
STORAGE_F32, STORAGE_F16 = 0, 1


class FrogError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} (code {code}, cuda {last_cuda_error()})")
        self.code = code


class IndexInfo(C.Structure):
    _fields_ = [("n", C.c_int64), ("d", C.c_int32), ("d_pad", C.c_int32), ("H", C.c_int32),
                ("m", C.c_int32), ("n_inv", C.c_int32), ("ef_c", C.c_int32), ("patience", C.c_int32),
                ("beta", C.c_float), ("gamma", C.c_float), ("seed", C.c_uint64),
                ("device", C.c_int32), ("device_bytes", C.c_int64)]


class Params(C.Structure):
    _fields_ = [("epn", C.c_int32), ("budget", C.c_int32), ("max_iters", C.c_int32),
                ("no_hotspot", C.c_int32), ("seed", C.c_uint64), ("hash_bits", C.c_int32),
                ("visited", C.c_int32), ("storage", C.c_int32), ("debug_flags", C.c_int32),
                ("exact_below", C.c_int32), ("eager_hash", C.c_int32)]


class BuildParams(C.Structure):
    _fields_ = [("m", C.c_int32), ("ef_c", C.c_int32), ("n_inv", C.c_int32), ("patience", C.c_int32),
                ("beta", C.c_float), ("gamma", C.c_float), ("seed", C.c_uint64),
                ("threads", C.c_int32), ("reserved", C.c_int32)]


def _load(path: str) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2608_16491_b200.build` "
                          "(there is no fallback implementation)")
    return C.CDLL(path)


class _SearchLib:
    """libfrog.so, loaded at the first use of any of its functions.  Importing the package must work
    on a fresh checkout (the build step lives in this package); every call into the search path
    without the compiled library raises ImportError — there is nothing to fall back to."""

    def __init__(self):
        self._dll = None

    def _get(self) -> C.CDLL:
        if self._dll is None:
            dll = _load(_LIB_SEARCH)
            dll.frog_strerror.restype = C.c_char_p
            self._dll = dll
        return self._dll

    def __getattr__(self, name):
        return getattr(self._get(), name)


_lib = _SearchLib()
_blib = None

_vp = C.c_void_p


def _build_lib() -> C.CDLL:
    global _blib
    if _blib is None:
        _blib = _load(_LIB_BUILD)
        _blib.frog_fusion_distance.restype = C.c_double
        _blib.frog_fusion_distance.argtypes = [C.c_double] * 4
        _blib.frog_retained_depth.restype = C.c_int32
        _blib.frog_retained_depth.argtypes = [C.c_int64, C.c_int32]
    return _blib


def strerror(code: int) -> str:
    return _lib.frog_strerror(C.c_int(code)).decode()


def last_cuda_error() -> int:
    return int(_lib.frog_last_cuda_error())


def fusion_distance(delta_v: float, delta_a: float, beta: float, gamma: float) -> float:
    return float(_build_lib().frog_fusion_distance(delta_v, delta_a, beta, gamma))


def retained_depth(n: int, n_inv: int) -> int:
    return int(_build_lib().frog_retained_depth(n, n_inv))


BUILD_NO_REVERSE_EDGES, BUILD_ENC_FUSION_NEAREST, BUILD_LITERAL = 1, 2, 3


def build_index(vectors: np.ndarray, attrs: np.ndarray, path: str, m: int = 0, ef_c: int = 0,
                n_inv: int = -1, patience: int = 0, beta: float = -1.0, gamma: float = 0.0,
                seed: int = 0, threads: int = 0, flags: int = 0) -> None:
    """Build the FROG index of (vectors, attrs) on the host and write it to ``path``.
    ``flags``: BUILD_* switches (BUILD_LITERAL = the construction of Sec. 6.1 as written)."""
    v = np.ascontiguousarray(vectors, dtype=np.float32)
    a = np.ascontiguousarray(attrs, dtype=np.int32)
    if v.ndim != 2 or a.shape != (v.shape[0],):
        raise ValueError("vectors must be [n, d] and attrs [n]")
    p = BuildParams(m=m, ef_c=ef_c, n_inv=n_inv, patience=patience, beta=beta, gamma=gamma,
                    seed=seed, threads=threads, reserved=flags)
    rc = _build_lib().frog_index_build(v.ctypes.data_as(_vp), a.ctypes.data_as(_vp),
                                       C.c_int64(v.shape[0]), C.c_int32(v.shape[1]), C.byref(p),
                                       path.encode())
    if rc != 0:
        raise FrogError(rc, "frog_index_build")


def build_index_gpu(vectors: np.ndarray, attrs: np.ndarray, path: str, device: int = 0, m: int = 0,
                    ef_c: int = 0, n_inv: int = -1, patience: int = 0, beta: float = -1.0,
                    gamma: float = 0.0, seed: int = 0, flags: int = 0) -> None:
    """Build the FROG index of (vectors, attrs) with the CUDA builder and write it to ``path``
    (the same file the host builder writes).  ``flags``: BUILD_* switches."""
    v = np.ascontiguousarray(vectors, dtype=np.float32)
    a = np.ascontiguousarray(attrs, dtype=np.int32)
    if v.ndim != 2 or a.shape != (v.shape[0],):
        raise ValueError("vectors must be [n, d] and attrs [n]")
    p = BuildParams(m=m, ef_c=ef_c, n_inv=n_inv, patience=patience, beta=beta, gamma=gamma,
                    seed=seed, threads=0, reserved=flags)
    rc = _lib.frog_index_build_gpu(v.ctypes.data_as(_vp), a.ctypes.data_as(_vp), C.c_int64(v.shape[0]),
                                   C.c_int32(v.shape[1]), C.byref(p), C.c_int(device), path.encode())
    if rc != 0:
        raise FrogError(rc, "frog_index_build_gpu")


def _ptr(t) -> C.c_void_p:
    return _vp(0) if t is None else _vp(t.data_ptr())


def _stream_ptr(stream) -> C.c_void_p:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return _vp(s.cuda_stream)


class Index:
    """Handle of an index resident on one GPU."""

    def __init__(self, handle: C.c_void_p):
        self._h = handle
        info = IndexInfo()
        rc = _lib.frog_index_info(self._h, C.byref(info))
        if rc:
            raise FrogError(rc, "frog_index_info")
        self.info = info

    @classmethod
    def load(cls, path: str, device: int = 0) -> "Index":
        h = _vp()
        rc = _lib.frog_index_load(path.encode(), C.c_int(device), C.byref(h))
        if rc:
            raise FrogError(rc, "frog_index_load")
        return cls(h)

    def enable_f16(self) -> None:
        """Add an fp16 copy of the vectors; searches read it with ``Params(storage=STORAGE_F16)``."""
        rc = _lib.frog_index_enable_f16(self._h)
        if rc:
            raise FrogError(rc, "frog_index_enable_f16")

    def close(self) -> None:
        if self._h:
            _lib.frog_index_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- device-resident search ---------------------------------------------------------------
    def _check(self, queries, lo, hi):
        import torch
        if not (queries.is_cuda and lo.is_cuda and hi.is_cuda):
            raise ValueError("queries, lo, hi must be CUDA tensors")
        if queries.dtype != torch.float32 or lo.dtype != torch.int32 or hi.dtype != torch.int32:
            raise ValueError("dtypes must be float32 / int32 / int32")
        if queries.dim() != 2 or queries.shape[1] != self.info.d or not queries.is_contiguous():
            raise ValueError("queries must be contiguous [nq, d]")
        nq = queries.shape[0]
        if lo.shape != (nq,) or hi.shape != (nq,) or not lo.is_contiguous() or not hi.is_contiguous():
            raise ValueError("lo, hi must be contiguous [nq]")
        return nq

    def search(self, queries, lo, hi, k: int, beam_width: int, out_ids=None, out_dists=None,
               stream=None, params: Optional[Params] = None, status=None, stats=None, trace=None):
        """Alg. 2 over the batch; returns (ids [nq,k] int32, dists [nq,k] float32) on the device."""
        import torch
        nq = self._check(queries, lo, hi)
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        plain = params is None and status is None and stats is None and trace is None
        if plain:
            rc = _lib.frog_search(self._h, _ptr(queries), _ptr(lo), _ptr(hi), C.c_int(nq), C.c_int(k),
                                  C.c_int(beam_width), _ptr(out_ids), _ptr(out_dists), _stream_ptr(stream))
        else:
            cap = 0 if trace is None else int(trace.shape[1])
            rc = _lib.frog_search_ex(self._h, _ptr(queries), _ptr(lo), _ptr(hi), C.c_int(nq), C.c_int(k),
                                     C.c_int(beam_width), C.byref(params) if params is not None else None,
                                     _ptr(out_ids), _ptr(out_dists), _ptr(status), _ptr(stats),
                                     _ptr(trace), C.c_int(cap), _stream_ptr(stream))
        if rc:
            raise FrogError(rc, "frog_search")
        return out_ids, out_dists

    def search_static(self, queries, lo, hi, k: int, beam_width: int, out_ids=None, out_dists=None,
                      stream=None, params: Optional[Params] = None):
        """The search through ``frog_search_static``: same results as :meth:`search`, but all scratch
        sits in a fixed 16 MiB device array inside the library, so the call never allocates device
        memory (for callers under stream capture, with a fixed memory budget, or next to another
        allocator that owns the free memory).  Output tensors are still the caller's: pass
        ``out_ids``/``out_dists`` to keep this wrapper allocation-free too.  Indexes of more than
        2,097,152 objects are refused; overlapping calls on one device must be serialised."""
        import torch
        nq = self._check(queries, lo, hi)
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        rc = _lib.frog_search_static(self._h, _ptr(queries), _ptr(lo), _ptr(hi), C.c_int(nq), C.c_int(k),
                                     C.c_int(beam_width), C.byref(params) if params is not None else None,
                                     _ptr(out_ids), _ptr(out_dists), _stream_ptr(stream))
        if rc:
            raise FrogError(rc, "frog_search_static")
        return out_ids, out_dists

    def exact_search(self, queries, lo, hi, k: int, out_ids=None, out_dists=None, stream=None):
        """Exact filtered kNN by slab scan (ground truth / pre-filtering reference)."""
        import torch
        nq = self._check(queries, lo, hi)
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
        rc = _lib.frog_exact_search(self._h, _ptr(queries), _ptr(lo), _ptr(hi), C.c_int(nq), C.c_int(k),
                                    _ptr(out_ids), _ptr(out_dists), _stream_ptr(stream))
        if rc:
            raise FrogError(rc, "frog_exact_search")
        return out_ids, out_dists

    # -- host buffers in, host buffers out (transfers inside the call) ---------------------------
    def search_host(self, queries, lo, hi, k: int, beam_width: int, out_ids=None, out_dists=None,
                    stream=None, params: Optional[Params] = None):
        """queries/lo/hi: CPU torch tensors or numpy arrays (pinned memory makes copies async)."""
        import torch
        tq, tlo, thi = (torch.as_tensor(x) for x in (queries, lo, hi))
        nq = tq.shape[0]
        if tq.dtype != torch.float32 or tq.dim() != 2 or tq.shape[1] != self.info.d or not tq.is_contiguous():
            raise ValueError("queries must be contiguous float32 [nq, d]")
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int32).pin_memory()
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=torch.float32).pin_memory()
        rc = _lib.frog_search_host(self._h, _ptr(tq), _ptr(tlo), _ptr(thi), C.c_int(nq), C.c_int(k),
                                   C.c_int(beam_width), C.byref(params) if params is not None else None,
                                   _ptr(out_ids), _ptr(out_dists), _stream_ptr(stream))
        if rc:
            raise FrogError(rc, "frog_search_host")
        return out_ids, out_dists

    def last_status(self, stream=None) -> int:
        """Launch-wide FROG_ST_* bits of the last search on ``stream`` (0 = nothing to report)."""
        flags = C.c_uint32()
        rc = _lib.frog_search_last_status(self._h, _stream_ptr(stream), C.byref(flags))
        if rc:
            raise FrogError(rc, "frog_search_last_status")
        return int(flags.value)

    def kernel_ms(self, stream=None) -> float:
        """Device time of the search kernel of the last search on ``stream`` made with
        ``Params(debug_flags=16)`` (waits for it)."""
        ms = C.c_float()
        rc = _lib.frog_search_kernel_ms(self._h, _stream_ptr(stream), C.byref(ms))
        if rc:
            raise FrogError(rc, "frog_search_kernel_ms")
        return float(ms.value)

    def launch_info(self, beam_width: int, params: Optional[Params] = None):
        g, b, s, qsm = C.c_int(), C.c_int(), C.c_int(), C.c_int()
        rc = _lib.frog_search_launch_info(self._h, C.c_int(beam_width),
                                          C.byref(params) if params is not None else None,
                                          C.byref(g), C.byref(b), C.byref(s), C.byref(qsm))
        if rc:
            raise FrogError(rc, "frog_search_launch_info")
        return dict(grid=g.value, block=b.value, smem_bytes=s.value, queries_per_sm=qsm.value)
