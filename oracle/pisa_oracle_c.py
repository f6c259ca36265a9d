"""Loader and driver of the compiled CPU oracle (oracle/pisa_oracle_c.c).  TEST INFRASTRUCTURE ONLY.

`build()` compiles the C file with gcc (-O2 -fopenmp, no fast-math) into oracle/build/;
`CProblem` offers the drivers of `pisa_oracle.Problem` (route_all, attend_all, flat_mean_all, pyramid)
on top of it, one (batch, KV head) unit at a time with OpenMP over the sampled queries.  Only storage
conversion (bf16 bits / fp32 -> fp64) and the grouping of sampled rows by unit happen in Python; all
arithmetic of the method is in the C file.  Imported only by tests, the smoke check and the benchmark's
CPU-baseline leg.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from typing import List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pisa_oracle_c.c")
_OUT_DIR = os.path.join(_HERE, "build")
_LIB = os.path.join(_OUT_DIR, "libpisa_oracle_c.so")
_lib = None

_MODE = {"lse": 0, "mean": 1, "mean_var": 2}
_DTYPE = {"bf16": 0, "fp32": 1}


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", _LIB, _SRC, "-lm"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("gcc failed on the C oracle:\n" + r.stdout + r.stderr)
    return _LIB


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(build())
    dp, ip = C.POINTER(C.c_double), C.POINTER(C.c_int32)
    L.oc_round_storage.restype = C.c_double
    L.oc_round_storage.argtypes = [C.c_double, C.c_int]
    L.oc_round_storage_array.restype = None
    L.oc_round_storage_array.argtypes = [dp, C.c_int64, C.c_int]
    L.oc_hierarchy.restype = C.c_int
    L.oc_hierarchy.argtypes = [C.c_int, C.c_int, C.c_int, ip]
    L.oc_pyramid_elems.restype = C.c_int64
    L.oc_pyramid_elems.argtypes = [C.c_int] * 4
    L.oc_pyramid.restype = None
    L.oc_pyramid.argtypes = [dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, dp]
    L.oc_route.restype = None
    L.oc_route.argtypes = [dp, ip, C.c_int, C.c_int, dp, dp] + [C.c_int] * 5 + [C.c_double, C.c_int, ip, dp, C.c_int]
    L.oc_flat_mean.restype = None
    L.oc_flat_mean.argtypes = [dp, ip, C.c_int, C.c_int, dp, C.c_int, C.c_int, C.c_int, C.c_double, ip, dp, C.c_int]
    L.oc_attend.restype = None
    L.oc_attend.argtypes = [dp, ip, C.c_int, C.c_int, dp, dp] + [C.c_int] * 4 + [C.c_double, ip, dp, dp, C.c_int]
    L.oc_backward_rows.restype = None
    L.oc_backward_rows.argtypes = ([dp, dp, ip, C.c_int, C.c_int, dp, dp] + [C.c_int] * 4 +
                                   [C.c_double, ip, dp, dp, dp, C.c_int, C.c_int, C.c_int])
    L.oc_max_threads.restype = C.c_int
    _lib = L
    return L


def _d(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _i(a: np.ndarray):
    assert a.dtype == np.int32 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _widen(a: np.ndarray, dtype: str) -> np.ndarray:
    """Storage form (uint16 bf16 bits or float32) -> fp64 values (exact)."""
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return np.ascontiguousarray((a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64))
    return np.ascontiguousarray(a, dtype=np.float64)


def hierarchy(N: int, C_: int, g: int) -> List[int]:
    M = np.zeros(40, dtype=np.int32)
    L = lib().oc_hierarchy(N, C_, g, _i(M))
    return [int(x) for x in M[:L + 1]]


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    flat = np.array(x, dtype=np.float64).reshape(-1)
    lib().oc_round_storage_array(_d(flat), flat.size, _DTYPE[dtype])
    return flat.reshape(np.shape(x))


def max_threads() -> int:
    return int(lib().oc_max_threads())


class CProblem:
    """Drivers of the compiled oracle with the interface of pisa_oracle.Problem."""

    def __init__(self, q, k, v, *, C: int, g: int, K: int, dtype: str, scale: Optional[float] = None,
                 mode: str = "lse", threads: int = 0):
        self.q_st, self.k_st, self.v_st = q, k, v
        self.B, self.N, self.Hq, self.d = q.shape
        self.Hkv = k.shape[2]
        self.G = self.Hq // self.Hkv
        self.C, self.g, self.K, self.dtype, self.mode = C, g, K, dtype, mode
        self.scale = (1.0 / math.sqrt(self.d)) if scale is None else float(scale)
        self.M = hierarchy(self.N, C, g)
        self.L = len(self.M) - 1
        self.threads = threads if threads > 0 else max_threads()
        self._key, self._unit = None, None

    # one (batch, KV head) unit in fp64 --------------------------------------------------
    def unit(self, b: int, h: int):
        """(k [N,d], v [N,d] or None, levels: concatenated levels 1..L)."""
        if self._key != (b, h):
            k = _widen(np.ascontiguousarray(self.k_st[b, :, h, :]), self.dtype)
            v = None if self.v_st is None else _widen(np.ascontiguousarray(self.v_st[b, :, h, :]), self.dtype)
            levels = np.empty(int(lib().oc_pyramid_elems(self.N, self.d, self.C, self.g)), dtype=np.float64)
            lib().oc_pyramid(_d(k), self.N, self.d, self.C, self.g, _DTYPE[self.dtype], _d(levels))
            self._key, self._unit = (b, h), (k, v, levels)
        return self._unit

    def level(self, levels: np.ndarray, l: int) -> np.ndarray:
        off = sum(self.M[j] for j in range(1, l)) * self.d
        return levels[off:off + self.M[l] * self.d].reshape(self.M[l], self.d)

    def pyramid(self):
        out = [None] + [np.empty((self.B, self.Hkv, self.M[l], self.d)) for l in range(1, self.L + 1)]
        for b in range(self.B):
            for h in range(self.Hkv):
                lv = self.unit(b, h)[2]
                for l in range(1, self.L + 1):
                    out[l][b, h] = self.level(lv, l)
        return out

    def _q_rows(self, b: int, h: int, ps: np.ndarray) -> np.ndarray:
        rows = self.q_st[b, ps][:, h * self.G:(h + 1) * self.G, :]
        return _widen(np.ascontiguousarray(rows), self.dtype)

    @staticmethod
    def _groups(triples: np.ndarray):
        """Yields ((b, h), row numbers) for the sampled rows of each unit."""
        tri = np.asarray(triples, dtype=np.int64).reshape(-1, 3)
        keys = tri[:, 0] * (1 << 20) + tri[:, 1]
        for key in np.unique(keys):
            rows = np.nonzero(keys == key)[0]
            yield (int(tri[rows[0], 0]), int(tri[rows[0], 1])), rows

    # drivers ------------------------------------------------------------------------------
    def route_all(self, triples: np.ndarray):
        tri = np.asarray(triples, dtype=np.int64).reshape(-1, 3)
        idx = np.empty((len(tri), self.K), dtype=np.int32)
        margin = np.empty((len(tri),), dtype=np.float64)
        for (b, h), rows in self._groups(tri):
            k, _, levels = self.unit(b, h)
            ps = np.ascontiguousarray(tri[rows, 2], dtype=np.int32)
            q = self._q_rows(b, h, tri[rows, 2])
            i_u = np.empty((len(rows), self.K), dtype=np.int32)
            m_u = np.empty((len(rows),), dtype=np.float64)
            lib().oc_route(_d(q), _i(ps), len(rows), self.G, _d(k), _d(levels), self.N, self.d, self.C, self.g,
                           self.K, self.scale, _MODE[self.mode], _i(i_u), _d(m_u), self.threads)
            idx[rows], margin[rows] = i_u, m_u
        return idx, margin

    def flat_mean_all(self, triples: np.ndarray):
        tri = np.asarray(triples, dtype=np.int64).reshape(-1, 3)
        idx = np.empty((len(tri), self.K), dtype=np.int32)
        margin = np.empty((len(tri),), dtype=np.float64)
        for (b, h), rows in self._groups(tri):
            _, _, levels = self.unit(b, h)
            lvl1 = np.ascontiguousarray(self.level(levels, 1))
            ps = np.ascontiguousarray(tri[rows, 2], dtype=np.int32)
            q = self._q_rows(b, h, tri[rows, 2])
            i_u = np.empty((len(rows), self.K), dtype=np.int32)
            m_u = np.empty((len(rows),), dtype=np.float64)
            lib().oc_flat_mean(_d(q), _i(ps), len(rows), self.G, _d(lvl1), self.d, self.C, self.K, self.scale,
                               _i(i_u), _d(m_u), self.threads)
            idx[rows], margin[rows] = i_u, m_u
        return idx, margin

    def attend_raw(self, triples: np.ndarray, idx: np.ndarray):
        """Outputs before storage rounding [S, G, d] and natural-log denominators [S, G]."""
        tri = np.asarray(triples, dtype=np.int64).reshape(-1, 3)
        out = np.empty((len(tri), self.G, self.d), dtype=np.float64)
        lse = np.empty((len(tri), self.G), dtype=np.float64)
        for (b, h), rows in self._groups(tri):
            k, v, _ = self.unit(b, h)
            ps = np.ascontiguousarray(tri[rows, 2], dtype=np.int32)
            q = self._q_rows(b, h, tri[rows, 2])
            ix = np.ascontiguousarray(idx[rows], dtype=np.int32)
            o_u = np.empty((len(rows), self.G, self.d), dtype=np.float64)
            l_u = np.empty((len(rows), self.G), dtype=np.float64)
            lib().oc_attend(_d(q), _i(ps), len(rows), self.G, _d(k), _d(v), self.N, self.d, self.C, self.K,
                            self.scale, _i(ix), _d(o_u), _d(l_u), self.threads)
            out[rows], lse[rows] = o_u, l_u
        return out, lse

    def attend_all(self, triples: np.ndarray, idx: np.ndarray):
        """As pisa_oracle.Problem.attend_all: outputs rounded to the storage dtype (fp64 holding stored values)."""
        out, lse = self.attend_raw(triples, idx)
        return round_to_storage(out, self.dtype), lse

    def backward_rows(self, triples: np.ndarray, idx_rows: np.ndarray, dout_rows: np.ndarray,
                      key_range=None):
        """dq [S, G, d] of the sampled rows (all of ONE unit when key_range is given) and, with
        key_range = (lo, hi), the rows' summed contributions to dk, dv of keys lo..hi-1 as [hi-lo, d]."""
        tri = np.asarray(triples, dtype=np.int64).reshape(-1, 3)
        dq = np.empty((len(tri), self.G, self.d), dtype=np.float64)
        dk = dv = None
        groups = list(self._groups(tri))
        if key_range is not None:
            assert len(groups) == 1, "key gradients are per unit"
            dk = np.zeros((self.N, self.d))
            dv = np.zeros((self.N, self.d))
        for (b, h), rows in groups:
            k, v, _ = self.unit(b, h)
            ps = np.ascontiguousarray(tri[rows, 2], dtype=np.int32)
            q = self._q_rows(b, h, tri[rows, 2])
            do = _widen(np.ascontiguousarray(dout_rows[rows]), self.dtype)
            ix = np.ascontiguousarray(idx_rows[rows], dtype=np.int32)
            dq_u = np.empty((len(rows), self.G, self.d), dtype=np.float64)
            lo, hi = key_range if key_range is not None else (0, 0)
            lib().oc_backward_rows(_d(q), _d(do), _i(ps), len(rows), self.G, _d(k), _d(v), self.N, self.d, self.C,
                                   self.K, self.scale, _i(ix), _d(dq_u),
                                   _d(dk) if dk is not None else None, _d(dv) if dv is not None else None,
                                   int(lo), int(hi), self.threads)
            dq[rows] = dq_u
        if key_range is not None:
            lo, hi = key_range
            return dq, dk[lo:hi].copy(), dv[lo:hi].copy()
        return dq
