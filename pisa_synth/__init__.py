"""Seeded synthetic inputs for the PISA forward path.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds none of the method's arithmetic (no pooling, scoring,
selection or attention): it only draws random tensors with the structure of
the paper's own selection benchmark (seeded random tensors, App. B) plus the
planted structure the workload table asks for, and converts fp32 values to bf16 bit patterns.

Layouts: q is [B, N, Hq, d]; k and v are [B, N, Hkv, d]; d contiguous.
bf16 tensors are returned as numpy uint16 bit patterns (numpy has no bf16).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np

__all__ = [
    "Workload",
    "WORKLOADS",
    "sweep_workload",
    "make_inputs",
    "f32_to_bf16_bits",
    "bf16_bits_to_f32",
    "sample_queries",
]


@dataclasses.dataclass(frozen=True)
class Workload:
    """One problem instance, in the paper's notation (Sec. 3.1-3.2)."""

    name: str
    B: int
    N: int
    Hq: int
    Hkv: int
    d: int
    C: int          # leaf block size
    g: int          # pooling fan-in above the leaves
    K: int          # block budget
    dtype: str      # "bf16" | "fp32"
    seed: int
    structure: str  # "iid" | "needle1" | "walk" | "needle64"
    q_scale: float = 1.0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def M1(self) -> int:
        return -(-self.N // self.C)


WORKLOADS: Dict[str, Workload] = {
    # tiny fp32 case
    "cfg1": Workload("cfg1", 1, 1024, 1, 1, 64, 64, 2, 4, "fp32", 0, "iid"),
    # MHA, one planted needle block per head, q scaled by 1/sqrt(d)
    "cfg2": Workload("cfg2", 1, 8192, 16, 16, 128, 64, 2, 16, "bf16", 1, "needle1",
                     q_scale=1.0 / math.sqrt(128.0)),
    # GQA, fan-in 4, random-walk mean
    "cfg3": Workload("cfg3", 2, 32768, 32, 8, 128, 64, 4, 16, "bf16", 2, "walk"),
    # headline workload
    "cfg4": Workload("cfg4", 1, 131072, 32, 8, 128, 128, 2, 32, "bf16", 3, "needle64"),
    # the paper's own benchmark shape (App. B), for a like-for-like row
    "paper128k": Workload("paper128k", 1, 131072, 32, 2, 64, 64, 2, 8, "bf16", 5, "iid"),
}


def sweep_workload(N: int) -> Workload:
    """The scaling sweep, one instance per N."""
    return Workload(f"cfg5_{N}", 1, N, 16, 4, 128, 64, 2, 16, "bf16", 4, "iid")


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> the fp32 value it denotes (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    return np.ascontiguousarray(x, dtype=np.float32)


def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def make_inputs(w: Workload, *, B: Optional[int] = None) -> dict:
    """Draw q, k, v for workload `w`.

    Returns {"q","k","v"} in storage form (uint16 bf16 bits or float32), plus
    "needles": int64 array [B, Hkv, n_needles, 2] of (leaf block, target query
    position) for the planted structures (empty for the others).
    """
    Bn = w.B if B is None else B
    ss = np.random.SeedSequence([w.seed, w.N, w.Hq, w.Hkv, w.d])
    s_q, s_k, s_v, s_n = ss.spawn(4)
    rq, rk, rv, rn = (np.random.Generator(np.random.PCG64(s)) for s in (s_q, s_k, s_v, s_n))

    q = _normal(rq, (Bn, w.N, w.Hq, w.d))
    k = _normal(rk, (Bn, w.N, w.Hkv, w.d))
    v = _normal(rv, (Bn, w.N, w.Hkv, w.d))
    if w.q_scale != 1.0:
        q *= np.float32(w.q_scale)

    needles = np.zeros((Bn, w.Hkv, 0, 2), dtype=np.int64)
    if w.structure == "walk":
        # slowly drifting per-position mean: independent random walk (step 0.02)
        # per tensor / batch / head, cumulated in fp64
        for t, r, H in ((q, rq, w.Hq), (k, rk, w.Hkv), (v, rv, w.Hkv)):
            for b in range(Bn):
                for h in range(H):
                    steps = r.standard_normal((w.N, w.d))
                    mu = np.cumsum(0.02 * steps, axis=0)
                    mu = np.vstack([np.zeros((1, w.d)), mu[:-1]])
                    t[b, :, h, :] += mu.astype(np.float32)
    elif w.structure in ("needle1", "needle64"):
        n_needles = 1 if w.structure == "needle1" else 64
        M1 = w.M1
        n_needles = min(n_needles, max(0, M1 - 3))
        needles = np.zeros((Bn, w.Hkv, n_needles, 2), dtype=np.int64)
        # the planted keys copy the direction of the (already stored) query
        q_st = bf16_bits_to_f32(f32_to_bf16_bits(q)) if w.dtype == "bf16" else q
        for b in range(Bn):
            for h in range(w.Hkv):
                blocks = rn.choice(np.arange(1, M1 - 2), size=n_needles, replace=False)
                for j, blk in enumerate(blocks):
                    lo = (int(blk) + 2) * w.C
                    t_star = int(rn.integers(lo, w.N)) if lo < w.N else w.N - 1
                    qv = q_st[b, t_star, h * w.G, :].astype(np.float64)
                    nrm = float(np.sqrt(np.sum(qv * qv)))
                    key = (4.0 * qv / max(nrm, 1e-30)).astype(np.float32)
                    k[b, int(blk) * w.C:min((int(blk) + 1) * w.C, w.N), h, :] = key
                    needles[b, h, j, 0] = int(blk)
                    needles[b, h, j, 1] = t_star
    elif w.structure != "iid":
        raise ValueError(f"unknown structure {w.structure!r}")

    return {"q": _store(q, w.dtype), "k": _store(k, w.dtype), "v": _store(v, w.dtype),
            "needles": needles, "workload": w}


def sample_queries(w: Workload, n_per_head: int, seed: int = 1234, *, B: Optional[int] = None) -> np.ndarray:
    """A stratified sample of (b, kv head, position) triples, int64 [S, 3].

    Per (b, kv head): the first few positions, both sides of the boundary where
    pruning starts (K*C), block boundaries, the last positions, and a uniform
    remainder; duplicates removed.
    """
    Bn = w.B if B is None else B
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, w.N, w.K])))
    out = []
    for b in range(Bn):
        for h in range(w.Hkv):
            fixed = [0, 1, w.C - 1, w.C, w.C + 1, 2 * w.C, 3 * w.C - 1, 3 * w.C,
                     w.K * w.C - 1, w.K * w.C, w.K * w.C + 1,
                     w.g * w.K * w.C - 1, w.g * w.K * w.C, w.N - w.C - 1, w.N - w.C, w.N - 2, w.N - 1]
            fixed = [p for p in fixed if 0 <= p < w.N]
            n_rand = max(0, n_per_head - len(fixed))
            rand = rng.integers(0, w.N, size=n_rand).tolist()
            # a few exact block boundaries deep in the sequence
            nb = min(8, n_rand)
            bounds = (rng.integers(1, max(2, w.M1), size=nb) * w.C).tolist()
            ps = sorted(set(fixed + rand + [p for p in bounds if p < w.N]))
            out.extend((b, h, p) for p in ps)
    return np.asarray(out, dtype=np.int64).reshape(-1, 3)
