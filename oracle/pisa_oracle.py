"""CPU oracle for the PISA forward path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct NumPy restatement (fp64 arithmetic) of what
the path computes, written from the paper's definitions.  It is imported only
by the tests, by the smoke check and by the benchmark's CPU-baseline leg; the
CUDA library never calls it and shares no code with it.

What follows which passage of the paper:

* `hierarchy`            Sec. 3.2 "Fine-to-coarse block aggregation": M_0 = N,
                         g_0 = C, g_l = g, M_{l+1} = ceil(M_l / g_l), Ch_l(i).
* `build_pyramid`        Eq. "mean pyramid": a summary is the unweighted mean of
                         its valid child summaries, level 0 being the raw keys.
* `lse_score`            Eq. "direct child LSE": log-sum-exp over the children's
                         scaled dot products (C raw keys at the leaf level, g
                         child summaries above it).
* `route_query`          Sec. 3.2 "Coarse-to-fine block selection" (candidate
                         sets A, Select_K, expansion), Eq. "grouped score"
                         (sum of the group's per-head scores), App. B "Causal
                         masking" (eligibility, forced first / previous /
                         current blocks and their ancestor paths).
* `attend_query`         Eq. "selected sparse attention" with the causal mask
                         inside selected blocks (App. B).
* `flat_lse_select`      exhaustive variant of the same leaf score (no pruning).
* `flat_mean_select`     Sec. 3.1 flat BSA: mean-pooled summaries, one score
                         per block, per-head normalisation before the head sum
                         (App. C), Top-K.
* `score_mode`           Sec. 4.3 / App. A.2: "lse" (PISA), "mean" (PISA-1),
                         "mean_var" (PISA-2).
* `attend_backward`      App. B: backward of the selected sparse attention with the
                         selected indices held fixed (softmax-attention gradients
                         restricted to the selected, visible keys).
* `decode_pyramid`,      Sec. 3.3 "Decoding" and App. B "Decode cache": when the
  `decode_step`          token at position p is generated the cached pyramid
                         holds the means of the keys seen so far, i.e. it is the
                         pyramid of the (p+1)-token sequence; selection walks
                         all levels down to the raw key blocks for that one
                         query and attention runs over the selected blocks.

Readings taken where the paper is silent (all 0-based here):
  - summaries are stored in the input dtype (bf16 or fp32, round to nearest
    even) and every level is pooled from the *stored* level below;
  - forced nodes count inside the budget K at every level and are never scored;
  - "at most K candidates" counts candidates after the existence and causal
    filters; ties in Select_K go to the smaller block index;
  - heads h*G .. h*G+G-1 share KV head h;
  - indices are returned ascending, padded with -1.

Pins (tests/test_oracle_pins.py): closed forms for the pyramid, identical-key
blocks for the leaf score, softmax block mass ranking, Jensen sandwich and the
Taylor identity for the intermediate score, a textbook flat Top-K built from
torch.logsumexp/topk in the unpruned regime, torch's dense causal attention
when K*C >= N, a hand-derived pruned example (tests/golden), and structural
invariants.  The pruned regime has no external numeric anchor beyond the
hand-derived example and the invariants.  Decoding is pinned by what the
definitions imply: the step at position p selects what the prefill of any
longer sequence selects for row p (every scored node lies strictly in the past),
equals torch's dense causal attention when K*C > p, and the cached pyramid's
completed nodes equal those of the longer sequence's pyramid.  The backward is
pinned by torch autograd on a dense masked attention built from the same index
sets and by finite differences of the forward (tests/test_oracle_backward_pins.py).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

NEG_INF = -np.inf


# --------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bits with a single round-to-nearest-even.

    Goes through fp32 with round-to-odd first, which makes the second rounding
    (fp32 -> bf16) exact with respect to the fp64 value.
    """
    x = np.asarray(x, dtype=np.float64)
    f = x.astype(np.float32)
    back = f.astype(np.float64)
    inexact = back != x
    # truncate toward zero where the fp32 rounding went away from zero
    away = inexact & (np.abs(back) > np.abs(x))
    f = np.where(away, np.nextafter(f, np.float32(0.0)), f).astype(np.float32)
    u = f.view(np.uint32).copy()
    u[inexact] |= np.uint32(1)  # sticky bit (round to odd)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 values to the storage dtype; result is fp64 holding the stored value."""
    if dtype == "bf16":
        return bf16_bits_to_f64(f64_to_bf16_bits(x))
    if dtype == "fp32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    raise ValueError(dtype)


def load_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Storage form (uint16 bf16 bits or float32) -> fp64 values."""
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return bf16_bits_to_f64(a)
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# hierarchy and pyramid
# --------------------------------------------------------------------------

def hierarchy(N: int, C: int, g: int) -> List[int]:
    """Block counts M[0..L]; M[0] = N, M[1] = ceil(N/C), M[l+1] = ceil(M[l]/g), M[L] = 1."""
    assert N >= 1 and C >= 1 and g >= 2
    M = [N, -(-N // C)]
    while M[-1] > 1:
        M.append(-(-M[-1] // g))
    return M


def children(level: int, i: int, M: Sequence[int], C: int, g: int) -> range:
    """Indices at level-1 of the children of node i of `level` (level >= 1)."""
    fan = C if level == 1 else g
    return range(i * fan, min((i + 1) * fan, M[level - 1]))


def build_pyramid(k: np.ndarray, C: int, g: int, dtype: str) -> List[Optional[np.ndarray]]:
    """k: fp64 values [B, N, Hkv, d].  Returns levels[0..L]; levels[0] is None
    (the raw keys), levels[l] is fp64 [B, Hkv, M_l, d] holding stored values."""
    B, N, Hkv, d = k.shape
    M = hierarchy(N, C, g)
    L = len(M) - 1
    levels: List[Optional[np.ndarray]] = [None]
    below = np.transpose(k, (0, 2, 1, 3))  # [B, Hkv, N, d]
    for l in range(1, L + 1):
        cur = np.empty((B, Hkv, M[l], d), dtype=np.float64)
        for i in range(M[l]):
            ch = children(l, i, M, C, g)
            cur[:, :, i, :] = below[:, :, ch.start:ch.stop, :].sum(axis=2) / float(len(ch))
        cur = round_to_storage(cur, dtype)
        levels.append(cur)
        below = cur
    return levels


# --------------------------------------------------------------------------
# scores
# --------------------------------------------------------------------------

def _logsumexp(z: np.ndarray, axis: int) -> np.ndarray:
    m = np.max(z, axis=axis, keepdims=True)
    return np.squeeze(m, axis=axis) + np.log(np.sum(np.exp(z - m), axis=axis))


def block_score(z: np.ndarray, mode: str = "lse") -> np.ndarray:
    """z: logits [..., m] of one candidate's children for one head."""
    if mode == "lse":
        return _logsumexp(z, axis=-1)
    zbar = z.mean(axis=-1)
    if mode == "mean":
        return zbar
    if mode == "mean_var":
        return zbar + 0.5 * ((z - zbar[..., None]) ** 2).mean(axis=-1)
    raise ValueError(mode)


def lse_score(q_heads: np.ndarray, x_children: np.ndarray, scale: float, mode: str = "lse") -> float:
    """Grouped score of one candidate: sum over the group's heads of the block
    score of the children's scaled dot products.  q_heads [G, d], x_children [m, d]."""
    z = (q_heads @ x_children.T) * scale          # [G, m]
    return float(np.sum(block_score(z, mode)))


# --------------------------------------------------------------------------
# routing
# --------------------------------------------------------------------------

def forced_nodes(level: int, c: int, g: int) -> List[int]:
    """Level-`level` ancestors of the first, previous and current leaf (deduplicated)."""
    span = g ** (level - 1)
    out = {0 // span, c // span}
    if c >= 1:
        out.add((c - 1) // span)
    return sorted(out)


def _select(valid: List[int], forced: List[int], scores: dict, K: int) -> Tuple[List[int], float]:
    """forced ∪ top-(K - |forced|) of the rest by score (desc., ties -> smaller index).
    Also returns the relative gap at the cut."""
    rest = [i for i in valid if i not in forced]
    keep = K - len(forced)
    order = sorted(rest, key=lambda i: (-scores[i], i))
    chosen = order[:keep]
    gap = math.inf
    if 0 < keep < len(order):
        a, b = scores[order[keep - 1]], scores[order[keep]]
        gap = (a - b) / max(abs(a), 1.0)
    return sorted(set(forced) | set(chosen)), gap


def route_query(q_heads: np.ndarray, levels_bh: Sequence[Optional[np.ndarray]], k_bh: np.ndarray,
                p: int, C: int, g: int, K: int, scale: float, mode: str = "lse",
                trace: Optional[list] = None) -> Tuple[List[int], float]:
    """Selected leaf blocks for query position p of one (batch, KV head).

    q_heads [G, d] (the group's query vectors at p); levels_bh[l] [M_l, d];
    k_bh [N, d].  Returns (ascending leaf indices, min relative cut margin
    over the scored levels).
    """
    N = k_bh.shape[0]
    M = hierarchy(N, C, g)
    L = len(M) - 1
    assert K >= 3
    c = p // C
    A = [0]
    margin = math.inf
    I: List[int] = []
    for l in range(L, 0, -1):
        span = g ** (l - 1)
        anc_c = c // span
        V = [i for i in A if i < M[l] and i <= anc_c]
        F = forced_nodes(l, c, g)
        assert all(f in V for f in F), "forced nodes must be candidates"
        scored = False
        if len(V) <= K:
            I = list(V)
        else:
            scores = {}
            for i in V:
                if i in F:
                    continue
                ch = children(l, i, M, C, g)
                x = k_bh[ch.start:ch.stop] if l == 1 else levels_bh[l - 1][ch.start:ch.stop]
                if l == 1:
                    assert ch.stop - 1 < p, "scored leaves lie entirely in the past"
                scores[i] = lse_score(q_heads, x, scale, mode)
            I, gap = _select(V, F, scores, K)
            margin = min(margin, gap)
            scored = True
        if trace is not None:
            trace.append({"level": l, "A": list(A), "V": list(V), "F": list(F), "I": list(I), "scored": scored})
        if l > 1:
            A = [r for i in I for r in children(l, i, M, C, g)]
    return sorted(I), margin


def flat_lse_select(q_heads: np.ndarray, k_bh: np.ndarray, p: int, C: int, K: int, scale: float,
                    mode: str = "lse") -> List[int]:
    """Exhaustive selection with the leaf score: every eligible non-forced leaf is scored."""
    N = k_bh.shape[0]
    c = p // C
    V = list(range(c + 1))
    F = forced_nodes(1, c, 2)
    if len(V) <= K:
        return V
    scores = {i: lse_score(q_heads, k_bh[i * C:min((i + 1) * C, N)], scale, mode) for i in V if i not in F}
    I, _ = _select(V, F, scores, K)
    return I


def flat_mean_select(q_heads: np.ndarray, level1_bh: np.ndarray, p: int, C: int, K: int,
                     scale: float) -> Tuple[List[int], float]:
    """Flat BSA (Sec. 3.1): s = q . kbar_i * scale for every eligible leaf; softmax over the
    eligible leaves within each head; sum over the group's heads; forced ∪ top."""
    c = p // C
    V = list(range(c + 1))
    F = forced_nodes(1, c, 2)
    if len(V) <= K:
        return V, math.inf
    s = (q_heads @ level1_bh[:c + 1].T) * scale            # [G, c+1]
    s = s - s.max(axis=1, keepdims=True)
    w = np.exp(s)
    w = w / w.sum(axis=1, keepdims=True)
    u = w.sum(axis=0)                                      # [c+1]
    scores = {i: float(u[i]) for i in V if i not in F}
    return _select(V, F, scores, K)


def pad_indices(I: Sequence[int], K: int) -> np.ndarray:
    out = np.full((K,), -1, dtype=np.int32)
    out[:len(I)] = np.asarray(sorted(I), dtype=np.int32)
    return out


# --------------------------------------------------------------------------
# attention
# --------------------------------------------------------------------------

def attend_query(q_vec: np.ndarray, k_bh: np.ndarray, v_bh: np.ndarray, p: int, blocks: Sequence[int],
                 C: int, scale: float) -> Tuple[np.ndarray, float]:
    """One query head at position p over the tokens j <= p of the selected blocks.
    Returns (output [d] in fp64 before storage rounding, natural-log softmax denominator)."""
    N = k_bh.shape[0]
    toks: List[int] = []
    for i in blocks:
        if i < 0:
            continue
        toks.extend(j for j in range(i * C, min((i + 1) * C, N)) if j <= p)
    toks_a = np.asarray(toks, dtype=np.int64)
    z = (k_bh[toks_a] @ q_vec) * scale
    m = z.max()
    e = np.exp(z - m)
    den = e.sum()
    out = (e[:, None] * v_bh[toks_a]).sum(axis=0) / den
    return out, float(m + math.log(den))


# --------------------------------------------------------------------------
# whole-problem drivers (loops over queries; use on small shapes or samples)
# --------------------------------------------------------------------------

class Problem:
    """One problem's tensors in storage form plus lazily built per-(b, KV head) fp64 views
    (raw keys, values, pyramid levels), so that sampled queries of a long sequence stay cheap."""

    def __init__(self, q, k, v, *, C: int, g: int, K: int, dtype: str, scale: Optional[float] = None,
                 mode: str = "lse"):
        self.q_st, self.k_st, self.v_st = q, k, v      # [B,N,Hq,d], [B,N,Hkv,d] storage form
        self.B, self.N, self.Hq, self.d = q.shape
        self.Hkv = k.shape[2]
        assert self.Hq % self.Hkv == 0
        self.G = self.Hq // self.Hkv
        self.C, self.g, self.K, self.dtype, self.mode = C, g, K, dtype, mode
        self.scale = (1.0 / math.sqrt(self.d)) if scale is None else float(scale)
        self.M = hierarchy(self.N, C, g)
        self.L = len(self.M) - 1
        self._cache_key = None
        self._cache = None

    # fp64 views -----------------------------------------------------------
    def head(self, b: int, h: int):
        """(k_bh [N,d], v_bh [N,d] or None, levels_bh[0..L] with levels_bh[l] [M_l,d])."""
        if self._cache_key != (b, h):
            k_bh = load_storage(np.ascontiguousarray(self.k_st[b, :, h, :]), self.dtype)
            v_bh = None if self.v_st is None else load_storage(np.ascontiguousarray(self.v_st[b, :, h, :]), self.dtype)
            lv = build_pyramid(k_bh[None, :, None, :], self.C, self.g, self.dtype)
            levels = [None] + [lv[l][0, 0] for l in range(1, self.L + 1)]
            self._cache_key, self._cache = (b, h), (k_bh, v_bh, levels)
        return self._cache

    def q_group(self, b: int, h: int, p: int) -> np.ndarray:
        return load_storage(np.ascontiguousarray(self.q_st[b, p, h * self.G:(h + 1) * self.G, :]), self.dtype)

    def pyramid(self) -> List[Optional[np.ndarray]]:
        """All levels, fp64 stored values, levels[l] [B,Hkv,M_l,d]."""
        out: List[Optional[np.ndarray]] = [None] + [np.empty((self.B, self.Hkv, self.M[l], self.d))
                                                     for l in range(1, self.L + 1)]
        for b in range(self.B):
            for h in range(self.Hkv):
                lv = self.head(b, h)[2]
                for l in range(1, self.L + 1):
                    out[l][b, h] = lv[l]
        return out

    # per-query ------------------------------------------------------------
    def route(self, b: int, h: int, p: int, trace: Optional[list] = None):
        k_bh, _, lv = self.head(b, h)
        return route_query(self.q_group(b, h, p), lv, k_bh, p, self.C, self.g, self.K, self.scale, self.mode, trace)

    def flat_lse(self, b: int, h: int, p: int):
        k_bh, _, _ = self.head(b, h)
        return flat_lse_select(self.q_group(b, h, p), k_bh, p, self.C, self.K, self.scale, self.mode)

    def flat_mean(self, b: int, h: int, p: int):
        _, _, lv = self.head(b, h)
        return flat_mean_select(self.q_group(b, h, p), lv[1], p, self.C, self.K, self.scale)

    def attend(self, b: int, hq: int, p: int, blocks: Sequence[int]):
        h = hq // self.G
        k_bh, v_bh, _ = self.head(b, h)
        qv = self.q_group(b, h, p)[hq - h * self.G]
        return attend_query(qv, k_bh, v_bh, p, blocks, self.C, self.scale)

    # drivers (loops over queries; use on small shapes or samples) -----------
    def all_triples(self) -> np.ndarray:
        return np.asarray([(b, h, p) for b in range(self.B) for h in range(self.Hkv)
                           for p in range(self.N)], dtype=np.int64)

    def route_all(self, triples: Optional[np.ndarray] = None):
        """idx int32 [S, K], margin fp64 [S] for the given (b, h, p) triples
        (default: every query, in (b, h, p) order)."""
        if triples is None:
            triples = self.all_triples()
        idx = np.empty((len(triples), self.K), dtype=np.int32)
        margin = np.empty((len(triples),), dtype=np.float64)
        for s, (b, h, p) in enumerate(triples):
            I, m = self.route(int(b), int(h), int(p))
            idx[s] = pad_indices(I, self.K)
            margin[s] = m
        return idx, margin

    def flat_mean_all(self, triples: np.ndarray):
        idx = np.empty((len(triples), self.K), dtype=np.int32)
        margin = np.empty((len(triples),), dtype=np.float64)
        for s, (b, h, p) in enumerate(triples):
            I, m = self.flat_mean(int(b), int(h), int(p))
            idx[s] = pad_indices(I, self.K)
            margin[s] = m
        return idx, margin

    def attend_all(self, triples: np.ndarray, idx: np.ndarray):
        """For each (b, h, p) and its block list idx[s]: the G heads' outputs (stored values,
        fp64 [S, G, d]) and natural-log denominators [S, G]."""
        S = len(triples)
        out = np.empty((S, self.G, self.d), dtype=np.float64)
        lse = np.empty((S, self.G), dtype=np.float64)
        for s, (b, h, p) in enumerate(triples):
            for j in range(self.G):
                o, l = self.attend(int(b), int(h) * self.G + j, int(p), idx[s])
                out[s, j] = o
                lse[s, j] = l
        return round_to_storage(out, self.dtype), lse


# --------------------------------------------------------------------------
# decoding (Sec. 3.3 "Decoding", App. B "Decode cache")
# --------------------------------------------------------------------------

def decode_pyramid(k_cache, pos: int, C: int, g: int, dtype: str) -> List[Optional[np.ndarray]]:
    """The cached pyramid after the token at `pos` has been appended: the mean pyramid of keys
    0..pos (each summary the mean of its valid children, the last leaf the mean of the keys it
    holds so far).  k_cache: [B, Ncap, Hkv, d] in storage form; returns levels[l] [B,Hkv,M_l(pos+1),d]."""
    k = load_storage(np.ascontiguousarray(k_cache[:, :pos + 1]), dtype)
    return build_pyramid(k, C, g, dtype)


def decode_step(q_new, k_cache, v_cache, pos: int, *, C: int, g: int, K: int, dtype: str,
                scale: Optional[float] = None, mode: str = "lse"):
    """One decoding step for the token at position `pos` (its key and value already in the caches).

    q_new: [B, Hq, d] storage form; k_cache, v_cache: [B, Ncap, Hkv, d] storage form, rows 0..pos valid.
    Returns idx int32 [B, Hkv, K] (ascending, -1 padded), margin [B, Hkv], out fp64 [B, Hq, d]
    (stored values) and lse [B, Hq]."""
    B, Hq, d = q_new.shape
    n = pos + 1
    q_seq = np.zeros((B, n, Hq, d), dtype=q_new.dtype)
    q_seq[:, pos] = q_new
    prob = Problem(q_seq, np.ascontiguousarray(k_cache[:, :n]), np.ascontiguousarray(v_cache[:, :n]),
                   C=C, g=g, K=K, dtype=dtype, scale=scale, mode=mode)
    idx = np.empty((B, prob.Hkv, K), dtype=np.int32)
    margin = np.empty((B, prob.Hkv), dtype=np.float64)
    out = np.empty((B, Hq, d), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    for b in range(B):
        for h in range(prob.Hkv):
            I, m = prob.route(b, h, pos)
            idx[b, h] = pad_indices(I, K)
            margin[b, h] = m
            for hq in range(h * prob.G, (h + 1) * prob.G):
                out[b, hq], lse[b, hq] = prob.attend(b, hq, pos, I)
    return idx, margin, round_to_storage(out, dtype), lse


# --------------------------------------------------------------------------
# backward of the selected sparse attention with frozen indices (App. B)
# --------------------------------------------------------------------------

def _backward_row(q_heads, k_bh, v_bh, do_heads, toks, sc):
    """One (b, KV head, position): q_heads, do_heads [G, d]; toks = its visible selected keys.
    Returns dq [G, d] and this row's contributions dk, dv [len(toks), d]."""
    G, d = q_heads.shape
    dq = np.zeros((G, d))
    dk = np.zeros((len(toks), d))
    dv = np.zeros((len(toks), d))
    for j in range(G):
        z = (k_bh[toks] @ q_heads[j]) * sc
        e = np.exp(z - z.max())
        pr = e / e.sum()
        dp = v_bh[toks] @ do_heads[j]
        ds = pr * (dp - float(pr @ dp))
        dq[j] = sc * (ds @ k_bh[toks])
        dk += sc * ds[:, None] * q_heads[j][None, :]
        dv += pr[:, None] * do_heads[j][None, :]
    return dq, dk, dv


def _visible_tokens(blocks, p: int, C: int, N: int) -> np.ndarray:
    toks: List[int] = []
    for i in blocks:
        if i >= 0:
            toks.extend(j for j in range(int(i) * C, min((int(i) + 1) * C, N)) if j <= p)
    return np.asarray(toks, dtype=np.int64)


def attend_backward(q, k, v, idx, dout, *, C: int, dtype: str, scale: Optional[float] = None):
    """Gradients of Eq. "selected sparse attention" with the selected block indices held fixed
    (App. B): idx is a constant, only q, k and v receive gradients.

    q, dout: [B, N, Hq, d]; k, v: [B, N, Hkv, d] storage form; idx: int [B, Hkv, N, K] (-1 padded).
    For one query row with probabilities p_j over its visible selected keys, o = sum_j p_j v_j:
        dv_j += p_j do,   dp_j = do . v_j,   ds_j = p_j (dp_j - sum_i p_i dp_i),
        dq   += scale * sum_j ds_j k_j,      dk_j += scale * ds_j q.
    Returns dq [B,N,Hq,d], dk, dv [B,N,Hkv,d] in fp64 (not rounded to the storage dtype)."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    sc = (1.0 / math.sqrt(d)) if scale is None else float(scale)
    qf, kf, vf, dof = (load_storage(np.ascontiguousarray(x), dtype) for x in (q, k, v, dout))
    dq = np.zeros((B, N, Hq, d))
    dk = np.zeros((B, N, Hkv, d))
    dv = np.zeros((B, N, Hkv, d))
    for b in range(B):
        for h in range(Hkv):
            k_bh, v_bh = kf[b, :, h], vf[b, :, h]
            for p in range(N):
                ta = _visible_tokens(idx[b, h, p], p, C, N)
                if len(ta) == 0:
                    continue
                rq, rk, rv = _backward_row(qf[b, p, h * G:(h + 1) * G], k_bh, v_bh, dof[b, p, h * G:(h + 1) * G], ta, sc)
                dq[b, p, h * G:(h + 1) * G] = rq
                dk[b, ta, h] += rk
                dv[b, ta, h] += rv
    return dq, dk, dv


def attend_backward_dq_rows(prob: "Problem", triples, idx_rows, dout_rows):
    """dq of sampled queries of a long sequence: triples [S, 3] (b, KV head, position), idx_rows [S, K],
    dout_rows [S, G, d] storage form.  Returns fp64 [S, G, d]."""
    out = np.empty((len(triples), prob.G, prob.d))
    for s, (b, h, p) in enumerate(triples):
        k_bh, v_bh, _ = prob.head(int(b), int(h))
        ta = _visible_tokens(idx_rows[s], int(p), prob.C, prob.N)
        do = load_storage(np.ascontiguousarray(dout_rows[s]), prob.dtype)
        out[s] = _backward_row(prob.q_group(int(b), int(h), int(p)), k_bh, v_bh, do, ta, prob.scale)[0]
    return out
