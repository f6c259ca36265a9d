"""Pins for the compiled oracle (oracle/pisa_oracle_c.c): closed forms, library routines, the
hand-derived pruned example, and the NumPy oracle as a second, independently written witness on the
shapes that have no external anchor (fan-in 4, several heads per group, ragged hierarchies)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import pisa_oracle as O
from oracle import pisa_oracle_c as OC
import pisa_synth as S

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cproblem(w, B=None, mode="lse"):
    t = S.make_inputs(w, B=B)
    return OC.CProblem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype, mode=mode), t


def _all_triples(P):
    return np.asarray([(b, h, p) for b in range(P.B) for h in range(P.Hkv) for p in range(P.N)], dtype=np.int64)


# ---------------------------------------------------------------- storage rounding, hierarchy, pyramid

def test_c_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        np.array([0.0, 1.0, 1.00390625, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9, 255.5, 1e-40])])
    ours = OC.round_to_storage(x, "bf16")
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, ref)
    # a single rounding from fp64: just above / below / at the midpoint of two bf16 neighbours (a route
    # through fp32 would lose the 2^-40 and round both to the even neighbour)
    ulp = 2.0 ** -7
    tricky = np.array([1.0 + ulp / 2 + 2.0 ** -40, 1.0 + ulp / 2 - 2.0 ** -40, 1.0 + ulp / 2, 1.0 + 3 * ulp / 2])
    assert OC.round_to_storage(tricky, "bf16").tolist() == [1.0 + ulp, 1.0, 1.0, 1.0 + 2 * ulp]
    x32 = OC.round_to_storage(x, "fp32")
    assert np.array_equal(x32, x.astype(np.float32).astype(np.float64))


def test_c_hierarchy_counts():
    assert OC.hierarchy(1024, 64, 2) == [1024, 16, 8, 4, 2, 1]
    assert OC.hierarchy(32768, 64, 4) == [32768, 512, 128, 32, 8, 2, 1]
    assert OC.hierarchy(1000, 24, 3) == [1000, 42, 14, 5, 2, 1]
    assert OC.hierarchy(40, 8, 2) == [40, 5, 3, 2, 1]


def test_c_pyramid_closed_forms():
    rng = np.random.default_rng(1)
    N, d, C, g = 512, 8, 16, 2
    k = rng.standard_normal((1, N, 1, d)).astype(np.float32)
    P = OC.CProblem(k, k, k, C=C, g=g, K=4, dtype="fp32")
    lv = P.pyramid()
    for l in range(1, P.L + 1):                      # equal children: the mean of all raw keys spanned
        span = C * g ** (l - 1)
        ref = k.astype(np.float64).reshape(1, P.M[l], span, 1, d).mean(axis=2).transpose(0, 2, 1, 3)
        np.testing.assert_allclose(lv[l], ref, rtol=0, atol=3e-7 * l)
    const = np.full((1, 256, 1, 4), 0.375, dtype=np.float32)
    Pc = OC.CProblem(const, const, const, C=8, g=4, K=4, dtype="fp32")
    assert all(np.all(a == 0.375) for a in Pc.pyramid()[1:])
    # ragged: mean of means, by hand (N = 37, C = 8, g = 2)
    kr = rng.standard_normal((1, 37, 1, 3)).astype(np.float32)
    Pr = OC.CProblem(kr, kr, kr, C=8, g=2, K=4, dtype="fp32")
    lr = Pr.pyramid()
    kk = kr[0, :, 0, :].astype(np.float64)
    f32 = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    s = [f32(kk[i * 8:min(i * 8 + 8, 37)].mean(axis=0)) for i in range(5)]
    np.testing.assert_array_equal(lr[1][0, 0], np.stack(s))
    l2 = [f32((s[0] + s[1]) / 2), f32((s[2] + s[3]) / 2), s[4]]
    np.testing.assert_array_equal(lr[2][0, 0], np.stack(l2))
    l3 = [f32((l2[0] + l2[1]) / 2), l2[2]]
    np.testing.assert_array_equal(lr[3][0, 0], np.stack(l3))


# ---------------------------------------------------------------- routing

def _textbook_flat_topk(P, b, h, p):
    """Flat Top-K by leaf LSE from torch.logsumexp / torch.topk on the dense logit matrix."""
    C, K, G = P.C, P.K, P.G
    c = p // C
    if c + 1 <= K:
        return list(range(c + 1))
    qh = torch.from_numpy(P._q_rows(b, h, np.asarray([p]))[0])
    kk = torch.from_numpy(P.unit(b, h)[0][:(c - 1) * C])
    z = (qh @ kk.T) * P.scale
    u = torch.logsumexp(z.reshape(G, c - 1, C), dim=2).sum(dim=0)
    u[0] = -float("inf")
    forced = sorted({0, c - 1, c})
    top = torch.topk(u, K - len(forced)).indices.tolist()
    return sorted(set(forced) | set(top))


def test_c_unpruned_regime_equals_textbook_flat_topk():
    w = S.WORKLOADS["cfg1"]                                       # no pruning above the leaves for p < 512
    P, _ = _cproblem(w)
    ps = list(range(0, 512, 7)) + [255, 256, 257, 319, 320, 511]
    idx, _ = P.route_all(np.asarray([(0, 0, p) for p in ps]))
    for row, p in zip(idx, ps):
        assert [int(x) for x in row if x >= 0] == _textbook_flat_topk(P, 0, 0, p), p
    w2 = S.Workload("t", 1, 1024, 8, 2, 32, 32, 4, 8, "bf16", 11, "iid")     # K >= M_2, GQA 4, fan-in 4
    P2, _ = _cproblem(w2)
    tri = np.asarray([(0, h, p) for h in range(2) for p in range(0, 1024, 13)])
    idx2, _ = P2.route_all(tri)
    for row, (b, h, p) in zip(idx2, tri):
        assert [int(x) for x in row if x >= 0] == _textbook_flat_topk(P2, 0, int(h), int(p)), (h, p)


def test_c_pruned_regime_hand_derived_example():
    a, meta, queries = None, {}, []
    with open(os.path.join(GOLDEN, "pruned_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, rest = line.split(":", 1)
            if key == "a":
                a = [float(x) for x in rest.split()]
            elif key == "query":
                p, rhs = rest.split("->")
                queries.append((int(p), list(map(int, rhs.split("|")[0].split()))))
            else:
                meta[key] = int(rest)
    N, C, g, K = meta["N"], meta["C"], meta["g"], meta["K"]
    k = np.repeat(np.asarray(a), C).reshape(1, N, 1, 1).astype(np.float32)
    q = np.ones((1, N, 1, 1), dtype=np.float32)
    P = OC.CProblem(q, k, k, C=C, g=g, K=K, dtype="fp32", scale=1.0)
    idx, margin = P.route_all(np.asarray([(0, 0, p) for p, _ in queries]))
    for row, m, (p, final) in zip(idx, margin, queries):
        assert [int(x) for x in row if x >= 0] == final, p
        if p == 31:
            m2 = ((1.75 + math.log1p(math.exp(-0.75))) - (2 + math.log1p(math.exp(-8)))) / \
                 (1.75 + math.log1p(math.exp(-0.75)))
            assert abs(m - m2) < 1e-12
        if p == 5:
            assert m == math.inf


def test_c_ties_go_to_smaller_index():
    N, C, g, K, d = 512, 8, 2, 6, 4
    k = np.full((1, N, 1, d), 0.5, dtype=np.float32)
    q = np.full((1, N, 1, d), 0.25, dtype=np.float32)
    P = OC.CProblem(q, k, k, C=C, g=g, K=K, dtype="fp32")
    idx, margin = P.route_all(np.asarray([(0, 0, N - 1)]))
    c = (N - 1) // C
    assert idx[0].tolist() == [0, 1, 2, 3, c - 1, c] and margin[0] == 0.0


DIFF_SHAPES = [
    S.Workload("d_fan4_gqa", 2, 4096, 4, 2, 64, 32, 4, 8, "bf16", 102, "walk"),
    S.Workload("d_ragged_g3", 1, 1000, 2, 1, 32, 24, 3, 5, "fp32", 107, "iid"),
    S.Workload("d_gqa4_ragged", 1, 2048 + 37, 8, 2, 128, 64, 2, 4, "bf16", 101, "iid"),
    S.Workload("d_g16", 1, 3072, 16, 1, 64, 64, 2, 6, "bf16", 104, "iid"),
]


@pytest.mark.parametrize("w", DIFF_SHAPES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", ["lse", "mean", "mean_var"])
def test_c_oracle_agrees_with_numpy_oracle(w, mode):
    """Two independently written restatements of the same definitions (pruned regime, fan-in 3 / 4,
    G > 1, ragged N and ragged levels).  Sets must be equal except where the cut is a near-tie in fp64
    (different summation orders); margins, outputs and denominators to fp64 rounding."""
    if mode != "lse" and w.name not in ("d_fan4_gqa", "d_ragged_g3"):
        pytest.skip("score modes on two shapes")
    Pc, t = _cproblem(w, mode=mode)
    Pn = O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype, mode=mode)
    tri = S.sample_queries(w, 60)
    ic, mc = Pc.route_all(tri)
    inn, mn = Pn.route_all(tri)
    differ = np.any(ic != inn, axis=1)
    assert np.all(mn[differ] < 1e-9), "sets differ away from an fp64 near-tie"
    same = ~differ
    fin = same & np.isfinite(mn)
    assert np.array_equal(np.isinf(mc[same]), np.isinf(mn[same]))
    np.testing.assert_allclose(mc[fin], mn[fin], rtol=0, atol=1e-9)
    for lc, ln in zip(Pc.pyramid()[1:], Pn.pyramid()[1:]):
        assert np.array_equal(lc, ln)
    oc, lc = Pc.attend_raw(tri, inn)
    on = np.empty_like(oc)
    ln = np.empty_like(lc)
    for s, (b, h, p) in enumerate(tri):
        for j in range(Pn.G):
            on[s, j], ln[s, j] = Pn.attend(int(b), int(h) * Pn.G + j, int(p), inn[s])
    np.testing.assert_allclose(oc, on, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lc, ln, rtol=0, atol=1e-11)
    fc, fmc = Pc.flat_mean_all(tri)
    fn, fmn = Pn.flat_mean_all(tri)
    fd = np.any(fc != fn, axis=1)
    assert np.all(fmn[fd] < 1e-9)


# ---------------------------------------------------------------- attention and its backward

def test_c_attention_equals_dense_causal_when_budget_covers_sequence():
    w = S.Workload("dense", 1, 256, 4, 2, 32, 16, 2, 16, "fp32", 31, "iid")
    P, t = _cproblem(w)
    f64 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    q = f64(t["q"]).permute(0, 2, 1, 3)
    k = f64(t["k"]).permute(0, 2, 1, 3).repeat_interleave(P.G, dim=1)
    v = f64(t["v"]).permute(0, 2, 1, 3).repeat_interleave(P.G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True).numpy()
    z = (q @ k.transpose(-1, -2)) / math.sqrt(w.d)
    z = z.masked_fill(torch.triu(torch.ones(w.N, w.N, dtype=torch.bool), 1), -float("inf"))
    ref_lse = torch.logsumexp(z, dim=-1).numpy()
    tri = _all_triples(P)
    idx, _ = P.route_all(tri)
    out, lse = P.attend_raw(tri, idx)
    for s, (b, h, p) in enumerate(tri):
        assert [int(x) for x in idx[s] if x >= 0] == list(range(int(p) // w.C + 1))
        for j in range(P.G):
            np.testing.assert_allclose(out[s, j], ref[0, h * P.G + j, p], rtol=1e-9, atol=1e-12)
            assert abs(lse[s, j] - ref_lse[0, h * P.G + j, p]) < 1e-10


def test_c_backward_rows_match_torch_autograd():
    """dq of every row and dk / dv of a key range against autograd on the masked dense attention built
    from the same index sets."""
    w = S.Workload("bwd", 1, 192, 4, 2, 16, 16, 2, 4, "fp32", 61, "iid")
    P, t = _cproblem(w)
    tri = _all_triples(P)
    idx, _ = P.route_all(tri)
    rng = np.random.default_rng(5)
    dout = rng.standard_normal((w.N, w.Hq, w.d)).astype(np.float32)
    q = torch.tensor(t["q"][0], dtype=torch.float64, requires_grad=True)          # [N, Hq, d]
    k = torch.tensor(t["k"][0], dtype=torch.float64, requires_grad=True)
    v = torch.tensor(t["v"][0], dtype=torch.float64, requires_grad=True)
    loss = 0.0
    for s, (b, h, p) in enumerate(tri):
        blocks = [int(x) for x in idx[s] if x >= 0]
        toks = [j for i in blocks for j in range(i * w.C, min((i + 1) * w.C, w.N)) if j <= p]
        for j in range(P.G):
            hq = h * P.G + j
            z = (k[toks, h] @ q[p, hq]) / math.sqrt(w.d)
            o = torch.softmax(z, 0) @ v[toks, h]
            loss = loss + (o * torch.from_numpy(dout[p, hq].astype(np.float64))).sum()
    loss.backward()
    for h in range(w.Hkv):
        rows = np.nonzero(tri[:, 1] == h)[0]
        do_rows = np.stack([dout[int(p), h * P.G:(h + 1) * P.G] for p in tri[rows, 2]])
        dq, dk, dv = P.backward_rows(tri[rows], idx[rows], do_rows, key_range=(32, 96))
        ref_dq = np.stack([q.grad[int(p), h * P.G:(h + 1) * P.G].numpy() for p in tri[rows, 2]])
        np.testing.assert_allclose(dq, ref_dq, rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dk, k.grad[32:96, h].numpy(), rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dv, v.grad[32:96, h].numpy(), rtol=1e-9, atol=1e-12)


def test_numpy_backward_dq_rows_helper_matches_full_backward():
    """attend_backward_dq_rows (the helper full-size tests use for sampled rows) against the pinned
    attend_backward on the same problem."""
    w = S.Workload("bwd2", 2, 160, 4, 2, 16, 16, 2, 4, "bf16", 62, "iid")
    t = S.make_inputs(w)
    Pn = O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype)
    tri = Pn.all_triples()
    idx_rows, _ = Pn.route_all(tri)
    idx = idx_rows.reshape(w.B, w.Hkv, w.N, w.K)
    dout = S.f32_to_bf16_bits(np.random.default_rng(9).standard_normal((w.B, w.N, w.Hq, w.d)).astype(np.float32))
    dq, _, _ = O.attend_backward(t["q"], t["k"], t["v"], idx, dout, C=w.C, dtype=w.dtype)
    pick = np.random.default_rng(3).choice(len(tri), 64, replace=False)
    do_rows = np.stack([dout[b, p, h * Pn.G:(h + 1) * Pn.G] for b, h, p in tri[pick]])
    got = O.attend_backward_dq_rows(Pn, tri[pick], idx_rows[pick], do_rows)
    ref = np.stack([dq[b, p, h * Pn.G:(h + 1) * Pn.G] for b, h, p in tri[pick]])
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)
