"""Pins for the CPU oracle: each check anchors it to something other than itself
(closed forms, textbook/library routines, a hand-derived example, invariants)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import pisa_oracle as O
import pisa_synth as S

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- storage rounding

def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9])])
    ours = O.f64_to_bf16_bits(x)
    # fp64 -> bf16 directly in torch (single rounding)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    # halfway cases between two bf16 neighbours that fp32 cannot see without a sticky bit
    base = 1.0
    ulp = 2.0 ** -7
    tricky = np.array([base + ulp / 2 + 2.0 ** -40, base + ulp / 2 - 2.0 ** -40, base + ulp / 2,
                       base + 3 * ulp / 2])
    got = O.bf16_bits_to_f64(O.f64_to_bf16_bits(tricky))
    assert got.tolist() == [base + ulp, base, base, base + 2 * ulp]
    # the generator's fp32->bf16 agrees with torch too
    xf = x.astype(np.float32)
    ref32 = torch.from_numpy(xf).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(S.f32_to_bf16_bits(xf), ref32)


# ---------------------------------------------------------------- hierarchy / pyramid

def test_hierarchy_counts():
    assert O.hierarchy(1024, 64, 2) == [1024, 16, 8, 4, 2, 1]
    assert O.hierarchy(32768, 64, 4) == [32768, 512, 128, 32, 8, 2, 1]
    assert O.hierarchy(131072, 128, 2)[1:] == [1024 >> i for i in range(11)]
    assert O.hierarchy(1000, 64, 2) == [1000, 16, 8, 4, 2, 1]      # ragged last leaf
    assert O.hierarchy(5 * 8, 8, 2) == [40, 5, 3, 2, 1]
    assert list(O.children(1, 15, O.hierarchy(1000, 64, 2), 64, 2)) == list(range(960, 1000))
    assert list(O.children(2, 2, [40, 5, 3, 2, 1], 8, 2)) == [4]


def test_pyramid_equal_children_is_mean_of_raw_keys():
    # Sec. 3.2: with equally sized children every summary equals the mean of all raw keys it spans
    rng = np.random.default_rng(1)
    B, N, H, d, C, g = 2, 512, 3, 8, 16, 2
    k = rng.standard_normal((B, N, H, d))
    lv = O.build_pyramid(k, C, g, "fp32")
    M = O.hierarchy(N, C, g)
    for l in range(1, len(M)):
        span = C * g ** (l - 1)
        ref = k.reshape(B, M[l], span, H, d).mean(axis=2).transpose(0, 2, 1, 3)
        assert lv[l].shape == (B, H, M[l], d)
        np.testing.assert_allclose(lv[l], ref, rtol=0, atol=3e-7 * l)


def test_pyramid_constant_and_ramp():
    B, N, H, d, C, g = 1, 256, 1, 4, 8, 4
    k = np.full((B, N, H, d), 0.375)
    for l, a in enumerate(O.build_pyramid(k, C, g, "bf16")):
        if l:
            assert np.all(a == 0.375)
    ramp = np.arange(N, dtype=np.float64)[None, :, None, None] * np.ones((B, N, H, d))
    lv = O.build_pyramid(ramp, C, g, "fp32")
    M = O.hierarchy(N, C, g)
    for l in range(1, len(M)):
        span = C * g ** (l - 1)
        lo = np.arange(M[l]) * span
        mid = (lo + np.minimum(lo + span, N) - 1) / 2.0    # equal-sized children at every step here
        np.testing.assert_allclose(lv[l][0, 0, :, 0], mid, rtol=1e-6)


def test_pyramid_ragged_is_mean_of_means():
    # N = 40, C = 8: 5 leaves; g = 2: level 2 = [m(0,1), m(2,3), s4], level 3 = [m(l2_0,l2_1), l2_2]
    rng = np.random.default_rng(2)
    k = rng.standard_normal((1, 37, 1, 3))          # last leaf short (5 keys)
    lv = O.build_pyramid(k, 8, 2, "fp32")
    kk = k[0, :, 0, :]
    s = [kk[i * 8:min(i * 8 + 8, 37)].mean(axis=0) for i in range(5)]
    f32 = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    s = [f32(x) for x in s]
    np.testing.assert_array_equal(lv[1][0, 0], np.stack(s))
    l2 = [f32((s[0] + s[1]) / 2), f32((s[2] + s[3]) / 2), s[4]]
    np.testing.assert_array_equal(lv[2][0, 0], np.stack(l2))
    l3 = [f32((l2[0] + l2[1]) / 2), l2[2]]
    np.testing.assert_array_equal(lv[3][0, 0], np.stack(l3))
    l4 = [f32((l3[0] + l3[1]) / 2)]
    np.testing.assert_array_equal(lv[4][0, 0], np.stack(l4))
    # the top is NOT the token mean when children are unequal (mean of means)
    assert not np.allclose(l4[0], kk.mean(axis=0), atol=1e-3)


def test_pyramid_levels_pool_the_stored_level_below():
    rng = np.random.default_rng(3)
    k = O.round_to_storage(rng.standard_normal((1, 64, 1, 16)), "bf16")
    lv = O.build_pyramid(k, 4, 2, "bf16")
    for l in range(2, len(lv)):
        pooled = lv[l - 1][0, 0].reshape(-1, 2, 16).mean(axis=1)
        ref = torch.from_numpy(pooled).to(torch.bfloat16).to(torch.float64).numpy()
        np.testing.assert_array_equal(lv[l][0, 0], ref)


# ---------------------------------------------------------------- scores

def test_leaf_score_identical_keys_closed_form():
    rng = np.random.default_rng(4)
    d, C, G = 16, 64, 4
    q = rng.standard_normal((G, d))
    kv = rng.standard_normal(d)
    x = np.tile(kv, (C, 1))
    scale = 1 / math.sqrt(d)
    expect = sum(math.log(C) + float(q[h] @ kv) * scale for h in range(G))
    assert abs(O.lse_score(q, x, scale) - expect) < 1e-12


def test_leaf_lse_ranks_like_dense_softmax_block_mass():
    # App. A: exp(raw-key LSE) is proportional to the block's full-attention mass (one head)
    rng = np.random.default_rng(5)
    N, d, C = 512, 8, 32
    q = rng.standard_normal((1, d)) * 2
    k = rng.standard_normal((N, d))
    scale = 1 / math.sqrt(d)
    probs = torch.softmax(torch.from_numpy((k @ q[0]) * scale), dim=0).numpy()
    mass = probs.reshape(N // C, C).sum(axis=1)
    lse = np.array([O.lse_score(q, k[i * C:(i + 1) * C], scale) for i in range(N // C)])
    assert np.array_equal(np.argsort(-mass, kind="stable"), np.argsort(-lse, kind="stable"))
    np.testing.assert_allclose(np.exp(lse - lse.max()) / np.exp(lse - lse.max()).sum(), mass, rtol=1e-10)


def test_intermediate_score_jensen_sandwich():
    # App. A.1: mean_j m_j <= log(1/g sum e^{m_j}) <= log(1/|B| sum e^{z_t}); equality on the
    # right when logits inside each child are equal
    rng = np.random.default_rng(6)
    d, C, g = 8, 16, 2
    q = rng.standard_normal((1, d)) * 1.5
    for trial in range(20):
        k = rng.standard_normal((1, g * C, 1, d))
        lv = O.build_pyramid(k, C, g, "fp32")
        child = lv[1][0, 0]                           # g leaf summaries
        s_mid = O.lse_score(q, child, 1.0) - math.log(g)
        z = k[0, :, 0, :] @ q[0]
        m = z.reshape(g, C).mean(axis=1)
        left = m.mean()
        right = float(torch.logsumexp(torch.from_numpy(z), 0)) - math.log(g * C)
        assert left <= s_mid + 1e-6 and s_mid <= right + 1e-6
        # PISA-1 is the left term
        assert abs(O.lse_score(q, child, 1.0, "mean") - left) < 1e-5
    k = np.repeat(rng.standard_normal((1, g, 1, d)), C, axis=1)   # equal logits inside each child
    lv = O.build_pyramid(k, C, g, "fp32")
    z = k[0, :, 0, :] @ q[0]
    right = float(torch.logsumexp(torch.from_numpy(z), 0)) - math.log(g * C)
    assert abs(O.lse_score(q, lv[1][0, 0], 1.0) - math.log(g) - right) < 1e-5


def test_score_taylor_identity():
    # Sec. 4.3: LSE = log m + mean + Var/2 + h.o.t.; PISA-1/2 truncate it
    rng = np.random.default_rng(7)
    m = 64
    z0 = rng.standard_normal(m)
    for eps in (1e-1, 1e-2, 1e-3):
        z = (eps * z0)[None, :]
        lse = float(O.block_score(z, "lse")[0])
        s1 = float(O.block_score(z, "mean")[0])
        s2 = float(O.block_score(z, "mean_var")[0])
        assert abs(s1 - z.mean()) < 1e-15
        assert abs(s2 - (z.mean() + 0.5 * z.var())) < 1e-15
        assert abs(lse - math.log(m) - s2) < 2.0 * eps ** 3          # third-order remainder
        assert abs(lse - math.log(m) - s1) < 2.0 * eps ** 2


# ---------------------------------------------------------------- routing

def _problem(w, B=None):
    t = S.make_inputs(w, B=B)
    return O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype), t


def _textbook_flat_topk(P, b, h, p):
    """Flat Top-K by leaf LSE from torch.logsumexp / torch.topk on the dense logit matrix."""
    C, K, G = P.C, P.K, P.G
    c = p // C
    if c + 1 <= K:
        return list(range(c + 1))
    qh = torch.from_numpy(P.q_group(b, h, p))                         # [G, d]
    kk = torch.from_numpy(P.head(b, h)[0][:(c - 1) * C])              # leaves 0..c-2, all in the past
    z = (qh @ kk.T) * P.scale                                         # [G, (c-1)C]
    u = torch.logsumexp(z.reshape(G, c - 1, C), dim=2).sum(dim=0)     # [c-1]
    u[0] = -float("inf")                                              # leaf 0 is forced
    forced = sorted({0, c - 1, c})
    top = torch.topk(u, K - len(forced)).indices.tolist()
    return sorted(set(forced) | set(top))


def test_unpruned_regime_equals_textbook_flat_topk_tiny():
    # cfg1: no pruning above the leaves while floor(c/g)+1 <= K, i.e. p < 512
    w = S.WORKLOADS["cfg1"]
    P, _ = _problem(w)
    for p in list(range(0, 512, 7)) + [255, 256, 257, 319, 320, 511]:
        I, _ = P.route(0, 0, p)
        assert I == _textbook_flat_topk(P, 0, 0, p), p
        assert I == P.flat_lse(0, 0, p)


def test_unpruned_regime_whole_sequence_gqa():
    # K >= M_2: only the leaf level prunes, for every query; GQA group of 4, bf16, g = 4
    w = S.Workload("t", 1, 1024, 8, 2, 32, 32, 4, 8, "bf16", 11, "iid")
    P, _ = _problem(w)
    assert P.M[2] <= w.K
    for h in range(2):
        for p in range(0, 1024, 13):
            I, _ = P.route(0, h, p)
            assert I == _textbook_flat_topk(P, 0, h, p), (h, p)


def _read_golden():
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
                final, l2, flat = (list(map(int, part.split(":")[-1].split())) for part in rhs.split("|"))
                queries.append((int(p), final, l2, flat))
            else:
                meta[key] = int(rest)
    return a, meta, queries


def test_pruned_regime_hand_derived_example():
    a, meta, queries = _read_golden()
    N, C, g, K = meta["N"], meta["C"], meta["g"], meta["K"]
    k = np.repeat(np.asarray(a), C).reshape(1, N, 1, 1)
    q = np.ones((1, N, 1, 1))
    P = O.Problem(q.astype(np.float32), k.astype(np.float32), k.astype(np.float32),
                  C=C, g=g, K=K, dtype="fp32", scale=1.0)
    for p, final, l2, flat in queries:
        tr = []
        I, margin = P.route(0, 0, p, trace=tr)
        assert I == final, (p, I)
        assert [t for t in tr if t["level"] == 2][0]["I"] == l2
        assert P.flat_lse(0, 0, p) == flat
        if p == 31:
            m2 = ((1.75 + math.log1p(math.exp(-0.75))) - (2 + math.log1p(math.exp(-8)))) / \
                 (1.75 + math.log1p(math.exp(-0.75)))
            m1 = (1.75 - 1.5) / (1.75 + math.log(2))
            assert m2 < m1 and abs(margin - m2) < 1e-12
        if p == 5:
            assert margin == math.inf


def test_ties_go_to_smaller_index():
    # all keys equal -> all scores tie at every level -> forced plus the smallest indices
    N, C, g, K, d = 512, 8, 2, 6, 4
    k = np.full((1, N, 1, d), 0.5, dtype=np.float32)
    q = np.full((1, N, 1, d), 0.25, dtype=np.float32)
    P = O.Problem(q, k, k, C=C, g=g, K=K, dtype="fp32")
    I, margin = P.route(0, 0, N - 1)
    c = (N - 1) // C
    assert I == [0, 1, 2, 3, c - 1, c]
    assert margin == 0.0


def _check_invariants(P, b, h, p):
    tr = []
    I, margin = P.route(b, h, p, trace=tr)
    C, g, K = P.C, P.g, P.K
    c = p // C
    assert len(I) == min(K, c + 1) and len(set(I)) == len(I) and I == sorted(I)
    assert all(0 <= i <= c for i in I)
    assert {0, c, max(c - 1, 0)} <= set(I)
    prev = None
    for t in tr:                                  # levels L .. 1
        l = t["level"]
        assert len(t["I"]) <= K and len(t["A"]) <= max(g * K, 1)
        assert set(t["F"]) <= set(t["I"]) <= set(t["V"]) <= set(t["A"])
        assert all(i * g ** (l - 1) <= c for i in t["V"])          # never starts after the query's leaf
        if prev is not None:
            assert all(i // g in prev for i in t["I"])             # parent-chain containment
        prev = set(t["I"])
        if not t["scored"]:
            assert t["I"] == t["V"]
    return I, margin


@pytest.mark.parametrize("name,B", [("cfg1", None), ("cfg2", None), ("cfg3", 1)])
def test_invariants_on_baseline_workloads(name, B):
    w = S.WORKLOADS[name]
    if name == "cfg3":      # same recipe, shorter sequence to keep the CPU suite quick
        w = S.Workload("cfg3s", 1, 8192, 8, 2, 128, 64, 4, 16, "bf16", 2, "walk")
    if name == "cfg2":
        w = S.Workload("cfg2s", 1, 8192, 2, 2, 128, 64, 2, 16, "bf16", 1, "needle1", q_scale=w.q_scale)
    P, t = _problem(w, B)
    tri = S.sample_queries(w, 40, B=B)
    for b, h, p in tri:
        _check_invariants(P, int(b), int(h), int(p))
    # planted needle blocks must be found by their target queries (pruned regime, dominant block)
    for b in range(t["needles"].shape[0]):
        for h in range(t["needles"].shape[1]):
            for blk, t_star in t["needles"][b, h]:
                I, _ = P.route(b, h, int(t_star))
                assert int(blk) in I


def test_ragged_shapes_route_and_attend():
    # N % C != 0 and M_l % g != 0
    w = S.Workload("rag", 1, 1000, 2, 1, 16, 24, 3, 4, "fp32", 21, "iid")
    P, _ = _problem(w)
    assert P.M == [1000, 42, 14, 5, 2, 1]
    for p in (0, 23, 24, 500, 983, 984, 999):
        I, _ = _check_invariants(P, 0, 0, p)
        out, lse = P.attend(0, 1, p, I)
        assert np.isfinite(out).all() and np.isfinite(lse)


# ---------------------------------------------------------------- attention

def test_attention_equals_dense_causal_when_budget_covers_sequence():
    w = S.Workload("dense", 1, 256, 4, 2, 32, 16, 2, 16, "fp32", 31, "iid")
    P, t = _problem(w)
    assert w.K * w.C >= w.N
    f64 = lambda a: torch.from_numpy(O.load_storage(a, w.dtype))
    q = f64(t["q"]).permute(0, 2, 1, 3)                               # [B, Hq, N, d]
    k = f64(t["k"]).permute(0, 2, 1, 3).repeat_interleave(P.G, dim=1)
    v = f64(t["v"]).permute(0, 2, 1, 3).repeat_interleave(P.G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True).numpy()
    z = (q @ k.transpose(-1, -2)) / math.sqrt(w.d)
    z = z.masked_fill(torch.triu(torch.ones(w.N, w.N, dtype=torch.bool), 1), -float("inf"))
    ref_lse = torch.logsumexp(z, dim=-1).numpy()
    for p in range(0, w.N, 5):
        for h in range(w.Hkv):
            I, _ = P.route(0, h, p)
            assert I == list(range(p // w.C + 1))
            for j in range(P.G):
                out, lse = P.attend(0, h * P.G + j, p, I)
                np.testing.assert_allclose(out, ref[0, h * P.G + j, p], rtol=1e-9, atol=1e-12)
                assert abs(lse - ref_lse[0, h * P.G + j, p]) < 1e-10


def test_attention_block_decomposition():
    # LSE_out = logsumexp of per-block LSEs; output is the LSE-weighted mix of per-block outputs;
    # one selected block = softmax inside the block; rows are convex combinations of V rows
    w = S.Workload("dec", 1, 512, 1, 1, 16, 32, 2, 4, "fp32", 41, "iid")
    P, _ = _problem(w)
    p = 500
    I = [0, 3, 14, 15]
    out, lse = P.attend(0, 0, p, I)
    parts = [P.attend(0, 0, p, [i]) for i in I]
    lses = torch.tensor([l for _, l in parts], dtype=torch.float64)
    assert abs(lse - float(torch.logsumexp(lses, 0))) < 1e-12
    wts = torch.softmax(lses, 0).numpy()
    np.testing.assert_allclose(out, sum(wi * o for wi, (o, _) in zip(wts, parts)), atol=1e-12)
    kk, vv, _ = P.head(0, 0)
    qv = P.q_group(0, 0, p)[0]
    z = torch.from_numpy(kk[96:128] @ qv) * P.scale
    ref = (torch.softmax(z, 0)[:, None] * torch.from_numpy(vv[96:128])).sum(0).numpy()
    np.testing.assert_allclose(parts[1][0], ref, atol=1e-12)
    # causal mask inside the current block: only tokens <= p
    zc = torch.from_numpy(kk[480:p + 1] @ qv) * P.scale
    assert abs(parts[3][1] - float(torch.logsumexp(zc, 0))) < 1e-12
    vmin, vmax = vv.min(axis=0), vv.max(axis=0)
    assert np.all(out >= vmin) and np.all(out <= vmax)


# ---------------------------------------------------------------- flat mean-BSA

def test_flat_mean_bsa_matches_definition_and_g1_normalisation_invariance():
    w = S.Workload("flat", 1, 2048, 4, 2, 32, 32, 2, 8, "bf16", 51, "iid")
    P, _ = _problem(w)
    for p in (100, 700, 2047):
        for h in range(2):
            I, _ = P.flat_mean(0, h, p)
            c = p // w.C
            if c + 1 <= w.K:
                assert I == list(range(c + 1))
                continue
            qh = torch.from_numpy(P.q_group(0, h, p))
            s = (qh @ torch.from_numpy(P.head(0, h)[2][1][:c + 1]).T) * P.scale
            u = torch.softmax(s, dim=1).sum(0)
            forced = sorted({0, c - 1, c})
            u[forced] = -1.0
            top = torch.topk(u, w.K - len(forced)).indices.tolist()
            assert I == sorted(set(forced) | set(top))
    # one head per group: the per-head softmax is monotone, so the set equals top-K of the raw scores
    w1 = S.Workload("flat1", 1, 2048, 2, 2, 32, 32, 2, 8, "bf16", 52, "iid")
    P1, _ = _problem(w1)
    p = 2000
    c = p // 32
    I, _ = P1.flat_mean(0, 1, p)
    s = (P1.head(0, 1)[2][1][:c + 1] @ P1.q_group(0, 1, p)[0]) * P1.scale
    s[[0, c - 1, c]] = -np.inf
    top = np.argsort(-s, kind="stable")[:8 - 3].tolist()
    assert I == sorted({0, c - 1, c} | set(top))
