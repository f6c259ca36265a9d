"""Pins for the oracle's decoding functions (Sec. 3.3 "Decoding", App. B "Decode cache").

None of them re-evaluates the decode function's own formula: they check what the definitions imply
(the step at position p must select what the prefill of a longer sequence selects for row p, because
every scored node lies strictly in the past of the query; completed nodes of the cached pyramid equal
those of the longer sequence's pyramid) and special cases that reduce to library routines."""
import math

import numpy as np
import torch

import pisa_synth as S
from oracle import pisa_oracle as O


def _w(name, N, Hq, Hkv, d, C, g, K, dtype, seed, structure="iid"):
    return S.Workload(name, 1, N, Hq, Hkv, d, C, g, K, dtype, seed, structure)


CASES = [
    _w("dec_a", 700, 4, 2, 32, 16, 2, 4, "bf16", 301),
    _w("dec_b", 530, 2, 1, 32, 8, 3, 5, "fp32", 302, "walk"),
    _w("dec_c", 1024, 8, 2, 64, 32, 4, 3, "bf16", 303),
]


def test_decode_step_selects_what_the_prefill_of_a_longer_sequence_selects():
    for w in CASES:
        t = S.make_inputs(w)
        full = O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype)
        rng = np.random.default_rng(w.seed)
        positions = sorted(set([0, 1, w.C - 1, w.C, w.K * w.C, w.K * w.C + 1, w.N - 1] +
                               rng.integers(0, w.N, size=12).tolist()))
        for p in positions:
            idx, margin, out, lse = O.decode_step(t["q"][:, p], t["k"], t["v"], p, C=w.C, g=w.g, K=w.K,
                                                  dtype=w.dtype)
            for h in range(w.Hkv):
                I, m = full.route(0, h, p)
                assert list(idx[0, h][idx[0, h] >= 0]) == list(I), (w.name, p, h)
                assert math.isclose(margin[0, h], m, rel_tol=1e-9, abs_tol=1e-12) or (np.isinf(m) and np.isinf(margin[0, h]))
                for hq in range(h * w.G, (h + 1) * w.G):
                    o, l = full.attend(0, hq, p, I)
                    assert np.allclose(out[0, hq], O.round_to_storage(o, w.dtype), rtol=0, atol=0)
                    assert math.isclose(lse[0, hq], l, rel_tol=1e-12)


def test_decode_step_is_dense_causal_attention_when_the_budget_covers_the_past():
    w = _w("dec_dense", 96, 4, 2, 32, 16, 2, 8, "fp32", 304)        # K*C = 128 > N
    t = S.make_inputs(w)
    q = torch.from_numpy(t["q"]).double().permute(0, 2, 1, 3)           # [B,Hq,N,d]
    k = torch.from_numpy(t["k"]).double().permute(0, 2, 1, 3).repeat_interleave(w.G, dim=1)
    v = torch.from_numpy(t["v"]).double().permute(0, 2, 1, 3).repeat_interleave(w.G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)   # [B,Hq,N,d]
    for p in (0, 15, 16, 50, 95):
        idx, _, out, lse = O.decode_step(t["q"][:, p], t["k"], t["v"], p, C=w.C, g=w.g, K=w.K, dtype=w.dtype)
        assert list(idx[0, 0][idx[0, 0] >= 0]) == list(range(p // w.C + 1))
        assert np.allclose(out[0], ref[0, :, p].numpy(), atol=2e-7)
        z = (q[0, :, p, None, :] * k[0, :, :p + 1]).sum(-1) / math.sqrt(w.d)
        assert np.allclose(lse[0], torch.logsumexp(z, dim=-1).numpy(), atol=1e-10)


def test_cached_pyramid_completed_nodes_match_the_longer_sequence():
    for w in CASES:
        t = S.make_inputs(w)
        full = O.build_pyramid(O.load_storage(t["k"], w.dtype), w.C, w.g, w.dtype)
        for p in (0, w.C - 1, w.C, 3 * w.C + 1, w.N // 2, w.N - 1):
            part = O.decode_pyramid(t["k"], p, w.C, w.g, w.dtype)
            c = p // w.C
            span = 1
            for l in range(1, len(part)):
                n_complete = (p + 1) // (w.C * span)         # nodes all of whose keys have been seen
                assert part[l].shape[2] == -(-(c + 1) // span)
                assert np.array_equal(part[l][:, :, :n_complete], full[l][:, :, :n_complete]), (w.name, p, l)
                span *= w.g


def test_current_leaf_summary_is_the_mean_of_the_keys_seen_so_far():
    w = CASES[1]                                                         # fp32: the mean in closed form
    t = S.make_inputs(w)
    k = t["k"].astype(np.float64)
    for p in (0, 5, w.C + 2, 4 * w.C - 1):
        part = O.decode_pyramid(t["k"], p, w.C, w.g, w.dtype)
        c = p // w.C
        want = k[0, c * w.C:p + 1, 0].mean(axis=0)
        assert np.allclose(part[1][0, 0, c], want.astype(np.float32).astype(np.float64), rtol=0, atol=1e-7)
