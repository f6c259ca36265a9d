"""Host-side logic of the parity helpers: the tie-band admissibility walk and the output tolerances."""
import numpy as np
import pytest

import pisa_synth as S
from oracle import pisa_oracle as O

import pisa_testlib as T


def _prob(w):
    t = S.make_inputs(w)
    return O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype), t


def test_admissible_walk_accepts_the_oracle_and_rejects_everything_else_without_ties():
    w = S.Workload("adm", 1, 2048, 4, 2, 32, 32, 2, 6, "bf16", 71, "iid")
    P, _ = _prob(w)
    rng = np.random.default_rng(0)
    for p in (2047, 1500, 900, 700):
        tr = []
        I, margin = P.route(0, 1, p, trace=tr)
        assert T.admissible_under_band(P, 0, 1, p, I)
        if margin > 10 * T.TIE_BAND:          # no near-tie anywhere: the oracle's set is the only admissible one
            c = p // w.C
            others = [i for i in range(1, c - 1) if i not in I]
            for _ in range(5):
                J = sorted(set(I) - {I[2]} | {int(rng.choice(others))})
                assert not T.admissible_under_band(P, 0, 1, p, J), (p, I, J)


def test_admissible_walk_follows_a_near_tie_and_its_consequences():
    # d = 1, scale 1, q = 1, C = 2, g = 2, K = 4: scores follow from the per-leaf key values a_i
    # (a leaf scores a_i + log 2, a level-2 node log(e^a + e^a')).  Nodes 1 and 2 of level 2 tie within
    # 1e-5; whichever is kept decides which leaves can follow.
    a = [0.0, 0.0, 1.0, 1.0, 1.00001, 1.00001, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, 0.0, 0.0,
         -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, -3.0, 0.0, 0.0]
    N, C = 64, 2
    k = np.repeat(np.asarray(a), C).reshape(1, N, 1, 1).astype(np.float32)
    q = np.ones((1, N, 1, 1), dtype=np.float32)
    P = O.Problem(q, k, k, C=C, g=2, K=4, dtype="fp32", scale=1.0)
    p = N - 1                                      # current leaf 31: forced leaves 0, 30, 31; one free slot
    I, margin = P.route(0, 0, p)
    assert I == [0, 4, 30, 31] and margin < T.TIE_BAND        # leaf 4 (a = 1.00001) wins by 1e-5
    assert T.admissible_under_band(P, 0, 0, p, [0, 4, 30, 31])
    assert T.admissible_under_band(P, 0, 0, p, [0, 5, 30, 31])   # its equal sibling: a tie at the leaf level
    assert T.admissible_under_band(P, 0, 0, p, [0, 2, 30, 31])   # the other side of the level-2 near-tie
    assert not T.admissible_under_band(P, 0, 0, p, [0, 1, 30, 31])   # a = 0: far from any cut
    assert not T.admissible_under_band(P, 0, 0, p, [0, 14, 30, 31])
    # and compare_index_sets uses it
    ref = O.pad_indices(I, 4)[None]
    tri = np.asarray([[0, 0, p]])
    for got, bad in (([0, 2, 30, 31], 0), ([0, 14, 30, 31], 1)):
        n_diff, n_bad, n_band = T.compare_index_sets(np.asarray([got], dtype=np.int32), ref, np.asarray([margin]),
                                                     prob=P, triples=tri)
        assert (n_diff, n_bad, n_band) == (1, bad, 1)


def test_output_bounds_are_the_flat_ones_for_outputs_of_order_one():
    ref = np.linspace(-2.0, 2.0, 4096).reshape(32, 1, 128)
    lse = np.zeros((32, 1))
    one = ref.copy()
    one[3, 0, 5] += 0.018
    T.check_outputs(one + 0.0015, lse, ref, lse, "bf16")
    bad = ref.copy()
    bad[3, 0, 5] += 0.021
    with pytest.raises(AssertionError):
        T.check_outputs(bad, lse, ref, lse, "bf16")
    with pytest.raises(AssertionError):
        T.check_outputs(ref + 0.0021, lse, ref, lse, "bf16")       # mean-abs 2e-3
    big = ref * 10.0                                                # reaches 20: one ulp there is 0.125
    rep = {}
    T.check_outputs(big + np.where(np.abs(big) > 19.5, 0.1, 0.0), lse, big, lse, "bf16", rep)
    assert rep["over_strict"] > 0
    with pytest.raises(AssertionError):
        T.check_outputs(big + 0.5, lse, big, lse, "bf16")
