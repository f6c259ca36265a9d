"""Causality pin of both oracles: the rows of a sequence do not depend on anything after them.  Every
scored node lies wholly in the query's past and the nodes on its own path are forced, never scored
(Sec. 3.2), so running a sequence as the head of a longer one -- zero-filled or followed by other
tokens -- must give the same index sets and the same attention outputs, bit for bit.  A selector that
looked at a partial node's summary, or a hierarchy walk that depended on the number of levels, fails this."""
import numpy as np
import pytest

import pisa_synth as S
from oracle import pisa_oracle as O
from oracle import pisa_oracle_c as OC

CASES = [  # N, N_long, C, g, K, Hq, Hkv, d
    (700, 2048, 16, 2, 8, 4, 2, 32),
    (333, 1024, 8, 2, 6, 2, 1, 32),
    (1000, 1536, 16, 4, 8, 4, 2, 32),
    (97, 4096, 8, 2, 5, 2, 2, 32),
    (64, 65, 8, 3, 4, 2, 1, 32),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("tail", ["zeros", "tokens"])
@pytest.mark.parametrize("which", ["numpy", "c"])
def test_rows_of_a_prefix_do_not_depend_on_what_follows(case, tail, which):
    N, NL, C, g, K, Hq, Hkv, d = case
    long = S.make_inputs(S.Workload("prefix", 1, NL, Hq, Hkv, d, C, g, K, "bf16", 31, "iid"))
    short = {key: np.ascontiguousarray(long[key][:, :N]) for key in ("q", "k", "v")}
    if tail == "zeros":
        long = {key: long[key].copy() for key in ("q", "k", "v")}
        for key in ("q", "k", "v"):
            long[key][:, N:] = 0
    make = (lambda t: O.Problem(t["q"], t["k"], t["v"], C=C, g=g, K=K, dtype="bf16", mode="lse")) if which == "numpy" \
        else (lambda t: OC.CProblem(t["q"], t["k"], t["v"], C=C, g=g, K=K, dtype="bf16", mode="lse"))
    a, b = make(short), make(long)
    rng = np.random.default_rng(5)
    ps = np.unique(np.concatenate([[0, N - 1, (N - 1) // C * C], rng.integers(0, N, size=40 if which == "numpy" else 200)]))
    tri = np.array([(0, h, p) for h in range(Hkv) for p in ps], dtype=np.int64)
    ia, _ = a.route_all(tri)
    ib, _ = b.route_all(tri)
    assert np.array_equal(ia, ib)
    oa, la = a.attend_all(tri, ia)
    ob, lb = b.attend_all(tri, ib)
    assert np.array_equal(np.asarray(oa), np.asarray(ob)) and np.array_equal(np.asarray(la), np.asarray(lb))
