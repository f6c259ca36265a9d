"""Exact ties.  Keys that repeat with a period of a few blocks give whole families of nodes with
bit-identical summaries and hence bit-identical scores at every level, on both sides; Select_K must
then break the ties towards the smaller block index (Algorithm 1).  The cut of such a row sits on a tie,
so its oracle margin is 0 and the usual tie band would excuse any answer: here every sampled row must
match exactly instead (distinct families have generic gaps, far outside rounding)."""
import numpy as np
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

CASES = {
    # name: (workload, period in blocks)
    "gqa4_k8_period4": (S.Workload("ties_gqa4", 1, 64 * 48, 8, 2, 64, 64, 2, 8, "bf16", 801, "iid"), 4),
    "gqa4_k32_period2": (S.Workload("ties_k32", 1, 128 * 160, 4, 1, 128, 128, 2, 32, "bf16", 802, "iid"), 2),
    "fan4_k6_period3": (S.Workload("ties_fan4", 2, 32 * 100, 4, 2, 64, 32, 4, 6, "bf16", 803, "iid"), 3),
}


@pytest.mark.parametrize("impl", [PB.IMPL_SIMT, PB.IMPL_AUTO])
@pytest.mark.parametrize("name", list(CASES))
def test_ties_go_to_the_smaller_block_index(name, impl):
    w, period = CASES[name]
    t = S.make_inputs(w)
    span = period * w.C
    k = t["k"].copy()
    k[:, span:] = np.tile(k[:, :span], (1, (w.N + span - 1) // span, 1, 1))[:, :w.N - span]
    t = dict(t, k=k)
    prob = T.oracle_problem(w, t)
    tri = S.sample_queries(w, 200)
    dev = T.Device(w, t, impl=impl)
    dev.forward()
    assert dev.sync_status() == 0
    got = T.gather_idx(dev.idx, tri)
    T.check_index_rows_valid(got, tri, w)
    ref_idx, ref_margin = prob.route_all(tri)
    n_tied = int((ref_margin <= T.TIE_BAND).sum())
    differ = np.any(got != ref_idx, axis=1)
    print(f"[{name}] rows={len(tri)} rows whose cut sits on a tie={n_tied} differ={int(differ.sum())}")
    assert n_tied > len(tri) // 4, "the construction should put most cuts on ties"
    assert not differ.any(), (tri[differ][:5], got[differ][:5], ref_idx[differ][:5])
