"""Seeded random shapes through pisa_forward against the oracle: tiny and ragged sequence lengths, every
supported group size, both leaf sizes and fan-ins of the tensor-core path."""
import os

import numpy as np
import pytest

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402


def _draw(rng, i):
    C = int(rng.choice([64, 128]))
    g = 2 if C == 128 else int(rng.choice([2, 4]))
    K = int(rng.integers(3, min(16, 128 // g) + 1))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2]))
    N = int(rng.choice([1, 2, C - 1, C, C + 1, int(rng.integers(2, 3000)), int(rng.integers(2, 3000))]))
    return S.Workload(f"fuzz{i}", int(rng.choice([1, 2])), N, G * Hkv, Hkv, int(rng.choice([64, 128])), C, g, K,
                      "bf16", 900 + i, str(rng.choice(["iid", "walk"])))


@pytest.mark.parametrize("i", range(16))
def test_random_shape_matches_oracle(i):
    w = _draw(np.random.default_rng(4242 + i), i)
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    dev.forward()
    assert dev.sync_status() == 0, w
    tri = S.sample_queries(w, 30)
    prob = T.oracle_problem(w, t)
    T.check_forward_dev(dev, prob, tri)


def _draw_wide(rng, i):
    C = int(rng.choice([64, 128]))
    g = 2 if C == 128 else int(rng.choice([2, 4]))
    K = int(rng.integers(3, min(32, 128 // g) + 1))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    Hkv = int(rng.choice([1, 2, 3]))
    N = int(rng.choice([int(rng.integers(2, 3000)), int(rng.integers(3000, 20000)), int(rng.integers(20000, 50000))]))
    B = int(rng.choice([1, 2])) if N < 20000 else 1
    mode = str(rng.choice(["lse", "lse", "mean", "mean_var"]))
    w = S.Workload(f"fz{i}", B, N, G * Hkv, Hkv, int(rng.choice([64, 128])), C, g, K, "bf16", 5000 + i,
                   str(rng.choice(["iid", "walk", "needle64"])))
    return w, mode


@pytest.mark.skipif(int(os.environ.get("PISA_FUZZ_EXTRA", "0")) <= 0,
                    reason="opt-in: PISA_FUZZ_EXTRA=<number of shapes> (about 0.7 s per shape)")
def test_extended_random_shapes_match_oracle():
    """The wider draw (sequence lengths to 50000, G = 16, K to 32, three KV heads, all three score modes, three input
    distributions), as many shapes as PISA_FUZZ_EXTRA asks for, sampled rows against the compiled oracle and the
    tie-band walk against the NumPy one."""
    n = int(os.environ["PISA_FUZZ_EXTRA"])
    for i in range(n):
        w, mode = _draw_wide(np.random.default_rng(10_000 + i), i)
        t = S.make_inputs(w)
        dev = T.Device(w, t, score_mode=mode)
        dev.forward()
        assert dev.sync_status() == 0, (i, w)
        tri = S.sample_queries(w, 24)
        T.check_forward_dev(dev, T.oracle_problem_c(w, t, mode=mode), tri, walk_prob=T.oracle_problem(w, t, mode=mode))
        del dev
