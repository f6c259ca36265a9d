"""Seeded random shapes through pisa_forward against the oracle: tiny and ragged sequence lengths, every
supported group size, both leaf sizes and fan-ins of the tensor-core path."""
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
