"""pisa_forward_host (host tensors in and out, one KV head at a time with copies overlapped) must give
what pisa_forward gives on device tensors, and what the oracle gives on sampled rows."""
import numpy as np
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

CASES = {
    # three KV heads: both arena slots are reused, the last unit sits alone in its slot
    "bf16_hkv3_b2": S.Workload("bf16_hkv3_b2", 2, 4096 + 19, 12, 3, 128, 64, 2, 8, "bf16", 201, "iid"),
    "fp32_hkv2": S.Workload("fp32_hkv2", 1, 1536, 4, 2, 64, 64, 2, 4, "fp32", 202, "iid"),
    "bf16_hkv1": S.Workload("bf16_hkv1", 1, 2048, 4, 1, 128, 128, 2, 6, "bf16", 203, "iid"),
}


@pytest.mark.parametrize("name", list(CASES))
def test_host_path_matches_device_path_and_oracle(name):
    w = CASES[name]
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    dev.forward()
    assert dev.sync_status() == 0

    td = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    qh, kh, vh = (x.cpu().pin_memory() for x in (dev.q, dev.k, dev.v))
    out_h = torch.zeros(dev.q.shape, dtype=td).pin_memory()
    lse_h = torch.zeros((w.B, w.Hq, w.N), dtype=torch.float32).pin_memory()
    idx_h = torch.full((w.B, w.Hkv, w.N, w.K), -9, dtype=torch.int32).pin_memory()
    arena = PB.alloc_workspace(dev.p, PB.OP_FORWARD_HOST)
    for _ in range(2):                       # the second call reuses a warm arena
        P.pisa_forward_host(dev.p, qh, kh, vh, out_h, lse_h, idx_h, arena)
    assert P.read_status(arena) == 0

    # selection is deterministic: same indices as the device path
    assert torch.equal(idx_h, dev.idx.cpu())
    # attention partials are added in a different order (fp32 atomics): one output ulp at most
    a, b = out_h.to(torch.float64), dev.out.cpu().to(torch.float64)
    tol = 2.0 ** -7 * b.abs() + 1e-3 if w.dtype == "bf16" else 1e-5 * (1 + b.abs())
    assert bool(((a - b).abs() <= tol).all())
    assert torch.allclose(lse_h, dev.lse.cpu(), rtol=1e-5, atol=1e-5)

    # and sampled rows against the oracle
    tri = S.sample_queries(w, 40)
    prob = T.oracle_problem(w, t)
    ti = torch.from_numpy(tri)
    got = idx_h[ti[:, 0], ti[:, 1], ti[:, 2]].numpy()
    G = w.Hq // w.Hkv
    heads = ti[:, 1:2] * G + torch.arange(G)[None, :]
    o = out_h[ti[:, 0:1], ti[:, 2:3], heads].to(torch.float64).numpy()
    l = lse_h[ti[:, 0:1], heads, ti[:, 2:3]].to(torch.float64).numpy()
    T.check_forward_rows(w, prob, tri, got, o, l)
