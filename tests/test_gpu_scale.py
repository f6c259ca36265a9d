"""A caller-supplied softmax scale (params.scale > 0 replaces 1 / sqrt(d) in every score and in the
attention): routing, forward, backward and one decoding step against the oracle run with the same scale."""
import numpy as np
import pytest
import torch

import pisa_synth as S
from oracle import pisa_oracle as O

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

W = S.Workload("scale_gqa4", 1, 2048 + 300, 8, 2, 128, 64, 2, 5, "bf16", 951, "iid")
SCALE = 0.21


@pytest.mark.parametrize("impl", [PB.IMPL_SIMT, PB.IMPL_AUTO])
def test_custom_scale(impl):
    w = W
    t = S.make_inputs(w)
    prob = O.Problem(t["q"], t["k"], t["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype, scale=SCALE)
    p = P.Params(w.B, w.N, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype="bf16", impl=impl, scale=SCALE)
    q, k, v = (T.to_torch(t[x], "bf16") for x in ("q", "k", "v"))
    pyramid = PB.alloc_pyramid(p)
    idx = torch.full((w.B, w.Hkv, w.N, w.K), -7, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    lse = torch.zeros((w.B, w.Hq, w.N), dtype=torch.float32, device="cuda")
    ws = PB.alloc_workspace(p, PB.OP_FORWARD)
    P.pisa_forward(p, q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    tri = S.sample_queries(w, 120)
    got = T.gather_idx(idx, tri)
    ti = torch.from_numpy(tri)
    G = w.Hq // w.Hkv
    o = out.view(w.B, w.N, w.Hkv, G, w.d)[ti[:, 0], ti[:, 2], ti[:, 1]].to(torch.float64).cpu().numpy()
    l = lse.view(w.B, w.Hkv, G, w.N)[ti[:, 0], ti[:, 1], :, ti[:, 2]].to(torch.float64).cpu().numpy()
    n_diff, n_band, _ = T.check_forward_rows(w, prob, tri, got, o, l)
    assert n_diff < 0.1 * len(tri)
    if impl == PB.IMPL_AUTO:
        rng = np.random.default_rng(3)
        dout_bits = S.f32_to_bf16_bits(rng.standard_normal(t["q"].shape).astype(np.float32))
        dout = T.to_torch(dout_bits, "bf16")
        dq, dk, dv = (torch.zeros_like(x) for x in (q, k, v))
        wsb = PB.alloc_workspace(p, PB.OP_BSA_BWD)
        P.pisa_bsa_bwd(p, q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
        torch.cuda.synchronize()
        assert P.read_status(wsb) == 0
        rq, rk, rv = O.attend_backward(t["q"], t["k"], t["v"], idx.cpu().numpy(), dout_bits, C=w.C, dtype="bf16",
                                       scale=SCALE)
        o64 = out.to(torch.float64).cpu().numpy()
        do64 = O.load_storage(dout_bits, "bf16")
        kmax = float(np.abs(O.load_storage(t["k"], "bf16")).max())
        d_delta = 2.0 ** -9 * np.abs(o64 * do64).sum(axis=-1, keepdims=True) * SCALE * kmax
        for nm, got_g, ref, extra in (("dq", dq, rq, d_delta), ("dk", dk, rk, 0.0), ("dv", dv, rv, 0.0)):
            T.check_gradient_rows(nm, got_g.to(torch.float64).cpu().numpy(), ref, extra)
        # one decoding step at the last position of the same sequence
        pd = P.Params(w.B, w.N, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype="bf16", scale=SCALE)
        pos = w.N - 1
        didx = torch.full((w.B, w.Hkv, w.K), -7, dtype=torch.int32, device="cuda")
        dout_t = torch.zeros((w.B, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
        dlse = torch.zeros((w.B, w.Hq), dtype=torch.float32, device="cuda")
        wsd = PB.alloc_workspace(pd, PB.OP_DECODE)
        P.pisa_decode_step(pd, pos, q[:, pos].contiguous(), k, v, pyramid, didx, dout_t, dlse, wsd)
        torch.cuda.synchronize()
        assert P.read_status(wsd) == 0
        ridx, rmargin, rout, rlse = O.decode_step(t["q"][:, pos], t["k"], t["v"], pos, C=w.C, g=w.g, K=w.K,
                                                  dtype="bf16", scale=SCALE)
        gi = didx.cpu().numpy()
        for b in range(w.B):
            for h in range(w.Hkv):
                if rmargin[b, h] > T.TIE_BAND:
                    assert np.array_equal(gi[b, h], ridx[b, h])
        if np.array_equal(gi, ridx):
            T.check_outputs(dout_t.to(torch.float64).cpu().numpy(), dlse.to(torch.float64).cpu().numpy(), rout, rlse, "bf16")
