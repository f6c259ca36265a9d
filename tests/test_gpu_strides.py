"""Strided tensors through the C ABI: q, k, v and out stored head-major ([B, H, N, d]) and described by
element strides must give what the dense token-major layout gives, on the exact-fp32 kernels, on the
tensor-core kernels, and for a problem large enough to run as chunks on two streams (whose sub-problems
are themselves strided views)."""
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

CASES = {
    "gqa4": S.Workload("strided_gqa4", 2, 3000, 8, 2, 128, 64, 2, 6, "bf16", 901, "iid"),
    "chunked": S.Workload("strided_chunked", 2, 40000, 8, 2, 64, 64, 2, 5, "bf16", 902, "iid"),
}


def _head_major(x):
    """[B, N, H, d] -> storage [B, H, N, d] and its (batch, token, head) element strides."""
    B, N, H, d = x.shape
    hm = x.permute(0, 2, 1, 3).contiguous()
    return hm, (H * N * d, d, N * d)


@pytest.mark.parametrize("name,impl", [("gqa4", PB.IMPL_SIMT), ("gqa4", PB.IMPL_AUTO), ("chunked", PB.IMPL_AUTO)])
def test_head_major_tensors_by_strides(name, impl):
    w = CASES[name]
    t = S.make_inputs(w)
    dev = T.Device(w, t, impl=impl)
    dev.forward()
    assert dev.sync_status() == 0
    q, qs = _head_major(dev.q)
    k, ks = _head_major(dev.k)
    v, vs = _head_major(dev.v)
    out = torch.zeros_like(q)
    p = P.Params(w.B, w.N, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype="bf16", impl=impl).set_strides(q=qs, k=ks, v=vs, o=qs)
    pyramid = PB.alloc_pyramid(p)
    idx = torch.full_like(dev.idx, -7)
    lse = torch.zeros_like(dev.lse)
    ws = PB.alloc_workspace(p, PB.OP_FORWARD)
    P.pisa_forward(p, q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    assert torch.equal(pyramid, dev.pyramid)
    assert torch.equal(idx, dev.idx)
    assert torch.allclose(lse, dev.lse, rtol=1e-5, atol=1e-5)
    got = out.permute(0, 2, 1, 3).float()
    want = dev.out.float()
    assert torch.allclose(got, want, rtol=0, atol=2.0 ** -7 * float(want.abs().max()))
    if impl == PB.IMPL_AUTO:
        # backward: out and dout strided like out; dq, dk, dv dense
        gen = torch.Generator(device="cuda").manual_seed(5)
        dout_dense = torch.randn(dev.out.shape, generator=gen, device="cuda").to(torch.bfloat16)
        dout, _ = _head_major(dout_dense)
        wsb = PB.alloc_workspace(p, PB.OP_BSA_BWD)
        g_s = [torch.zeros_like(x) for x in (dev.q, dev.k, dev.v)]
        P.pisa_bsa_bwd(p, q, k, v, idx, out, lse, dout, g_s[0], g_s[1], g_s[2], wsb)
        wsd = PB.alloc_workspace(dev.p, PB.OP_BSA_BWD)
        g_d = [torch.zeros_like(x) for x in (dev.q, dev.k, dev.v)]
        P.pisa_bsa_bwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dout_dense, g_d[0], g_d[1], g_d[2], wsd)
        torch.cuda.synchronize()
        assert P.read_status(wsb) == 0 and P.read_status(wsd) == 0
        for a, b in zip(g_s, g_d):
            assert torch.allclose(a.float(), b.float(), rtol=0, atol=2.0 ** -6 * float(b.float().abs().max()))
