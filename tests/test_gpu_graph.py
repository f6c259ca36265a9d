"""The asynchronous entry points are plain stream work: no allocation, no synchronisation, no host
read-back.  So a call can be captured into a CUDA graph and replayed, and the replay gives what the
eager call gives (indices exactly; outputs up to the order of the fp32 accumulator additions).
The forward here is large enough to run as chunks on the caller's stream and the library's internal
one (fork after the pyramid, join before the end), which the capture must follow; and chunked and
unsplit forwards must agree."""
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

W = S.Workload("graph_gqa4", 2, 40000, 8, 2, 128, 128, 2, 6, "bf16", 501, "iid")     # 2 chunks (one batch each)


def _capture(fn):
    """Warm up on a side stream (first calls configure kernel attributes), then capture one call."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fn()
    return graph


def test_forward_replays_from_a_cuda_graph():
    t = S.make_inputs(W)
    dev = T.Device(W, t)
    dev.forward()
    assert dev.sync_status() == 0
    idx, out, lse = dev.idx.clone(), dev.out.clone(), dev.lse.clone()
    graph = _capture(dev.forward)
    for _ in range(2):
        dev.idx.fill_(-7)
        dev.out.zero_()
        dev.lse.zero_()
        graph.replay()
        assert dev.sync_status() == 0
        assert torch.equal(dev.idx, idx)
        assert torch.allclose(dev.out.float(), out.float(), rtol=0, atol=2.0 ** -7 * float(out.float().abs().max()))
        assert torch.allclose(dev.lse, lse, rtol=1e-5, atol=1e-5)


def test_backward_replays_from_a_cuda_graph():
    t = S.make_inputs(W)
    dev = T.Device(W, t)
    dev.forward()
    gen = torch.Generator(device="cuda").manual_seed(7)
    dout = torch.randn(dev.out.shape, generator=gen, device="cuda").to(torch.bfloat16)
    dq, dk, dv = torch.zeros_like(dev.q), torch.zeros_like(dev.k), torch.zeros_like(dev.v)
    ws = PB.alloc_workspace(dev.p, PB.OP_BSA_BWD)

    def bwd():
        P.pisa_bsa_bwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dout, dq, dk, dv, ws)

    bwd()
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    ref = [x.float().clone() for x in (dq, dk, dv)]
    graph = _capture(bwd)
    for x in (dq, dk, dv):
        x.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    for got, want in zip((dq, dk, dv), ref):
        assert torch.allclose(got.float(), want, rtol=0, atol=2.0 ** -6 * float(want.abs().max()))


@pytest.mark.parametrize("B,Hkv,N", [(3, 2, 50000), (4, 1, 70000), (1, 4, 66000)])
def test_chunked_forward_equals_the_unsplit_one(B, Hkv, N):
    """Chunks of whole batches, of one batch each, and of head ranges of a single batch."""
    w = S.Workload(f"chunks_b{B}", B, N, 4 * Hkv, Hkv, 64, 64, 2, 5, "bf16", 510 + B, "iid")
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    P.set_forward_chunks(1)
    try:
        dev.forward()
        assert dev.sync_status() == 0
    finally:
        P.set_forward_chunks(0)
    idx, out, lse, pyr = dev.idx.clone(), dev.out.clone(), dev.lse.clone(), dev.pyramid.clone()
    dev.idx.fill_(-7)
    dev.out.zero_()
    dev.lse.zero_()
    dev.pyramid.zero_()
    dev.forward()
    assert dev.sync_status() == 0
    assert torch.equal(dev.pyramid, pyr)
    assert torch.equal(dev.idx, idx)
    assert torch.allclose(dev.lse, lse, rtol=1e-5, atol=1e-5)
    assert torch.allclose(dev.out.float(), out.float(), rtol=0, atol=2.0 ** -7 * float(out.float().abs().max()))
