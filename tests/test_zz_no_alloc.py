"""pisa_route_static: routing for callers that may not allocate device memory (the scratch is a
device array inside the library).  Collected last on purpose, so that a failure here cannot hide the
other tests in a run that stops at the first failure.  It has to pass alone in a fresh process and
after everything else has used the library."""
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

CASES = [
    # tensor-core path (bf16, GQA) and the exact-fp32 path; both use routing scratch
    S.Workload("static_bf16", 1, 4096, 8, 2, 128, 64, 2, 8, "bf16", 301, "iid"),
    S.Workload("static_fp32", 1, 1536, 2, 1, 64, 64, 2, 4, "fp32", 302, "iid"),
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_static_scratch_routing_equals_workspace_routing_twice(w):
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    assert P.workspace_bytes(dev.p, PB.OP_ROUTE) <= P.route_static_capacity()
    dev.build_pyramid()
    dev.route()                                   # existing entry point, caller-provided workspace
    assert dev.sync_status() == 0
    ref_idx, ref_margin = dev.idx.clone(), dev.margin.clone()
    for call in range(2):                         # two calls in a row share the library's array
        dev.idx.fill_(-9)
        dev.margin.fill_(-1.0)
        P.pisa_route_static(dev.p, dev.q, dev.k, dev.pyramid, dev.idx, dev.margin)
        torch.cuda.synchronize()
        assert torch.equal(dev.idx, ref_idx), f"call {call}: indices differ"
        # margins are the same arithmetic on the same data; the tolerance is the one the parity tests use
        fin = torch.isfinite(ref_margin)
        assert torch.equal(torch.isfinite(dev.margin), fin)
        assert torch.allclose(dev.margin[fin], ref_margin[fin], rtol=0, atol=2e-5)


def test_static_scratch_call_on_a_large_problem_allocates_nothing_and_uses_no_second_stream():
    """B * Hkv * N >= 131072: pisa_route would cut this problem into chunks on a library-owned second
    stream (created on first use).  The allocation-free entry point must run it as one sequence on the
    caller's stream: same result, and the device's free memory does not move across the call."""
    w = S.Workload("static_large", 1, 65536, 2, 2, 128, 64, 2, 4, "bf16", 303, "iid")
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    assert P.workspace_bytes(dev.p, PB.OP_ROUTE) <= P.route_static_capacity()
    dev.build_pyramid()
    dev.route()
    assert dev.sync_status() == 0
    ref_idx = dev.idx.clone()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for call in range(2):
            dev.idx.fill_(-9)
            stream.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            P.pisa_route_static(dev.p, dev.q, dev.k, dev.pyramid, dev.idx, None)
            stream.synchronize()            # only the caller's stream: work on any other stream would not be waited for
            free_after = torch.cuda.mem_get_info()[0]
            assert torch.equal(dev.idx, ref_idx), f"call {call}: indices differ"
            if call == 1:                   # the first call may look up the array's address; the second does nothing but launch
                assert free_after == free_before


def test_static_scratch_refuses_problems_beyond_its_capacity():
    big = P.Params(1, 131072, 32, 8, 128, 128, 2, 32)      # needs > 1 GB of routing scratch
    assert P.workspace_bytes(big, PB.OP_ROUTE) > P.route_static_capacity()
    dummy = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(P.PisaError, match="built-in device array"):
        P.pisa_route_static(big, dummy, dummy, dummy, idx, None)
