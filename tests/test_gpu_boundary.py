"""The boundary's extras on a GPU: the sel_lse hand-over between pisa_route and pisa_bsa_fwd, the
device-side index checks (PISA_DEBUG_BOUNDS), the bounded-wait self-test, and pointer-alignment
rejections."""
import numpy as np
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

W_TENSOR = S.Workload("b_gqa4", 1, 4096 + 51, 8, 2, 128, 64, 2, 8, "bf16", 401, "iid")
W_FP32 = S.Workload("b_fp32", 1, 1536, 4, 2, 64, 64, 2, 4, "fp32", 402, "iid")


@pytest.mark.parametrize("w,impl,mode", [(W_TENSOR, PB.IMPL_AUTO, "lse"), (W_TENSOR, PB.IMPL_AUTO, "mean_var"),
                                         (W_TENSOR, PB.IMPL_SIMT, "lse"), (W_FP32, PB.IMPL_AUTO, "lse")],
                         ids=["tensor_lse", "tensor_mean_var", "simt_bf16", "fp32"])
def test_route_then_attention_with_sel_lse_equals_forward(w, impl, mode):
    t = S.make_inputs(w)
    dev = T.Device(w, t, impl=impl, score_mode=mode)
    dev.forward()
    assert dev.sync_status() == 0
    idx_f, out_f, lse_f = dev.idx.clone(), dev.out.clone(), dev.lse.clone()
    sel = torch.full((w.B, w.Hq, w.N, w.K), 7.0, dtype=torch.float32, device="cuda")
    dev.idx.fill_(-5)
    P.pisa_route(dev.p, dev.q, dev.k, dev.pyramid, dev.idx, None, dev.ws, sel_lse=sel)
    assert dev.sync_status() == 0
    assert torch.equal(dev.idx, idx_f)
    # the numbers themselves: the denominator of each kept leaf alone, against the oracle on sampled rows
    prob = T.oracle_problem(w, t, mode=mode)
    tri = S.sample_queries(w, 12)
    G = w.Hq // w.Hkv
    for b, h, p in tri[::3]:
        row = dev.idx[b, h, p].cpu().numpy()
        for s_, leaf in enumerate(row):
            got = sel[b, h * G:(h + 1) * G, p, s_].cpu().numpy()
            if leaf < 0:
                assert np.all(np.isneginf(got))
                continue
            ref = [prob.attend(int(b), int(h) * G + j, int(p), [int(leaf)])[1] for j in range(G)]
            np.testing.assert_allclose(got, ref, rtol=0, atol=1e-3 if w.dtype == "bf16" else 1e-4)
    dev.out.zero_()
    dev.lse.zero_()
    P.pisa_bsa_fwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dev.ws, sel_lse=sel)
    assert dev.sync_status() == 0
    assert torch.allclose(dev.lse, lse_f, rtol=1e-5, atol=1e-5)
    a, b_ = dev.out.double(), out_f.double()
    tol = 2.0 ** -7 * b_.abs() + 1e-3 if w.dtype == "bf16" else 1e-5 * (1 + b_.abs())
    assert bool(((a - b_).abs() <= tol).all())
    # and without the hand-over (attention computes the denominators itself): the same again
    dev.out.zero_()
    P.pisa_bsa_fwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dev.ws)
    assert dev.sync_status() == 0
    assert torch.allclose(dev.lse, lse_f, rtol=1e-4, atol=1e-4)
    assert bool(((dev.out.double() - b_).abs() <= tol).all())


@pytest.mark.parametrize("w,impl", [(W_TENSOR, PB.IMPL_AUTO), (W_TENSOR, PB.IMPL_SIMT),
                                    (S.Workload("b_win2", 1, 16384 + 700, 4, 1, 64, 64, 4, 16, "bf16", 403, "iid"), PB.IMPL_AUTO)],
                         ids=["tensor", "simt", "two_windows"])
def test_bounds_check_mode_is_silent_on_valid_runs_and_flags_bad_indices(w, impl):
    t = S.make_inputs(w)
    plain = T.Device(w, t, impl=impl)
    plain.forward()
    assert plain.sync_status() == 0
    dbg = T.Device(w, t, impl=impl)
    dbg.p = P.Params(dbg.p.B, w.N, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype=w.dtype, impl=impl, debug=P.DEBUG_BOUNDS)
    dbg.forward()
    assert dbg.sync_status() == 0                      # every gathered index was in range
    assert torch.equal(dbg.idx, plain.idx)
    assert torch.allclose(dbg.lse, plain.lse, rtol=1e-5, atol=1e-5)
    if impl == PB.IMPL_SIMT:
        return                                          # the exact-fp32 attention reads idx directly; checks live in the tensor path
    # malformed idx handed to the attention: a leaf that does not exist, and one in the row's future
    bad = plain.idx.clone()
    bad[0, 0, w.N - 1, 1] = 10 ** 6
    bad[0, 0, 100, 1] = (w.N - 1) // w.C
    dbg.bsa(idx=bad)
    torch.cuda.synchronize()
    st = P.read_status(dbg.ws)
    assert st == -6, st                                 # PISA_ERR_BOUNDS, nothing trapped
    # without the mode such entries are skipped silently, and the GPU is fine either way
    plain.bsa(idx=bad)
    assert plain.sync_status() == 0
    dbg.forward()
    assert dbg.sync_status() == 0
    assert torch.equal(dbg.idx, plain.idx)


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_gpu_usable():
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    P.debug_wait_timeout(ws, 2_000_000)                 # 2 ms on a barrier nobody arrives at
    torch.cuda.synchronize()
    assert P.read_status(ws) == -5                      # PISA_ERR_TIMEOUT
    w = W_TENSOR
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    dev.forward()
    assert dev.sync_status() == 0                       # the context still works
    n_diff, n_band, _ = T.check_forward_dev(dev, T.oracle_problem(w, t), S.sample_queries(w, 12))


def test_pyramid_must_be_32_byte_aligned_everywhere():
    w = W_TENSOR
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    off = dev.pyramid[8:]                               # 16-byte aligned only
    assert off.data_ptr() % 32 == 16
    for call in (lambda: P.pisa_build_pyramid(dev.p, dev.k, off),
                 lambda: P.pisa_route(dev.p, dev.q, dev.k, off, dev.idx, None, dev.ws),
                 lambda: P.pisa_forward(dev.p, dev.q, dev.k, dev.v, off, dev.idx, dev.out, dev.lse, dev.ws),
                 lambda: P.pisa_flat_select(dev.p, dev.q, off, dev.idx, dev.ws),
                 lambda: P.pisa_route_static(dev.p, dev.q, dev.k, off, dev.idx, None)):
        with pytest.raises(P.PisaError, match="invalid argument"):
            call()
