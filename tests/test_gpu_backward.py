"""Backward of the block-sparse attention with frozen indices (App. B) against the oracle.

Both sides use the index sets the CUDA forward selected.  Tolerance: the kernel rounds P and dS to bf16
before the gradient products and the results to bf16 at the end (2^-9 relative each).  A gradient row (one
token and head of dq, one key of dk / dv) is a signed sum of terms whose size is set by the row, not by the
element, and rows differ by orders of magnitude (the first tokens see a handful of keys with probabilities
near one), so the bound is per row.  The softmax-gradient correction delta = rowsum(dO o O) is taken from the
bf16 `out` the caller passes (as every fused attention backward does) while the oracle uses the unrounded O:
that shifts dS of a whole row by up to ~2^-9 sqrt(d) |dO||O|, which matters for rows with few keys.
Bound: |err| <= 2^-5 max|ref_row| + 1e-2 rms(ref), plus for dq the delta term scale * 2^-9 sum_d |dO_d O_d| *
max|k| of its row; the mean error must stay below 4e-3 rms(ref) (measured: about 1.5e-3)."""
import numpy as np
import pytest
import torch

import pisa_synth as S
from oracle import pisa_oracle as O

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402

CASES = {
    "gqa4_c64_ragged": S.Workload("bwd_gqa4_c64", 1, 1024 + 21, 8, 2, 128, 64, 2, 4, "bf16", 601, "iid"),
    "gqa4_c128": S.Workload("bwd_gqa4_c128", 1, 1536, 4, 1, 128, 128, 2, 3, "bf16", 602, "iid"),
    "mha_c64_fan4_b2": S.Workload("bwd_mha_c64", 2, 640, 2, 2, 128, 64, 4, 5, "bf16", 603, "walk"),
    "g16_c128": S.Workload("bwd_g16_c128", 1, 768, 16, 1, 128, 128, 2, 4, "bf16", 604, "iid"),
    "d64_c64_g16": S.Workload("bwd_d64_c64", 1, 1100, 16, 1, 64, 64, 2, 4, "bf16", 605, "iid"),
    "d64_c128_gqa2": S.Workload("bwd_d64_c128", 1, 900, 4, 2, 64, 128, 2, 3, "bf16", 606, "walk"),
    # shapes whose forward runs on the SIMT kernels (g*C = 512; a single partial leaf): the backward only
    # needs the leaf-level lists
    "fan4_c128": S.Workload("bwd_fan4_c128", 1, 1100, 4, 2, 128, 128, 4, 4, "bf16", 607, "iid"),
    "single_leaf": S.Workload("bwd_single_leaf", 2, 50, 8, 2, 128, 64, 2, 4, "bf16", 608, "iid"),
}


def _close(name, got, ref, extra=0.0):
    rms = float(np.sqrt(np.mean(ref * ref)))
    err = np.abs(got - ref)
    bound = 2.0 ** -5 * np.abs(ref).max(axis=-1, keepdims=True) + 1e-2 * rms + extra
    assert np.all(err <= bound), f"{name}: max excess {(err - bound).max():.3e} (rms {rms:.3e})"
    assert err.mean() <= 4e-3 * rms, f"{name}: mean err {err.mean():.3e} vs rms {rms:.3e}"
    return float(err.max() / rms), float(err.mean() / rms)


@pytest.mark.parametrize("name", list(CASES))
def test_backward_matches_oracle(name):
    w = CASES[name]
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    dev.forward()
    assert dev.sync_status() == 0
    rng = np.random.default_rng(w.seed)
    dout_bits = S.f32_to_bf16_bits(rng.standard_normal(t["q"].shape).astype(np.float32))
    dout = T.to_torch(dout_bits, "bf16")
    dq = torch.full_like(dev.q, float("nan"))
    dk = torch.full_like(dev.k, float("nan"))
    dv = torch.full_like(dev.v, float("nan"))
    ws = PB.alloc_workspace(dev.p, PB.OP_BSA_BWD)
    for _ in range(2):                                     # a second call on a used workspace gives the same
        P.pisa_bsa_bwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dout, dq, dk, dv, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    idx = dev.idx.cpu().numpy()
    rq, rk, rv = O.attend_backward(t["q"], t["k"], t["v"], idx, dout_bits, C=w.C, dtype="bf16")
    # delta term of dq rows: |d(delta)| <= 2^-9 sum_d |dO_d O_d|, carried into dq by scale * sum_j p_j k_j
    o64 = dev.out.to(torch.float64).cpu().numpy()
    do64 = O.load_storage(dout_bits, "bf16")
    kmax = float(np.abs(O.load_storage(t["k"], "bf16")).max())
    d_delta = 2.0 ** -9 * np.abs(o64 * do64).sum(axis=-1, keepdims=True) / np.sqrt(w.d) * kmax
    res = {}
    for nm, got, ref, extra in (("dq", dq, rq, d_delta), ("dk", dk, rk, 0.0), ("dv", dv, rv, 0.0)):
        g64 = got.to(torch.float64).cpu().numpy()
        assert np.isfinite(g64).all(), nm
        res[nm] = _close(nm, g64, ref, extra)
    print(f"[{name}] max/rms, mean/rms: " + ", ".join(f"{k}: {v[0]:.2e} {v[1]:.2e}" for k, v in res.items()))


def test_backward_rejects_unsupported_head_dim():
    p = P.Params(1, 1024, 4, 2, 32, 64, 2, 4)
    with pytest.raises(P.PisaError, match="unsupported"):
        P.workspace_bytes(p, PB.OP_BSA_BWD)


def test_backward_at_the_headline_size_sampled_rows_and_identities():
    """cfg4 in the launch configuration bench.py --backward times: sampled dq rows against the oracle and two
    identities that hold at any size: sum over keys of dv = sum over the group's rows of dO (probabilities of a
    row add up to one) and sum over keys of dk = 0 (the dS of a row add up to zero)."""
    w = S.WORKLOADS["cfg4"]
    t = S.make_inputs(w)
    dev = T.Device(w, t)
    dev.forward()
    assert dev.sync_status() == 0
    gen = torch.Generator(device="cuda").manual_seed(5)
    dout = torch.randn(dev.q.shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    dq, dk, dv = torch.empty_like(dev.q), torch.empty_like(dev.k), torch.empty_like(dev.v)
    del dev.ws
    ws = PB.alloc_workspace(dev.p, PB.OP_BSA_BWD)
    P.pisa_bsa_bwd(dev.p, dev.q, dev.k, dev.v, dev.idx, dev.out, dev.lse, dout, dq, dk, dv, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    G = w.G
    # identities, per (b, KV head), in fp64 on the device
    dv_sum = dv.double().sum(dim=1)                                              # [B, Hkv, d]
    do_sum = dout.double().view(w.B, w.N, w.Hkv, G, w.d).sum(dim=(1, 3))         # [B, Hkv, d]
    scale_v = dout.double().abs().view(w.B, w.N, w.Hkv, G, w.d).sum(dim=(1, 3))
    assert bool(((dv_sum - do_sum).abs() <= 2.0 ** -8 * scale_v).all())
    dk_sum = dk.double().sum(dim=1)
    assert bool((dk_sum.abs() <= 2.0 ** -8 * dk.double().abs().sum(dim=1)).all())
    # sampled dq rows (the compiled oracle: 256 positions per KV head)
    tri = S.sample_queries(w, 256)
    prob = T.oracle_problem_c(w, t)
    ti = torch.from_numpy(tri).cuda()
    idx_rows = dev.idx[ti[:, 0], ti[:, 1], ti[:, 2]].cpu().numpy()
    heads = ti[:, 1:2] * G + torch.arange(G, device="cuda")[None, :]
    do_rows = T.from_torch(dout[ti[:, 0:1], ti[:, 2:3], heads], "bf16")
    ref = prob.backward_rows(tri, idx_rows, do_rows)                            # [S, G, d]
    got = dq[ti[:, 0:1], ti[:, 2:3], heads].double().cpu().numpy()
    o64 = dev.out[ti[:, 0:1], ti[:, 2:3], heads].double().cpu().numpy()
    do64 = O.load_storage(do_rows, "bf16")
    kmax = float(dev.k.abs().max())
    d_delta = 2.0 ** -9 * np.abs(o64 * do64).sum(axis=-1, keepdims=True) / np.sqrt(w.d) * kmax
    _close("dq rows", got, ref, d_delta)

    # dk and dv of two whole key blocks of one KV head: the oracle's contributions of EVERY row that selected
    # the block (found in the index tensor the backward was given), accumulated in fp64
    for h, blk0 in ((1, 517), (6, 40)):
        blk = blk0
        while True:                                                             # a block a bounded number of rows selected
            rows_sel = (dev.idx[0, h] == blk).any(dim=1).nonzero().flatten()    # positions that selected the block
            if 0 < len(rows_sel) <= 8192:
                break
            blk += 1
        tri_b = np.stack([np.zeros(len(rows_sel), dtype=np.int64), np.full(len(rows_sel), h, dtype=np.int64),
                          rows_sel.cpu().numpy()], axis=1)
        tb = torch.from_numpy(tri_b).cuda()
        idx_b = dev.idx[0, h][rows_sel].cpu().numpy()
        heads_b = tb[:, 1:2] * G + torch.arange(G, device="cuda")[None, :]
        do_b = T.from_torch(dout[tb[:, 0:1], tb[:, 2:3], heads_b], "bf16")
        lo, hi = blk * w.C, (blk + 1) * w.C
        _, rdk, rdv = prob.backward_rows(tri_b, idx_b, do_b, key_range=(lo, hi))
        T.check_gradient_rows(f"dk block {blk}", dk[0, lo:hi, h].double().cpu().numpy(), rdk)
        T.check_gradient_rows(f"dv block {blk}", dv[0, lo:hi, h].double().cpu().numpy(), rdv)
        print(f"[cfg4 backward] head {h} block {blk}: {len(rows_sel)} rows contribute")
