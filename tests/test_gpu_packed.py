"""Packed variable-length batches: every sequence of the pack must come out exactly as pisa_forward gives it
alone (own block grid, own hierarchy), and sampled rows must match the oracle run on that sequence."""
import numpy as np
import pytest
import torch

import pisa_synth as S

pytestmark = pytest.mark.gpu

import pisa_testlib as T  # noqa: E402
import paper_2609_31093_b200 as P  # noqa: E402
from paper_2609_31093_b200 import binding as PB  # noqa: E402


launches = {}


@pytest.mark.parametrize("op", ["forward", "packed"])
def test_packed_sequences_equal_the_sequences_alone_and_the_oracle(op):
    """op = "forward": a workspace sized for one sequence (the call then runs the sequences one after the
    other); "packed": the padded groups (700/640/600 share one, 130/120/100 another, 64/60 a third; 2085, 1
    and 70000 run alone)."""
    lens = [700, 64, 1, 2085, 0, 130, 70000, 640, 600, 120, 100, 60]   # 70000: long enough to run as two chunks
    Hq, Hkv, d, C, g, K = 8, 2, 128, 64, 2, 4
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    parts = []
    for i, n in enumerate(lens):
        parts.append(S.make_inputs(S.Workload(f"pk{i}", 1, max(n, 1), Hq, Hkv, d, C, g, K, "bf16", 700 + i, "iid")))
    cat = lambda key: np.concatenate([p_[key][0, :n] for p_, n in zip(parts, lens)], axis=0)
    q, k, v = (T.to_torch(cat(x), "bf16") for x in ("q", "k", "v"))          # [total, H, d]
    p = P.Params(1, max(lens), Hq, Hkv, d, C, g, K, dtype="bf16")
    pyramid = PB.alloc_pyramid(p)
    ws = PB.alloc_workspace(p, PB.OP_FORWARD_PACKED if op == "packed" else PB.OP_FORWARD)
    assert P.workspace_bytes(p, PB.OP_FORWARD_PACKED) > P.workspace_bytes(p, PB.OP_FORWARD)
    idx = torch.full((Hkv * K * total,), -7, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    lse = torch.zeros((Hq * total,), dtype=torch.float32, device="cuda")
    n0 = P.launch_count()
    P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    launches[op] = P.launch_count() - n0
    if "packed" in launches and "forward" in launches:
        assert launches["packed"] < launches["forward"]
    for i, n in enumerate(lens):
        if n == 0:
            continue
        t0 = int(cu[i])
        w = S.Workload(f"pk{i}", 1, n, Hq, Hkv, d, C, g, K, "bf16", 700 + i, "iid")
        t = {key: parts[i][key][:, :n] for key in ("q", "k", "v")}
        alone = T.Device(w, t)
        alone.forward()
        assert alone.sync_status() == 0
        got_idx = idx[Hkv * K * t0:Hkv * K * (t0 + n)].view(Hkv, n, K)
        got_lse = lse[Hq * t0:Hq * (t0 + n)].view(Hq, n)
        if op == "forward":
            assert torch.equal(got_idx, alone.idx[0]), i
        else:                                   # other tile compositions: rows may differ only inside the tie band
            differ = (got_idx != alone.idx[0]).any(dim=-1)
            assert int(differ.sum()) <= max(1, got_idx.shape[0] * n // 200), (i, int(differ.sum()))
        same = ~(got_idx != alone.idx[0]).any(dim=-1)                       # [Hkv, n] rows with equal index sets
        same_q = same.repeat_interleave(Hq // Hkv, dim=0)                     # [Hq, n]
        assert bool((((got_lse - alone.lse[0]).abs() <= 1e-5 * alone.lse[0].abs() + 1e-5) | ~same_q).all()), i
        a, b = out[t0:t0 + n].double(), alone.out[0].double()                 # [n, Hq, d]
        ok = ((a - b).abs() <= 2.0 ** -7 * b.abs() + 1e-3).all(dim=-1)
        assert bool((ok | ~same_q.t()).all()), i
        # sampled rows of this sequence against the oracle
        tri = S.sample_queries(w, 12)
        prob = T.oracle_problem(w, t)
        ref_idx, ref_margin = prob.route_all(tri)
        ti = torch.from_numpy(tri)
        gi = got_idx.cpu()[ti[:, 1], ti[:, 2]].numpy()
        n_diff, n_bad, n_band = T.compare_index_sets(gi, ref_idx, ref_margin, prob=prob, triples=tri)
        assert n_bad == 0, i


@pytest.mark.parametrize("op", ["loop", "groups"])
def test_packed_backward_matches_the_oracle_per_sequence(op):
    """Forward then backward over a pack; every sequence's gradients against the oracle run on that sequence
    alone with the indices the forward selected (one sequence is a single partial block, two a single token).
    "loop": a workspace sized for one sequence, one backward per sequence; "groups": the larger workspace, the
    short sequences of similar length as padded batches (six groups here, the two one-token sequences among them)."""
    from oracle import pisa_oracle as O
    lens = [700, 64, 1, 1500, 0, 130, 37, 690, 650, 60, 1400, 1, 125, 33]
    Hq, Hkv, d, C, g, K = 8, 2, 128, 64, 2, 4
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    parts = [S.make_inputs(S.Workload(f"pb{i}", 1, max(n, 1), Hq, Hkv, d, C, g, K, "bf16", 720 + i, "iid"))
             for i, n in enumerate(lens)]
    cat = lambda key: np.concatenate([p_[key][0, :n] for p_, n in zip(parts, lens)], axis=0)
    q, k, v = (T.to_torch(cat(x), "bf16") for x in ("q", "k", "v"))
    p = P.Params(1, max(lens), Hq, Hkv, d, C, g, K, dtype="bf16")
    pyramid = PB.alloc_pyramid(p)
    ws = PB.alloc_workspace(p, PB.OP_FORWARD)
    idx = torch.full((Hkv * K * total,), -7, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    lse = torch.zeros((Hq * total,), dtype=torch.float32, device="cuda")
    P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)
    rng = np.random.default_rng(77)
    dout_bits = S.f32_to_bf16_bits(rng.standard_normal((total, Hq, d)).astype(np.float32))
    dout = T.to_torch(dout_bits, "bf16")
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (q, k, v))
    group, _, n_groups = P.packed_plan(p, cu.tolist())
    assert n_groups == 6 and sum(1 for x in group if x < 0) == 1          # (the empty sequence belongs to no group)
    wsb = PB.alloc_workspace(p, PB.OP_BSA_BWD_PACKED if op == "groups" else PB.OP_BSA_BWD)
    n0 = P.launch_count()
    P.pisa_bsa_bwd_packed(p, cu.tolist(), q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    launches["bwd_" + op] = P.launch_count() - n0
    assert P.read_status(ws) == 0 and P.read_status(wsb) == 0
    if "bwd_loop" in launches and "bwd_groups" in launches:   # 13 backwards against 6 groups
        assert launches["bwd_groups"] < launches["bwd_loop"], launches
    for i, n in enumerate(lens):
        if n == 0:
            continue
        t0 = int(cu[i])
        t = {key: parts[i][key][:, :n] for key in ("q", "k", "v")}
        idx_i = idx[Hkv * K * t0:Hkv * K * (t0 + n)].view(1, Hkv, n, K).cpu().numpy()
        do_i = dout_bits[None, t0:t0 + n]
        rq, rk, rv = O.attend_backward(t["q"], t["k"], t["v"], idx_i, do_i, C=C, dtype="bf16")
        o64 = out[t0:t0 + n].to(torch.float64).cpu().numpy()[None]
        do64 = O.load_storage(do_i, "bf16")
        kmax = float(np.abs(O.load_storage(t["k"], "bf16")).max())
        d_delta = 2.0 ** -9 * np.abs(o64 * do64).sum(axis=-1, keepdims=True) / np.sqrt(d) * kmax
        # a one-token sequence has dS = 0 exactly, so the rounding of delta is all there is in dk too
        qmax = float(np.abs(O.load_storage(t["q"], "bf16")).max())
        dk_extra = float(d_delta.sum()) / kmax * qmax if n == 1 else 0.0
        for nm, got, ref, extra in (("dq", dq, rq, d_delta), ("dk", dk, rk, dk_extra), ("dv", dv, rv, 0.0)):
            g64 = got[t0:t0 + n].to(torch.float64).cpu().numpy()[None]
            assert np.isfinite(g64).all(), (i, nm)
            T.check_gradient_rows(f"seq{i}.{nm}", g64, ref, extra)


def test_many_short_sequences_run_as_a_few_launch_sets():
    """256 sequences of at most 512 tokens: the padded groups against the one-after-the-other loop of the
    same call (same rows up to tie-band differences, far fewer launches, less time), and sampled rows of
    sampled sequences against the oracle run on each sequence alone."""
    rng = np.random.default_rng(4242)
    lens = rng.integers(1, 513, size=256).tolist()
    Hq, Hkv, d, C, g, K = 8, 2, 128, 64, 2, 4
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    w_all = S.Workload("pk_many", 1, total, Hq, Hkv, d, C, g, K, "bf16", 4243, "iid")
    t_all = S.make_inputs(w_all)
    q, k, v = (T.to_torch(t_all[x][0], "bf16") for x in ("q", "k", "v"))      # [total, H, d]
    p = P.Params(1, max(lens), Hq, Hkv, d, C, g, K, dtype="bf16")
    pyramid = PB.alloc_pyramid(p)
    res = {}
    for op in ("forward", "packed"):
        ws = PB.alloc_workspace(p, PB.OP_FORWARD_PACKED if op == "packed" else PB.OP_FORWARD)
        idx = torch.full((Hkv * K * total,), -7, dtype=torch.int32, device="cuda")
        out = torch.zeros_like(q)
        lse = torch.zeros((Hq * total,), dtype=torch.float32, device="cuda")
        P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)      # warm-up
        torch.cuda.synchronize()
        n0 = P.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)
        e1.record()
        torch.cuda.synchronize()
        assert P.read_status(ws) == 0
        res[op] = (idx, out, lse, P.launch_count() - n0, e0.elapsed_time(e1))
    print(f"\n256 sequences <= 512 tokens ({total} tokens): loop {res['forward'][3]} launches {res['forward'][4]:.2f} ms, "
          f"padded groups {res['packed'][3]} launches {res['packed'][4]:.2f} ms")
    assert res["packed"][3] * 4 < res["forward"][3]
    assert res["packed"][4] < res["forward"][4]
    # the two modes against each other: index rows equal except inside the tie band
    ia, ib = res["forward"][0].view(-1, K), res["packed"][0].view(-1, K)
    differ = (ia != ib).any(dim=-1)
    assert int(differ.sum()) <= ia.shape[0] // 200, int(differ.sum())
    assert int((res["packed"][0] == -7).sum()) == 0                               # every row was written
    # sampled sequences against the oracle on the sequence alone
    idx, out, lse = res["packed"][:3]
    for i in rng.choice(256, size=12, replace=False).tolist() + [int(np.argmax(lens)), int(np.argmin(lens))]:
        n, t0 = lens[i], int(cu[i])
        w = S.Workload(f"pk_many{i}", 1, n, Hq, Hkv, d, C, g, K, "bf16", 0, "iid")
        t = {key: t_all[key][:, t0:t0 + n] for key in ("q", "k", "v")}
        tri = S.sample_queries(w, 8)
        prob = T.oracle_problem(w, t)
        ti = torch.from_numpy(tri)
        got_idx = idx[Hkv * K * t0:Hkv * K * (t0 + n)].view(Hkv, n, K)
        gi = got_idx.cpu()[ti[:, 1], ti[:, 2]].numpy()
        G = Hq // Hkv
        heads = ti[:, 1:2] * G + torch.arange(G)[None, :]
        o_g = out[t0:t0 + n].cpu()[ti[:, 2:3], heads].double().numpy()            # [S, G, d]
        l_g = lse[Hq * t0:Hq * (t0 + n)].view(Hq, n).cpu()[heads, ti[:, 2:3]].double().numpy()
        T.check_forward_rows(w, prob, tri, gi, o_g, l_g)


def test_packed_groups_on_the_exact_fp32_path():
    """fp32 inputs (d = 32: the SIMT kernels) through the padded groups: batches of several sequences through the
    exact-arithmetic path, sampled sequences against the oracle run on each sequence alone."""
    rng = np.random.default_rng(99)
    lens = rng.integers(1, 301, size=40).tolist()
    Hq, Hkv, d, C, g, K = 4, 2, 32, 64, 2, 5
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    w_all = S.Workload("pk_f32", 1, total, Hq, Hkv, d, C, g, K, "fp32", 4250, "iid")
    t_all = S.make_inputs(w_all)
    q, k, v = (T.to_torch(t_all[x][0], "fp32") for x in ("q", "k", "v"))
    p = P.Params(1, max(lens), Hq, Hkv, d, C, g, K, dtype="fp32")
    group, padded, n_groups = P.packed_plan(p, cu.tolist())
    assert n_groups >= 3
    pyramid = PB.alloc_pyramid(p)
    ws = PB.alloc_workspace(p, PB.OP_FORWARD_PACKED)
    idx = torch.full((Hkv * K * total,), -7, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    lse = torch.zeros((Hq * total,), dtype=torch.float32, device="cuda")
    P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    assert int((idx == -7).sum()) == 0
    G = Hq // Hkv
    for i in rng.choice(40, size=6, replace=False).tolist() + [int(np.argmax(lens))]:
        n, t0 = lens[i], int(cu[i])
        w = S.Workload(f"pk_f32_{i}", 1, n, Hq, Hkv, d, C, g, K, "fp32", 0, "iid")
        t = {key: t_all[key][:, t0:t0 + n] for key in ("q", "k", "v")}
        tri = S.sample_queries(w, 8)
        prob = T.oracle_problem(w, t)
        ti = torch.from_numpy(tri)
        gi = idx[Hkv * K * t0:Hkv * K * (t0 + n)].view(Hkv, n, K).cpu()[ti[:, 1], ti[:, 2]].numpy()
        heads = ti[:, 1:2] * G + torch.arange(G)[None, :]
        o_g = out[t0:t0 + n].cpu()[ti[:, 2:3], heads].double().numpy()
        l_g = lse[Hq * t0:Hq * (t0 + n)].view(Hq, n).cpu()[heads, ti[:, 2:3]].double().numpy()
        T.check_forward_rows(w, prob, tri, gi, o_g, l_g)


def test_thousands_of_tiny_sequences():
    """5000 sequences of 1 .. 8 tokens: every length up to 15 is on the padded-length grid, so they run as five
    groups (45 launches, not one forward per sequence); sampled sequences against the oracle on each sequence alone;
    the grouped backward runs on the same groups and returns finite gradients for every row."""
    rng = np.random.default_rng(1)
    lens = rng.integers(1, 9, size=5000).tolist()
    Hq, Hkv, d, C, g, K = 8, 2, 128, 64, 2, 4
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    w_all = S.Workload("pk_tiny", 1, total, Hq, Hkv, d, C, g, K, "bf16", 77, "iid")
    t_all = S.make_inputs(w_all)
    q, k, v = (T.to_torch(t_all[x][0], "bf16") for x in ("q", "k", "v"))
    p = P.Params(1, max(lens), Hq, Hkv, d, C, g, K, dtype="bf16")
    group, padded, n_groups = P.packed_plan(p, cu.tolist())
    assert n_groups == 5 and min(group) >= 0
    pyramid = PB.alloc_pyramid(p)
    ws = PB.alloc_workspace(p, PB.OP_FORWARD_PACKED)
    idx = torch.full((Hkv * K * total,), -7, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    lse = torch.zeros((Hq * total,), dtype=torch.float32, device="cuda")
    n0 = P.launch_count()
    P.pisa_forward_packed(p, cu.tolist(), q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    assert P.read_status(ws) == 0
    assert P.launch_count() - n0 < 100
    assert int((idx == -7).sum()) == 0
    G = Hq // Hkv
    for i in rng.choice(5000, size=16, replace=False).tolist():
        n, t0 = lens[i], int(cu[i])
        w = S.Workload(f"pk_tiny{i}", 1, n, Hq, Hkv, d, C, g, K, "bf16", 0, "iid")
        t = {key: t_all[key][:, t0:t0 + n] for key in ("q", "k", "v")}
        tri = S.sample_queries(w, 8)
        prob = T.oracle_problem(w, t)
        ti = torch.from_numpy(tri)
        gi = idx[Hkv * K * t0:Hkv * K * (t0 + n)].view(Hkv, n, K).cpu()[ti[:, 1], ti[:, 2]].numpy()
        heads = ti[:, 1:2] * G + torch.arange(G)[None, :]
        o_g = out[t0:t0 + n].cpu()[ti[:, 2:3], heads].double().numpy()
        l_g = lse[Hq * t0:Hq * (t0 + n)].view(Hq, n).cpu()[heads, ti[:, 2:3]].double().numpy()
        T.check_forward_rows(w, prob, tri, gi, o_g, l_g)
    dout = torch.randn_like(q)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (q, k, v))
    wsb = PB.alloc_workspace(p, PB.OP_BSA_BWD_PACKED)
    n0 = P.launch_count()
    P.pisa_bsa_bwd_packed(p, cu.tolist(), q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert P.read_status(wsb) == 0 and P.launch_count() - n0 < 200
    assert bool(torch.isfinite(dq).all() and torch.isfinite(dk).all() and torch.isfinite(dv).all())
