"""Pins for the oracle's attention backward (App. B: frozen indices): torch autograd on a dense masked
softmax attention built from the same index sets, central finite differences of the oracle's own
forward, and the dense causal special case."""
import math

import numpy as np
import torch

import pisa_synth as S
from oracle import pisa_oracle as O


def _case(seed=501, N=96, Hq=4, Hkv=2, d=16, C=8, g=2, K=4, dtype="fp32"):
    w = S.Workload("bwd", 1, N, Hq, Hkv, d, C, g, K, dtype, seed, "iid")
    t = S.make_inputs(w)
    prob = O.Problem(t["q"], t["k"], t["v"], C=C, g=g, K=K, dtype=dtype)
    idx, _ = prob.route_all()
    idx = idx.reshape(1, Hkv, N, K)
    rng = np.random.default_rng(seed)
    dout = rng.standard_normal(t["q"].shape).astype(np.float32)
    if dtype == "bf16":
        dout = S.f32_to_bf16_bits(dout)
    return w, t, idx, dout


def _mask_from_idx(idx, N, C):
    """[Hkv, N, N] boolean: key j visible to query p."""
    Hkv = idx.shape[1]
    m = np.zeros((Hkv, N, N), dtype=bool)
    for h in range(Hkv):
        for p in range(N):
            for i in idx[0, h, p]:
                if i >= 0:
                    lo, hi = int(i) * C, min((int(i) + 1) * C, N)
                    m[h, p, lo:min(hi, p + 1)] = True
    return m


def test_backward_matches_torch_autograd_on_the_masked_dense_attention():
    w, t, idx, dout = _case()
    dq, dk, dv = O.attend_backward(t["q"], t["k"], t["v"], idx, dout, C=w.C, dtype=w.dtype)
    q = torch.tensor(t["q"], dtype=torch.float64, requires_grad=True)
    k = torch.tensor(t["k"], dtype=torch.float64, requires_grad=True)
    v = torch.tensor(t["v"], dtype=torch.float64, requires_grad=True)
    mask = torch.from_numpy(_mask_from_idx(idx, w.N, w.C)).repeat_interleave(w.G, dim=0)[None]   # [1,Hq,N,N]
    out = torch.nn.functional.scaled_dot_product_attention(
        q.permute(0, 2, 1, 3), k.permute(0, 2, 1, 3).repeat_interleave(w.G, dim=1),
        v.permute(0, 2, 1, 3).repeat_interleave(w.G, dim=1), attn_mask=mask)
    out.backward(torch.tensor(dout, dtype=torch.float64).permute(0, 2, 1, 3))
    assert np.allclose(dq, q.grad.numpy(), atol=1e-10)
    assert np.allclose(dk, k.grad.numpy(), atol=1e-10)
    assert np.allclose(dv, v.grad.numpy(), atol=1e-10)


def test_backward_matches_finite_differences_of_the_oracle_forward():
    w, t, idx, dout = _case(seed=502, N=40, Hq=2, Hkv=1, d=8, C=8, K=3)
    dq, dk, dv = O.attend_backward(t["q"], t["k"], t["v"], idx, dout, C=w.C, dtype=w.dtype)

    def loss(q_, k_, v_):
        tot = 0.0
        for p in range(w.N):
            for hq in range(w.Hq):
                o, _ = O.attend_query(q_[0, p, hq], k_[0, :, 0], v_[0, :, 0], p, idx[0, 0, p], w.C, 1.0 / math.sqrt(w.d))
                tot += float(o @ dout[0, p, hq].astype(np.float64))
        return tot

    base = [t[n].astype(np.float64) for n in ("q", "k", "v")]
    rng = np.random.default_rng(3)
    for which, grad in enumerate((dq, dk, dv)):
        for _ in range(6):
            pos = tuple(int(rng.integers(0, s)) for s in base[which].shape)
            eps = 1e-5
            hi = [x.copy() for x in base]; hi[which][pos] += eps
            lo = [x.copy() for x in base]; lo[which][pos] -= eps
            fd = (loss(*hi) - loss(*lo)) / (2 * eps)
            assert math.isclose(fd, grad[pos], rel_tol=1e-6, abs_tol=1e-8), (which, pos, fd, grad[pos])


def test_backward_is_dense_causal_when_the_budget_covers_everything():
    w = S.Workload("bwd_dense", 1, 48, 2, 1, 16, 8, 2, 6, "fp32", 503, "iid")       # K*C = 48 = N
    t = S.make_inputs(w)
    idx = np.full((1, 1, w.N, w.K), -1, dtype=np.int32)
    for p in range(w.N):
        c = p // w.C
        idx[0, 0, p, :c + 1] = np.arange(c + 1)
    dout = np.random.default_rng(5).standard_normal(t["q"].shape).astype(np.float32)
    dq, dk, dv = O.attend_backward(t["q"], t["k"], t["v"], idx, dout, C=w.C, dtype=w.dtype)
    q = torch.tensor(t["q"], dtype=torch.float64, requires_grad=True)
    k = torch.tensor(t["k"], dtype=torch.float64, requires_grad=True)
    v = torch.tensor(t["v"], dtype=torch.float64, requires_grad=True)
    out = torch.nn.functional.scaled_dot_product_attention(
        q.permute(0, 2, 1, 3), k.permute(0, 2, 1, 3).repeat_interleave(2, dim=1),
        v.permute(0, 2, 1, 3).repeat_interleave(2, dim=1), is_causal=True)
    out.backward(torch.tensor(dout, dtype=torch.float64).permute(0, 2, 1, 3))
    assert np.allclose(dq, q.grad.numpy(), atol=1e-10) and np.allclose(dk, k.grad.numpy(), atol=1e-10)
    assert np.allclose(dv, v.grad.numpy(), atol=1e-10)
