"""Decoding step (one launch per token) against the oracle: selected blocks, output, log-sum-exp and
the cached pyramid, for caches grown token by token, for a prefill-built cache continued by steps,
and across a capacity growth."""
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
    # name: (workload, positions checked against the oracle)
    "gqa4_c64": S.Workload("dec_gqa4_c64", 2, 1500, 8, 2, 128, 64, 2, 4, "bf16", 401, "iid"),
    "fan4_c32": S.Workload("dec_fan4_c32", 1, 1400, 4, 2, 64, 32, 4, 6, "bf16", 402, "walk"),
    "g16_c64": S.Workload("dec_g16_c64", 1, 1100, 16, 1, 64, 64, 2, 5, "bf16", 403, "iid"),
    "mha_c128_k8": S.Workload("dec_mha_c128_k8", 1, 4200, 2, 2, 128, 128, 2, 8, "bf16", 404, "iid"),
}


class Cache:
    """KV caches of capacity `cap` filled as a decoder would: row pos is written just before its step;
    everything not yet written is NaN, so any read of the future shows up in the results."""

    def __init__(self, w, t, cap, filled=0, score_mode="lse"):
        self.w, self.cap, self.mode = w, cap, score_mode
        self.p = P.Params(w.B, cap, w.Hq, w.Hkv, w.d, w.C, w.g, w.K, dtype="bf16", score_mode=score_mode)
        self.k_src, self.v_src = T.to_torch(t["k"], "bf16"), T.to_torch(t["v"], "bf16")
        self.k = torch.full((w.B, cap, w.Hkv, w.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        self.v = torch.full_like(self.k, float("nan"))
        self.k[:, :filled] = self.k_src[:, :filled]
        self.v[:, :filled] = self.v_src[:, :filled]
        self.pyr = PB.alloc_pyramid(self.p)
        self.pyr.fill_(float("nan"))
        self.q = T.to_torch(t["q"], "bf16")
        self.idx = torch.full((w.B, w.Hkv, w.K), -7, dtype=torch.int32, device="cuda")
        self.out = torch.zeros((w.B, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
        self.lse = torch.zeros((w.B, w.Hq), dtype=torch.float32, device="cuda")
        self.ws = PB.alloc_workspace(self.p, PB.OP_DECODE)
        self.L, self.M, self.off, _ = P.pyramid_layout(self.p)

    def step(self, pos):
        self.k[:, pos] = self.k_src[:, pos]
        self.v[:, pos] = self.v_src[:, pos]
        P.pisa_decode_step(self.p, pos, self.q[:, pos].contiguous(), self.k, self.v, self.pyr, self.idx, self.out,
                           self.lse, self.ws)

    def level(self, l):
        n = self.w.B * self.w.Hkv * self.M[l] * self.w.d
        return self.pyr[self.off[l]:self.off[l] + n].view(self.w.B, self.w.Hkv, self.M[l], self.w.d)


def _check_step(cache, t, pos):
    w = cache.w
    torch.cuda.synchronize()
    assert P.read_status(cache.ws) == 0
    idx_ref, margin, out_ref, lse_ref = O.decode_step(t["q"][:, pos], t["k"], t["v"], pos, C=w.C, g=w.g, K=w.K,
                                                      dtype="bf16", mode=cache.mode)
    got = cache.idx.cpu().numpy()
    c = pos // w.C
    for b in range(w.B):
        for h in range(w.Hkv):
            row = got[b, h]
            n = min(w.K, c + 1)
            assert np.all(row[n:] == -1) and np.all(np.diff(row[:n]) > 0) and row[n - 1] == c and row[0] == 0, (pos, row)
            if margin[b, h] > T.TIE_BAND:
                assert np.array_equal(row, idx_ref[b, h]), (pos, b, h, row, idx_ref[b, h], margin[b, h])
    same = np.all(got == idx_ref, axis=2)                               # [B, Hkv]
    G = w.Hq // w.Hkv
    mask = np.repeat(same, G, axis=1)                                   # [B, Hq]
    if mask.any():
        o = cache.out.to(torch.float64).cpu().numpy()[mask]
        l = cache.lse.to(torch.float64).cpu().numpy()[mask]
        T.check_outputs(o, l, out_ref[mask], lse_ref[mask], "bf16")
    return int((~same).sum())


@pytest.mark.parametrize("name", list(CASES))
def test_decode_from_an_empty_cache_token_by_token(name):
    w = CASES[name]
    t = S.make_inputs(w)
    cache = Cache(w, t, cap=w.N)
    rng = np.random.default_rng(w.seed)
    check = set([0, 1, w.C - 1, w.C, w.C + 1, w.K * w.C - 1, w.K * w.C, w.K * w.C + 1, w.g * w.K * w.C, w.N - 1])
    check |= set(rng.integers(0, w.N, size=24).tolist())
    in_band = 0
    for pos in range(w.N):
        cache.step(pos)
        if pos in check:
            in_band += _check_step(cache, t, pos)
    print(f"[{name}] checked {len(check)} steps, {in_band} (b, head) rows differed inside the tie band")
    # the cache now holds the pyramid of the whole sequence (bf16: at most one ulp off where the
    # fp32 and fp64 means round differently)
    ref = O.decode_pyramid(t["k"], w.N - 1, w.C, w.g, "bf16")
    for l in range(1, len(ref)):
        got = cache.level(l)[:, :, :ref[l].shape[2]].to(torch.float64).cpu().numpy()
        want = ref[l]
        assert np.isfinite(got).all()
        diff = np.abs(got - want)
        ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
        assert np.all(diff <= ulp), (l, diff.max())
        assert (diff > 0).mean() <= 0.01


def test_decode_continues_a_prefill_built_cache_and_survives_a_capacity_growth():
    w = CASES["gqa4_c64"]
    t = S.make_inputs(w)
    n0 = 1000                                   # tokens seen by the prefill
    small = Cache(w, t, cap=1024, filled=n0)
    # prefill over the capacity layout: completed nodes are right; the partial ones (NaN here, from the
    # unwritten rows) are refreshed by the steps before anything reads them
    P.pisa_build_pyramid(small.p, small.k, small.pyr)
    for pos in range(n0, 1024):
        small.step(pos)
        if pos in (n0, n0 + 1, 1023):
            _check_step(small, t, pos)
    # grow: a larger cache takes over the keys, values and summaries
    big = Cache(w, t, cap=w.N, filled=1024)
    P.pisa_pyramid_regrow(small.p, big.p, small.pyr, big.pyr)
    for pos in range(1024, w.N):
        big.step(pos)
        if pos in (1024, 1025, 1100, w.N - 1):
            _check_step(big, t, pos)


def test_decode_rejects_what_it_does_not_support():
    p = P.Params(1, 1024, 2, 2, 64, 64, 2, 4, dtype="fp32")
    with pytest.raises(P.PisaError, match="unsupported"):
        P.workspace_bytes(p, PB.OP_DECODE)


def test_decode_long_context():
    """A deep hierarchy (2250 leaves, twelve levels, ten of them pruning) continued from a prefill-built cache."""
    w = S.Workload("dec_long_c32", 1, 72000, 2, 1, 64, 32, 2, 4, "bf16", 405, "iid")
    t = S.make_inputs(w)
    n0 = w.N - 40
    cache = Cache(w, t, cap=w.N, filled=n0)
    P.pisa_build_pyramid(cache.p, cache.k, cache.pyr)
    in_band = 0
    for pos in range(n0, w.N):
        cache.step(pos)
        if pos % 4 == 0 or pos == w.N - 1:
            in_band += _check_step(cache, t, pos)
    print(f"[long] rows inside the tie band: {in_band}")


@pytest.mark.parametrize("B,Hkv", [(5, 4), (10, 4), (20, 4)])
def test_decode_large_batches_use_narrower_clusters(B, Hkv):
    """20, 40 and 80 (batch, KV head) units: clusters of four and of two CTAs at one CTA per SM, then of two at
    two per SM; a warp then runs its online softmax across several half blocks (2 K = 40 of them per unit)."""
    w = S.Workload(f"dec_batch{B}", B, 2000, 2 * Hkv, Hkv, 64, 32, 2, 20, "bf16", 406 + B, "iid")
    t = S.make_inputs(w)
    n0 = w.N - 12
    cache = Cache(w, t, cap=w.N, filled=n0)
    P.pisa_build_pyramid(cache.p, cache.k, cache.pyr)
    in_band = 0
    for pos in range(n0, w.N):
        cache.step(pos)
        if pos % 4 == 0 or pos == w.N - 1:
            in_band += _check_step(cache, t, pos)
    print(f"[batch {B}] rows inside the tie band: {in_band}")


@pytest.mark.parametrize("mode", ["mean", "mean_var"])
@pytest.mark.parametrize("name", ["gqa4_c64", "fan4_c32"])
def test_decode_score_modes(name, mode):
    """The mean and mean + variance / 2 scores (Sec. 4.3) in the decoding step, fan-in 2 and 4."""
    w = CASES[name]
    t = S.make_inputs(w)
    n0 = w.N - 48
    cache = Cache(w, t, cap=w.N, filled=n0, score_mode=mode)
    P.pisa_build_pyramid(cache.p, cache.k, cache.pyr)
    in_band = 0
    for pos in range(n0, w.N):
        cache.step(pos)
        if pos % 3 == 0 or pos == w.N - 1:
            in_band += _check_step(cache, t, pos)
    print(f"[{name} {mode}] rows inside the tie band: {in_band}")
