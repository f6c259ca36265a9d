"""Host logic of pisa_forward_packed's grouping (no GPU): which sequences share a padded batch.  The rules,
from the header: only sequences of 1 .. 8192 tokens are grouped; a group's padded length is the smallest
m * 2^k (m = 8..15; below 16 every length is on the grid) that holds its longest member; every member is at least 3/4 of it; a group holds at
most 32768 padded tokens (at least one sequence); a group of one runs alone."""
import numpy as np
import pytest

import paper_2609_31093_b200 as P


def _grid(n):
    k = 0
    while (15 << k) < n:
        k += 1
    return -(-n // (1 << k)) << k


def _plan(lens, N=None):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64).tolist()
    p = P.Params(1, N or max(max(lens), 1), 8, 2, 128, 64, 2, 4, dtype="bf16")
    return P.packed_plan(p, cu)


def test_rules_hold_on_random_length_mixes():
    rng = np.random.default_rng(5)
    for trial in range(40):
        hi = int(rng.choice([40, 600, 5000, 20000]))
        lens = rng.integers(0, hi + 1, size=int(rng.integers(1, 400))).tolist()
        if max(lens) == 0:
            lens[0] = 3
        group, padded, ng = _plan(lens)
        members = {}
        for i, (gi, n) in enumerate(zip(group, lens)):
            if gi < 0:
                assert padded[i] == n
            else:
                assert 1 <= n <= 8192
                members.setdefault(gi, []).append(i)
        assert sorted(members) == list(range(ng))
        for gi, idxs in members.items():
            assert len(idxs) >= 2
            np_ = padded[idxs[0]]
            assert all(padded[i] == np_ for i in idxs)
            longest = max(lens[i] for i in idxs)
            assert np_ == _grid(longest)                                   # smallest grid length holding the longest member
            assert all(4 * lens[i] >= 3 * np_ for i in idxs)               # nobody is padded by more than a third
            assert len(idxs) <= max(1, 32768 // np_)                       # token cap of a padded batch
        # a sequence runs alone only if the rules leave it no partner in the order the groups are formed:
        # here, at least, never two ungrouped groupable sequences of the same grid length that are both >= 3/4 of it
        alone = [i for i, gi in enumerate(group) if gi < 0 and 1 <= lens[i] <= 8192]
        seen = {}
        for i in alone:
            key = _grid(lens[i])
            if 4 * lens[i] >= 3 * key:
                assert key not in seen or 32768 // key <= 1, (lens[i], lens[seen.get(key, i)])
                seen[key] = i


def test_edge_cases():
    assert _plan([0, 0, 5]) == ([-1, -1, -1], [0, 0, 5], 0)                # empty sequences, a single short one
    group, padded, ng = _plan([512, 512, 512, 9000])
    assert group == [0, 0, 0, -1] and padded[:3] == [512, 512, 512] and ng == 1
    group, padded, ng = _plan([8192] * 9)                                   # four per padded batch of 8192
    assert ng == 2 and sorted(group) == [-1, 0, 0, 0, 0, 1, 1, 1, 1]
    group, padded, ng = _plan([100, 70])                                    # 70 < 3/4 of 104: no group
    assert ng == 0 and group == [-1, -1]
    group, padded, ng = _plan([100, 80])
    assert ng == 1 and padded == [104, 104]


def test_argument_errors():
    p = P.Params(1, 64, 8, 2, 128, 64, 2, 4, dtype="bf16")
    with pytest.raises(Exception):
        P.packed_plan(p, [0, 65])                                           # longer than p.N
    with pytest.raises(Exception):
        P.packed_plan(p, [1, 5])                                            # cu[0] != 0
    with pytest.raises(Exception):
        P.packed_plan(p, [0, 10, 5])                                        # negative length


def test_group_size_is_capped_by_the_kv_head_count():
    """A group's (sequence, KV head) units index a grid dimension: at most 65535 / Hkv sequences per group."""
    lens = [8] * 5000
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64).tolist()
    for Hkv, cap in ((2, 4096), (16, 4095), (32, 2047)):          # 32768 / 8 = 4096 sequences by the token rule
        p = P.Params(1, 8, 2 * Hkv, Hkv, 128, 64, 2, 4, dtype="bf16")
        group, padded, n_groups = P.packed_plan(p, cu)
        sizes = np.bincount(np.asarray(group))
        assert sizes.max() == cap and n_groups == -(-5000 // cap), (Hkv, sizes.max(), n_groups)
        assert set(padded) == {8}
