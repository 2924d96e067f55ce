"""The scan's balanced partition, restated in Python and checked by brute force (no GPU).

The kernel deals the U (problem, 8-page group) units of a launch, in problem order, to the first
Weff = min(W, U) warps: with U = q Weff + rem the first rem warps own q + 1 units, the others q.  A warp writes
one log Z partial per problem it touches, at slot (warp - first warp that touches the problem); the warp that
owns the problem's last unit publishes the count.  The selector reads slots [0, count) of a row that has
`max_groups` slots.  These tests pin the arithmetic those claims rest on; the kernel itself is covered by the
GPU parity tests that force this partition.
"""
import math

import numpy as np
import pytest

B, GROUP = 16, 8


def groups_of(T, k):
    P = -(-T // B)
    return 0 if P <= k else -(-(P - 1) // GROUP)


def ranges(U, W):
    Weff = min(W, U)
    if Weff == 0:
        return []
    q, rem = divmod(U, Weff)
    out = []
    for w in range(Weff):
        lo = w * q + min(w, rem)
        out.append((lo, lo + q + (1 if w < rem else 0)))
    return out


def owner(u, U, W):
    """The kernel's closed form for the warp that owns unit u."""
    Weff = min(W, U)
    q, rem = divmod(U, Weff)
    big = rem * (q + 1)
    return u // (q + 1) if u < big else rem + (u - big) // q


@pytest.mark.parametrize("seed", range(40))
def test_balanced_partition_invariants(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 70))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    k = int(rng.choice([2, 16, 128]))
    W = int(rng.choice([8, 64, 296 * 8]))
    lens = [int(rng.integers(1, 40000)) if rng.random() < 0.8 else int(rng.integers(1, 200)) for _ in range(n)]
    ng = [groups_of(T, k) for T in lens]
    # units in problem order: problem p = b * Hkv + h holds ng[b] consecutive units
    starts, U = [], 0
    for b in range(n):
        for _ in range(Hkv):
            starts.append(U)
            U += ng[b]
    rs = ranges(U, W)
    if U == 0:
        assert rs == []
        return
    # every unit is owned exactly once, ranges are contiguous and differ by at most one unit
    assert rs[0][0] == 0 and rs[-1][1] == U
    assert all(rs[i][1] == rs[i + 1][0] for i in range(len(rs) - 1))
    sizes = [hi - lo for lo, hi in rs]
    assert min(sizes) >= 1 and max(sizes) - min(sizes) <= 1
    for u in rng.integers(0, U, size=50):
        w = owner(int(u), U, W)
        assert rs[w][0] <= u < rs[w][1]
    max_groups = max(1, max(ng))
    for p, s in enumerate(starts):
        g = ng[p // Hkv]
        if g == 0:
            continue
        wf, wl = owner(s, U, W), owner(s + g - 1, U, W)
        touching = [w for w, (lo, hi) in enumerate(rs) if lo < s + g and hi > s]
        assert touching == list(range(wf, wl + 1))            # contiguous: slot = warp - wf has no gaps
        assert len(touching) <= g <= max_groups               # fits the row of max_groups slots
        # every warp after the first enters the problem in mid-range or at its own first unit, never at group 0
        # of the problem unless it owns that unit: only warp wf has slot 0, and the warp that owns the last unit
        # (slot wl - wf) knows the count
        assert all(rs[w][0] > s for w in touching[1:])


def test_partition_suggestion_rule():
    """Iterations of the longest warp: strided = rounds * ceil(max groups / wpp), balanced = ceil(U / W); the
    balanced partition is suggested only when it wins by more than 1/16 plus half an iteration."""
    def suggest(ng, Hkv, W):
        nprob = len(ng) * Hkv
        wpp = max(1, W // nprob)
        nslots = W // wpp
        rounds = -(-nprob // nslots)
        strided = rounds * -(-max(ng) // wpp)
        even = -(-sum(ng) * Hkv // W)
        return strided * 16 > even * 17 + 8
    W = 296 * 8
    assert not suggest([256] * 8, 8, W)                        # equal lengths (8 x 32K tokens)
    assert not suggest([128] * 32, 8, W)                       # equal lengths (32 x 16K tokens)
    assert suggest([990, 520, 700, 810, 600, 930, 560, 1000], 8, W)   # lengths spread over a factor of two
    assert suggest([1125, 19, 25, 15, 23], 2, W)               # one long request among short ones
