"""Host logic of the work split (CPU only): fd_plan_ranges_host runs the very routine the plan kernel runs."""
import numpy as np
import pytest

import paper_2605_20022_b200 as fd
from paper_2605_20022_b200 import workload as wl

PIECE_COST, MIN_RANGE, TILE = 5, 2, 128


def tiles_of(pl, ql):
    pl, ql = np.asarray(pl, np.int64), np.asarray(ql, np.int64)
    return np.where(ql > 0, (pl + ql + TILE - 1) // TILE, 0)


def cuts_reference(pl, ql, hkv, n):
    """The split written out segment by segment (no scans, no search): walk the cost axis."""
    nt = tiles_of(pl, ql)
    segs = [(int(t)) for t in nt for _ in range(hkv) if t > 0]            # tiles of every segment, in order
    W = sum(t + PIECE_COST for t in segs)
    total = sum(segs)
    n_use = max(1, min(n, W // (PIECE_COST + MIN_RANGE)))
    out = []
    for c in range(n + 1):
        if c >= n_use or total == 0:
            out.append(total); continue
        x = c * W // n_use
        pos, tile0 = 0, 0
        for t in segs:                                                    # the segment whose span holds x
            if x < pos + t + PIECE_COST:
                out.append(tile0 + max(0, x - pos - PIECE_COST)); break
            pos += t + PIECE_COST; tile0 += t
    return out


def cost_of_range(a, b, seg_starts, seg_tiles):
    """tiles + start-up charge of every segment the range [a, b) touches."""
    cost = b - a
    for s0, t in zip(seg_starts, seg_tiles):
        if max(a, s0) < min(b, s0 + t):
            cost += PIECE_COST
    return cost


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5, 6])
def test_workload_splits(idx):
    step = wl.workload(idx)
    hkv, n = step.shape.n_kv_heads, 148
    got = fd.fd_plan_ranges_host(step.prefix_lens.numpy(), step.q_lens.numpy(), hkv, n)
    assert got == cuts_reference(step.prefix_lens.numpy(), step.q_lens.numpy(), hkv, n)
    nt = tiles_of(step.prefix_lens.numpy(), step.q_lens.numpy())
    total = int(nt.sum()) * hkv
    assert got[0] == 0 and got[-1] == total and all(b >= a for a, b in zip(got, got[1:]))
    seg_tiles = [int(t) for t in nt for _ in range(hkv) if t > 0]
    seg_starts = np.concatenate([[0], np.cumsum(seg_tiles)[:-1]]).tolist()
    costs = [cost_of_range(a, b, seg_starts, seg_tiles) for a, b in zip(got, got[1:]) if b > a]
    W = sum(t + PIECE_COST for t in seg_tiles)
    # equal cost: no range is charged more than its share plus one start-up (a cut inside a segment starts it twice)
    assert max(costs) <= W / len(costs) + 2 * PIECE_COST + 1
    if idx == 1:   # a one-sequence call does not use every CTA: few partials to merge
        assert len(costs) == W // (PIECE_COST + MIN_RANGE) < n
    if idx == 4:   # the long-context call does
        assert len(costs) == n


def test_random_and_degenerate_splits():
    rng = np.random.default_rng(0)
    for _ in range(200):
        B = int(rng.integers(1, 40)); hkv = int(rng.choice([1, 2, 8])); n = int(rng.choice([1, 7, 148, 300]))
        pl = rng.integers(0, 5000, size=B); ql = rng.integers(0, 33, size=B)
        got = fd.fd_plan_ranges_host(pl, ql, hkv, n)
        assert got == cuts_reference(pl, ql, hkv, n), (pl, ql, hkv, n)
    assert fd.fd_plan_ranges_host([100, 7], [0, 0], 8, 4) == [0, 0, 0, 0, 0]          # nothing to do
    assert fd.fd_plan_ranges_host([0], [1], 1, 3) == [0, 1, 1, 1]                     # one tile: one range
    with pytest.raises(fd.FlexDraftError):
        fd.fd_plan_ranges_host([-1], [1], 1, 3)
