"""Pins for the all-hypotheses form of the hybrid mask (several mask blocks, Eq. 2) and for branch selection."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_20022_b200 import workload as wl
from test_oracle_attn import gather_kv


def dense_mask_blocks(n, C, M, nb):
    """[Lq, n+Lq] visibility, one statement per rule: every token sees the clean prefix; clean tokens are
    causal among themselves; the mask tokens form nb blocks of M/nb; the block prepared under the hypothesis
    "r drafts accepted" sees the clean tokens 0..r (the bonus token and the first r drafts); a block sees
    itself in both directions; blocks are mutually invisible; clean tokens never see a mask token."""
    Lq, kb = C + M, M // nb
    vis = np.zeros((Lq, n + Lq), dtype=bool)
    vis[:, :n] = True
    for i in range(C):
        vis[i, n:n + i + 1] = True
    for g in range(nb):
        r = C - nb + g
        rows = slice(C + g * kb, C + (g + 1) * kb)
        vis[rows, n:n + r + 1] = True
        vis[rows, n + C + g * kb:n + C + (g + 1) * kb] = True
    assert not vis[:C, n + C:].any()
    for g, h in itertools.permutations(range(nb), 2):
        assert not vis[C + g * kb:C + (g + 1) * kb, n + C + h * kb:n + C + (h + 1) * kb].any()
    return vis


def sdpa_blocks(step, q, kv, n_blocks):
    s = step.shape
    G = s.n_q_heads // s.n_kv_heads
    out = torch.zeros((step.total_q_rows, s.n_q_heads, s.head_dim), dtype=torch.float64)
    r0 = 0
    for b in range(step.batch):
        n, Lq, M = int(step.prefix_lens[b]), int(step.q_lens[b]), int(step.n_mask[b])
        K, V = gather_kv(step, kv, b)
        K = K.repeat_interleave(G, dim=1).permute(1, 0, 2); V = V.repeat_interleave(G, dim=1).permute(1, 0, 2)
        Q = q[r0:r0 + Lq].double().permute(1, 0, 2)
        vis = torch.from_numpy(dense_mask_blocks(n, Lq - M, M, max(int(n_blocks[b]), 1)))
        out[r0:r0 + Lq] = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=vis).permute(1, 0, 2)
        r0 += Lq
    return out.numpy()


CASES = [  # (prefix_lens, C, M, n_blocks) per sequence
    ([30, 0, 17], [4, 3, 5], [12, 6, 10], [4, 3, 5]),        # all hypotheses: one block per candidate
    ([9, 64], [6, 4], [8, 8], [2, 4]),                       # the last 2 of 6 hypotheses; all 4
    ([20, 20, 20], [5, 5, 1], [6, 6, 4], [1, 0, 1]),         # one block == the plain form
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_blocks_match_dense_mask_library_attention(case):
    pl, C, M, nb = CASES[case]
    step = wl.make_step("blocks", wl.Shape(4, 2, 32, 100), pl, [c + m for c, m in zip(C, M)], M, seed=300 + case)
    q, kv = wl.make_q(step), wl.make_kv(step)
    got = oracle.attn_blocks(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, np.array(nb))
    np.testing.assert_allclose(got, sdpa_blocks(step, q, kv, nb), rtol=1e-11, atol=1e-12)
    if max(nb) <= 1:
        np.testing.assert_array_equal(got, oracle.attn(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask))


def test_blocks_are_isolated_and_conditioned_on_their_hypothesis_only():
    n, C, M, nb = 26, 4, 12, 4
    kb = M // nb
    step = wl.make_step("iso", wl.Shape(4, 2, 32, 100), [n], [C + M], [M], seed=310)
    q, kv = wl.make_q(step), wl.make_kv(step)
    run = lambda kv_: oracle.attn_blocks(q, kv_, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, np.array([nb]))
    base = run(kv)
    P = step.shape.page_size

    def poke(j):
        k2 = kv.clone()
        k2[int(step.page_table[0, j // P]), :, :, j % P] = 1.75
        return run(k2)

    for g in range(nb):                                   # a token of block g changes block g only
        got = poke(n + C + g * kb + 1)
        rows = np.arange(C + g * kb, C + (g + 1) * kb)
        other = np.setdiff1d(np.arange(C + M), rows)
        np.testing.assert_array_equal(got[other], base[other])
        assert np.abs(got[rows] - base[rows]).max() > 1e-3
    for t in range(1, C):                                 # candidate t changes clean rows >= t and blocks with r >= t
        got = poke(n + t)
        for g in range(nb):
            rows = np.arange(C + g * kb, C + (g + 1) * kb)
            r = C - nb + g
            if r >= t:
                assert np.abs(got[rows] - base[rows]).max() > 1e-3
            else:
                np.testing.assert_array_equal(got[rows], base[rows])
        np.testing.assert_array_equal(got[:t], base[:t])


def test_select_branch_picks_the_block_of_the_accepted_length():
    ql = np.array([4 + 12, 6 + 8, 5 + 6, 3 + 0, 2 + 4], np.int32)
    nm = np.array([12, 8, 6, 0, 4], np.int32)
    nb = np.array([4, 2, 1, 0, 2], np.int32)
    tokens = np.arange(100, 100 + int(nm.sum()), dtype=np.int32)
    for acc in ([0, 4, 4, 1, -1], [3, 5, 2, 0, 1], [2, 3, 0, 2, 0]):
        nd, nl = oracle.select_branch(tokens, ql, nm, nb, np.array(acc, np.int32), max_kb=6)
        m0 = 0
        for b in range(5):
            C, M, n_b = int(ql[b] - nm[b]), int(nm[b]), max(int(nb[b]), 1)
            kb = M // n_b if M else 0
            g = acc[b] - (C - n_b)
            if M and acc[b] >= 0 and 0 <= g < n_b:
                assert nl[b] == kb and list(nd[b, :kb]) == list(tokens[m0 + g * kb:m0 + (g + 1) * kb]) and (nd[b, kb:] == -1).all()
            else:
                assert nl[b] == 0 and (nd[b] == -1).all()
            m0 += M
    # all hypotheses prepared: the selected block index is the accepted length itself
    nd, nl = oracle.select_branch(tokens[:12], ql[:1], nm[:1], nb[:1], np.array([2], np.int32), max_kb=3)
    assert list(nd[0]) == [106, 107, 108] and nl[0] == 3
