"""Pins for the CPU oracle's attention: each test checks it against something it
does not itself compute -- a textbook formula through a library routine, an
explicitly built dense mask, a closed form, or an invariant the paper states."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_20022_b200 import workload as wl


def gather_kv(step, kv, b):
    """Un-page sequence b: (K, V) each [kv_len, Hkv, d] float64, via the page table."""
    L = int(step.kv_lens[b])
    P = step.shape.page_size
    pos = torch.arange(L)
    pages = step.page_table[b, pos // P].long()
    K = kv[pages, 0, :, pos % P, :].double()
    V = kv[pages, 1, :, pos % P, :].double()
    return K, V


def dense_mask(n, C, M):
    """[Lq, n+Lq] boolean visibility matrix, one statement per sentence of Sec. 4.1:
    every query token sees the clean prefix; clean (candidate) tokens are causal among
    themselves, as in a standard forward pass; mask tokens see the clean tokens fed in
    this pass; mask tokens see their whole block, both directions; clean tokens never
    see a mask token."""
    Lq = C + M
    vis = np.zeros((Lq, n + Lq), dtype=bool)
    vis[:, :n] = True
    for i in range(C):
        for t in range(C):
            if t <= i:
                vis[i, n + t] = True
    vis[C:, n:n + C] = True
    vis[C:, n + C:] = True
    assert not vis[:C, n + C:].any()
    return vis


def sdpa_reference(step, q, kv):
    """Library attention (float64 scaled_dot_product_attention) with the dense mask."""
    s = step.shape
    G = s.n_q_heads // s.n_kv_heads
    out = torch.zeros((step.total_q_rows, s.n_q_heads, s.head_dim), dtype=torch.float64)
    r0 = 0
    for b in range(step.batch):
        n, Lq, M = int(step.prefix_lens[b]), int(step.q_lens[b]), int(step.n_mask[b])
        if Lq == 0:
            continue
        K, V = gather_kv(step, kv, b)
        K = K.repeat_interleave(G, dim=1).permute(1, 0, 2)   # [Hq, kv_len, d]
        V = V.repeat_interleave(G, dim=1).permute(1, 0, 2)
        Q = q[r0:r0 + Lq].double().permute(1, 0, 2)           # [Hq, Lq, d]
        vis = torch.from_numpy(dense_mask(n, Lq - M, M))
        o = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=vis)
        out[r0:r0 + Lq] = o.permute(1, 0, 2)
        r0 += Lq
    return out.numpy()


def run_oracle(step, q, kv):
    return oracle.attn(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask)


def test_plain_decode_equals_textbook_softmax():
    """n_mask = 0, q_len = 1 is ordinary causal decode attention."""
    shape = wl.Shape(8, 2, 64, 100)
    step = wl.make_step("decode", shape, [37, 1, 160, 0], [1, 1, 1, 1], [0, 0, 0, 0], seed=11)
    q, kv = wl.make_q(step), wl.make_kv(step)
    got = run_oracle(step, q, kv)
    G = shape.n_q_heads // shape.n_kv_heads
    for b in range(step.batch):
        K, V = gather_kv(step, kv, b)
        for h in range(shape.n_q_heads):
            s = (K[:, h // G, :] @ q[b, h].double()) / np.sqrt(shape.head_dim)
            ref = torch.softmax(s, dim=0) @ V[:, h // G, :]
            np.testing.assert_allclose(got[b, h], ref.numpy(), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("C,M", [(c, m) for c, m in itertools.product(range(6), range(6)) if c + m > 0])
def test_dense_mask_bruteforce(C, M):
    """All (C, M) in {0..5}^2 on three ragged sequences against library attention."""
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("tiny", shape, [0, 19, 70 - C - M], [C + M] * 3, [M] * 3, seed=100 + 7 * C + M)
    q, kv = wl.make_q(step), wl.make_kv(step)
    np.testing.assert_allclose(run_oracle(step, q, kv), sdpa_reference(step, q, kv), rtol=1e-11, atol=1e-12)


def test_dense_mask_bruteforce_mixed_lengths_gqa():
    shape = wl.Shape(6, 2, 64, 100)
    step = wl.make_step("mixed", shape, [5, 33, 16], [9, 1, 20], [4, 0, 16], seed=5)
    q, kv = wl.make_q(step), wl.make_kv(step)
    np.testing.assert_allclose(run_oracle(step, q, kv), sdpa_reference(step, q, kv), rtol=1e-11, atol=1e-12)


def test_tiny_workload_matches_library_attention():
    step = wl.workload(0)
    q, kv = wl.make_q(step), wl.make_kv(step)
    np.testing.assert_allclose(run_oracle(step, q, kv), sdpa_reference(step, q, kv), rtol=1e-11, atol=1e-12)


def test_softmax_rows_sum_to_one():
    """With V == 1 everywhere the output is exactly the sum of the softmax weights."""
    step = wl.make_step("ones", wl.Shape(4, 2, 32, 100), [40, 3], [12, 7], [6, 0], seed=3)
    q, kv = wl.make_q(step), wl.make_kv(step, poison=None)
    kv[:, 1] = 1.0
    np.testing.assert_allclose(run_oracle(step, q, kv), 1.0, rtol=0, atol=1e-12)


def test_single_visible_key_returns_its_value():
    """Prefix 0: the bonus row sees only itself, so its output is its own V exactly."""
    step = wl.make_step("self", wl.Shape(4, 2, 32, 100), [0], [5], [2], seed=4, shuffle=False)
    q, kv = wl.make_q(step), wl.make_kv(step)
    got = run_oracle(step, q, kv)
    page = int(step.page_table[0, 0])
    for h in range(4):
        np.testing.assert_array_equal(got[0, h], kv[page, 1, h // 2, 0].double().numpy())


def test_clean_rows_ignore_mask_tokens_and_later_candidates():
    """Candidate rows are the target's own autoregressive computation: bit-identical when
    any mask-token K/V, or the K/V of a later candidate, changes."""
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("inv", shape, [21], [11], [5], seed=8)
    q, kv = wl.make_q(step), wl.make_kv(step)
    base = run_oracle(step, q, kv)
    n, C = 21, 6
    P = shape.page_size

    def slot(j):
        return int(step.page_table[0, j // P]), j % P

    kv2 = kv.clone()
    for j in range(n + C, n + 11):                  # every mask token
        pg, sl = slot(j)
        kv2[pg, :, :, sl, :] = torch.randn_like(kv2[pg, :, :, sl, :].float()).bfloat16() * 3
    got = run_oracle(step, q, kv2)
    np.testing.assert_array_equal(got[:C], base[:C])
    assert np.abs(got[C:] - base[C:]).max() > 1e-3   # mask rows do see their block

    kv3 = kv.clone()
    pg, sl = slot(n + 3)                            # candidate 3
    kv3[pg, :, :, sl, :] = 2.5
    got = run_oracle(step, q, kv3)
    np.testing.assert_array_equal(got[:3], base[:3])
    assert np.abs(got[3:] - base[3:]).max() > 1e-3   # rows 3.. and the mask rows see it


def test_mask_block_is_bidirectional_permutation_equivariant():
    """Reordering the tokens of the mask block reorders the mask rows' outputs and
    changes nothing else."""
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("perm", shape, [18], [10], [6], seed=9)
    q, kv = wl.make_q(step), wl.make_kv(step)
    base = run_oracle(step, q, kv)
    n, C, M, P = 18, 4, 6, shape.page_size
    perm = [3, 0, 5, 1, 4, 2]
    q2, kv2 = q.clone(), kv.clone()
    for u, w in enumerate(perm):                    # new token u = old token perm[u]
        q2[C + u] = q[C + w]
        ju, jw = n + C + u, n + C + w
        kv2[int(step.page_table[0, ju // P]), :, :, ju % P] = kv[int(step.page_table[0, jw // P]), :, :, jw % P]
    got = run_oracle(step, q2, kv2)
    np.testing.assert_allclose(got[:C], base[:C], rtol=0, atol=1e-13)
    np.testing.assert_allclose(got[C:], base[C:][perm], rtol=1e-12, atol=1e-13)


def test_no_mask_equals_causal_prefill_with_prefix():
    """M = 0: ordinary causal attention of a chunk appended to a prefix (library is_causal
    on the full square sequence, last Lq rows)."""
    shape = wl.Shape(2, 2, 32, 100)
    n, Lq = 29, 7
    step = wl.make_step("causal", shape, [n], [Lq], [0], seed=12)
    q, kv = wl.make_q(step), wl.make_kv(step)
    got = run_oracle(step, q, kv)
    K, V = gather_kv(step, kv, 0)
    Qfull = torch.zeros((2, n + Lq, 32), dtype=torch.float64)
    Qfull[:, n:] = q.double().permute(1, 0, 2)
    o = torch.nn.functional.scaled_dot_product_attention(Qfull, K.permute(1, 0, 2), V.permute(1, 0, 2),
                                                         is_causal=True)
    np.testing.assert_allclose(got, o[:, n:].permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)


def test_physical_page_order_and_poison_do_not_matter():
    shape = wl.Shape(4, 1, 32, 100)
    a = wl.make_step("a", shape, [50, 17], [9, 12], [4, 6], seed=21, shuffle=True)
    b = wl.make_step("b", shape, [50, 17], [9, 12], [4, 6], seed=21, shuffle=False)
    q = wl.make_q(a)
    kva = wl.make_kv(a, poison=float("nan"))
    kvb = torch.full_like(wl.make_kv(b, poison=None), 1e30)
    P = shape.page_size
    for s in range(2):
        for j in range(int(a.kv_lens[s])):
            kvb[int(b.page_table[s, j // P]), :, :, j % P] = kva[int(a.page_table[s, j // P]), :, :, j % P]
    ra, rb = run_oracle(a, q, kva), run_oracle(b, q, kvb)
    assert np.isfinite(ra).all()
    np.testing.assert_array_equal(ra, rb)


def test_custom_scale_and_row_entry_point():
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("row", shape, [23, 40], [8, 5], [3, 5], seed=31)
    q, kv = wl.make_q(step), wl.make_kv(step)
    full = run_oracle(step, q, kv)
    for (b, i, h) in [(0, 0, 0), (0, 7, 3), (1, 4, 2), (1, 0, 1)]:
        row = oracle.attn_row(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, b, i, h)
        r = (0 if b == 0 else 8) + i
        np.testing.assert_array_equal(row, full[r, h])
    # scale = 0 makes the softmax uniform over the visible set: output = mean of visible V
    out0 = oracle.attn(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, scale=1e-300)
    K, V = gather_kv(step, kv, 0)
    vis = dense_mask(23, 5, 3)
    for i in range(8):
        ref = V[vis[i], 0, :].mean(dim=0).numpy()
        np.testing.assert_allclose(out0[i, 1], ref, rtol=1e-12, atol=1e-13)
