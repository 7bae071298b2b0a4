"""Pins for the oracle's KV append: the written tokens are found where the attention looks for them, nothing
else moves, and "append, then attend" equals attention over a cache that held those tokens all along."""
import numpy as np
import torch

import oracle
from paper_2605_20022_b200 import workload as wl
from test_oracle_attn import gather_kv


def test_append_places_tokens_where_unpaging_finds_them_and_touches_nothing_else():
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("app", shape, [0, 15, 16, 40], [5, 3, 17, 1], [2, 0, 9, 0], seed=21, extra_table_cols=1)
    kv = wl.make_kv(step, poison=None)
    g = torch.Generator().manual_seed(2)
    T = step.total_q_rows
    k_new = torch.randn((T, 2, 32), generator=g).bfloat16(); v_new = torch.randn((T, 2, 32), generator=g).bfloat16()
    out_bits = oracle.kv_append(k_new, v_new, kv, step.page_table, step.prefix_lens, step.q_lens)
    out = torch.from_numpy(out_bits.view(np.int16)).view(torch.bfloat16)
    r0 = 0
    touched = torch.zeros(kv.shape[:1] + kv.shape[3:4], dtype=torch.bool)          # (page, slot)
    for b in range(step.batch):
        n, Lq = int(step.prefix_lens[b]), int(step.q_lens[b])
        K, V = gather_kv(step, out, b)                                              # independent un-paging
        Kold, Vold = gather_kv(step, kv, b)
        assert torch.equal(K[n:n + Lq], k_new[r0:r0 + Lq].double()) and torch.equal(V[n:n + Lq], v_new[r0:r0 + Lq].double())
        assert torch.equal(K[:n], Kold[:n]) and torch.equal(V[:n], Vold[:n])
        for j in range(n, n + Lq):
            touched[int(step.page_table[b, j // 16]), j % 16] = True
        r0 += Lq
    same = (out == kv).all(dim=4).all(dim=2).all(dim=1)                             # (page, slot) unchanged?
    assert same[~touched].all()


def test_append_then_attend_equals_attention_on_the_full_cache():
    shape = wl.Shape(4, 2, 32, 100)
    step = wl.make_step("ata", shape, [33, 7], [9, 12], [4, 6], seed=22)
    q, kv_full = wl.make_q(step), wl.make_kv(step)
    ref = oracle.attn(q, kv_full, step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
    # pull the query block's K/V out of the full cache, scrub them in a copy, append them back
    k_new = torch.zeros((step.total_q_rows, 2, 32), dtype=torch.bfloat16); v_new = torch.zeros_like(k_new)
    kv_hole = kv_full.clone()
    r0 = 0
    for b in range(2):
        for i in range(int(step.q_lens[b])):
            j = int(step.prefix_lens[b]) + i
            pg, sl = int(step.page_table[b, j // 16]), j % 16
            k_new[r0 + i] = kv_full[pg, 0, :, sl]; v_new[r0 + i] = kv_full[pg, 1, :, sl]
            kv_hole[pg, :, :, sl] = float("nan")
        r0 += int(step.q_lens[b])
    bits = oracle.kv_append(k_new, v_new, kv_hole, step.page_table, step.prefix_lens, step.q_lens)
    kv_back = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    got = oracle.attn(q, kv_back, step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
    np.testing.assert_array_equal(got, ref)
