"""The seeded input generator: shapes, ranges and page-table structure of the five workloads."""
import torch

from paper_2605_20022_b200 import workload as wl


def check_tables(step):
    P = step.shape.page_size
    need = (step.kv_lens + P - 1) // P
    used = []
    for b in range(step.batch):
        row = step.page_table[b]
        assert (row[:int(need[b])] >= 0).all() and (row[int(need[b]):] == -1).all()
        used += row[:int(need[b])].tolist()
    assert len(set(used)) == len(used) and max(used) < step.num_pages
    assert step.num_pages == len(used) + 64
    assert sorted(used + step.spare_pages.tolist()) == list(range(step.num_pages))


def test_lengths_of_the_five_workloads():
    s0, s1, s2, s3, s4 = (wl.workload(i) for i in range(5))
    assert (s0.batch, s0.prefix_lens.tolist(), s0.q_lens.tolist(), s0.n_mask.tolist()) == (1, [128], [9], [4])
    assert (s0.shape.n_q_heads, s0.shape.n_kv_heads, s0.shape.head_dim, s0.shape.vocab) == (4, 1, 64, 1000)
    assert (s1.prefix_lens.tolist(), s1.q_lens.tolist(), s1.n_mask.tolist()) == ([2048], [32], [16])
    assert s2.batch == 8 and (s2.n_mask == 16).all()
    assert (s2.prefix_lens >= 512).all() and (s2.prefix_lens <= 8192).all()
    assert (s2.cand_rows >= 4).all() and (s2.cand_rows <= 16).all()
    assert s3.batch == 64 and (s3.n_mask == 0).all() and (s3.q_lens >= 1).all() and (s3.q_lens <= 16).all()
    assert (s3.prefix_lens >= 1024).all() and (s3.prefix_lens <= 4096).all()
    assert s4.batch == 16 and (s4.prefix_lens == 32768).all() and s4.shape.n_layers == 36
    assert s4.attn_bytes() == 16 * 32800 * 4096 + 2 * 16 * 32 * 32 * 128 * 2
    for s in (s0, s1, s2, s3, s4):
        check_tables(s)
        assert s.shape.page_size == 16
    for s in (s1, s2, s3, s4):
        assert (s.shape.n_q_heads, s.shape.n_kv_heads, s.shape.head_dim, s.shape.vocab) == (32, 8, 128, 151936)
    s5 = wl.workload(5)
    assert s5.batch == 8 and (s5.n_blocks == 4).all() and (s5.cand_rows == 4).all() and (s5.n_mask == 28).all()
    check_tables(s5)
    s6 = wl.workload(6)
    assert s6.batch == 64 and (s6.cand_rows == 1).all() and (s6.n_mask == 16).all()
    assert (s6.prefix_lens >= 1024).all() and (s6.prefix_lens <= 4096).all()
    check_tables(s6)
    s7 = wl.workload(7)
    assert s7.batch == 4 and (s7.cand_rows == 17).all() and (s7.n_mask == 272).all() and (s7.n_blocks == 17).all()
    check_tables(s7)
    # same seed -> same lengths
    assert torch.equal(wl.workload(2).prefix_lens, s2.prefix_lens)


def test_tensors_are_seeded_and_poisoned():
    step = wl.workload(0)
    q1, q2 = wl.make_q(step), wl.make_q(step)
    assert torch.equal(q1, q2) and q1.dtype == torch.bfloat16 and tuple(q1.shape) == (9, 4, 64)
    assert not torch.equal(q1, wl.make_q(step, layer=1))
    kv = wl.make_kv(step)
    assert tuple(kv.shape) == (step.num_pages, 2, 1, 16, 64)
    assert (kv[step.spare_pages] == 1e30).all()
    last = int(step.page_table[0, 137 // 16])
    assert (kv[last, :, :, 137 % 16:] == 1e30).all() and (kv[last, :, :, :137 % 16].abs() < 10).all()
    logits, drafts, target = wl.make_logits(step)
    assert tuple(logits.shape) == (5, 1000) and drafts.dtype == torch.int32
    assert (logits[torch.arange(5), target.long()] >= 6).all()
    assert (logits.sum(dim=1) - logits[torch.arange(5), target.long()]).abs().max() < 200


def test_draft_match_rate():
    shape = wl.Shape(4, 2, 32, 64)
    step = wl.make_step("rate", shape, [0] * 4000, [5] * 4000, [0] * 4000, seed=1, p_match=0.75, spare=0)
    _, drafts, target = wl.make_logits(step)
    d, t = drafts.view(4000, 5), target.view(4000, 5)
    rate = (d[:, 1:] == t[:, :-1]).float().mean().item()
    assert abs(rate - 0.75) < 0.02


def test_query_block_kv_reads_the_block_through_the_page_table():
    step = wl.make_step("blk", wl.Shape(8, 2, 64, 100), [0, 15, 33], [5, 17, 1], [2, 16, 0], seed=3)
    kv = wl.make_kv(step)
    k_new, v_new = wl.query_block_kv(step, kv)
    assert k_new.shape == (step.total_q_rows, 2, 64) and v_new.shape == k_new.shape
    row = 0
    for b in range(step.batch):
        for i in range(int(step.q_lens[b])):
            j = int(step.prefix_lens[b]) + i
            page = int(step.page_table[b, j // 16])
            assert torch.equal(k_new[row], kv[page, 0, :, j % 16, :]) and torch.equal(v_new[row], kv[page, 1, :, j % 16, :])
            row += 1
