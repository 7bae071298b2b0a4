"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Attention within |err| <= 2e-2 + 2e-2 |ref|; accept and commit bit-exact."""
import zlib

import numpy as np
import pytest
import torch

import oracle
import paper_2605_20022_b200 as fd
from paper_2605_20022_b200 import workload as wl
from helpers import Ctx, assert_close, dev, gpu_accept, gpu_attn, gpu_commit, worst_vector_error

pytestmark = pytest.mark.gpu

# the CUDA-core kernel; the tensor-core kernel as a call is routed by default (one cluster per segment, self-planned
# or planned, by size); the tensor-core kernel always on the plan kernel's work list; and always self-planned where legal
PATHS = [fd.FD_ATTN_SIMT, fd.FD_ATTN_AUTO, fd.FD_ATTN_TCGEN05_PLANNED, fd.FD_ATTN_TCGEN05_SELF_PLANNED]


def _one_float_off(t):
    """A device copy of `t` that starts 4 bytes past a 16-byte boundary: the sweeps cannot use their aligned vector loads."""
    buf = torch.empty(t.numel() + 1, dtype=t.dtype, device="cuda")
    v = buf[1:].view(t.shape)
    v.copy_(t)
    assert v.data_ptr() % 16 == 4
    return v


def oracle_attn(step, q, kv):
    return oracle.attn(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("idx", [0, 1, 2, 3, 6])
def test_attention_workloads(idx, path):
    step = wl.workload(idx)
    q, kv = wl.make_q(step), wl.make_kv(step)
    with Ctx(step, path) as ctx:
        # the auto path must be the tensor-core kernel for every benchmark shape
        assert fd.fd_attn_path(ctx.h) == (fd.FD_ATTN_SIMT if path == fd.FD_ATTN_SIMT else fd.FD_ATTN_TCGEN05)
        got, status = gpu_attn(ctx, step, q, kv)
    assert status == 0
    assert_close(got.numpy(), oracle_attn(step, q, kv), step.name)


def _random_step(seed):
    """A seeded random shape and batch: heads, group size, head dimension, ragged prefixes (some empty, some a few
    tiles long), block lengths up to what one 128-row tile holds, any number of mask rows, sometimes several mask blocks."""
    g = torch.Generator().manual_seed(seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))
    G = [1, 2, 4, 8][ri(0, 3)]
    Hkv = [1, 2, 4, 8][ri(0, 3)]
    while G * Hkv > 32:
        Hkv //= 2
    d = [64, 128][ri(0, 1)]
    B = ri(1, 7)
    max_rows = min(32, 128 // G)
    pl, ql, nm, nb = [], [], [], []
    for _ in range(B):
        kind = ri(0, 9)
        pl.append(0 if kind == 0 else ri(1, 40) if kind == 1 else ri(100, 140) if kind == 2 else ri(0, 1500))
        L = 0 if ri(0, 11) == 0 else ri(1, max_rows)
        M = ri(0, L) if L else 0
        C = L - M
        blocks = 1
        if M > 1 and C >= 2 and ri(0, 2) == 0:             # several branches: M = blocks * tokens, at most one per candidate row
            cands = [k for k in range(2, min(M, C) + 1) if M % k == 0]
            if cands:
                blocks = cands[ri(0, len(cands) - 1)]
        ql.append(L); nm.append(M); nb.append(blocks)
    step = wl.make_step(f"fuzz{seed}", wl.Shape(G * Hkv, Hkv, d, 1000), pl, ql, nm, seed=seed, extra_table_cols=ri(0, 2))
    return step, torch.tensor(nb, dtype=torch.int32)


@pytest.mark.parametrize("seed", list(range(40)))
def test_random_shapes_against_the_oracle(seed):
    """Forty seeded random batches through the default routing and through the plan kernel's work list: every output
    element against the oracle, poisoned slots beyond every sequence's length, NaN in the output buffer beforehand."""
    step, n_blocks = _random_step(seed)
    if step.total_q_rows == 0:
        pytest.skip("all blocks empty")
    s = step.shape
    q, kv = wl.make_q(step), wl.make_kv(step)
    ref = oracle.attn_blocks(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, n_blocks)
    for path in (fd.FD_ATTN_AUTO, fd.FD_ATTN_TCGEN05_PLANNED):
        with Ctx(step, path) as ctx:
            out = torch.full((step.total_q_rows, s.n_q_heads, s.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
            fd.fd_attn_draft_verify_blocks(ctx.h, step.batch, step.total_q_rows, q.cuda(), kv.cuda(), step.num_pages, step.page_table.cuda(),
                                           step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda(), n_blocks.cuda(), out)
            assert fd.fd_last_device_status(ctx.h) == 0
            assert_close(out.float().cpu().numpy(), ref, f"{step.name} path {path}")


def test_tensor_core_call_routing():
    """Which form of the tensor-core kernel a call takes: few segments -> one cluster per segment; few sequences ->
    self-planned; otherwise (or under a pinned plan) the plan kernel's work list.  All forms agree with the oracle."""
    want = {1: fd.FD_TC_CLUSTER, 2: fd.FD_TC_SELF_PLANNED, 3: fd.FD_TC_PLANNED}
    for idx, mode in want.items():
        step = wl.workload(idx)
        q, kv = wl.make_q(step), wl.make_kv(step)
        ref = oracle_attn(step, q, kv)
        for path, expect in ((fd.FD_ATTN_AUTO, mode), (fd.FD_ATTN_TCGEN05_PLANNED, fd.FD_TC_PLANNED),
                             (fd.FD_ATTN_TCGEN05_SELF_PLANNED, fd.FD_TC_SELF_PLANNED if step.batch <= 24 else fd.FD_TC_PLANNED)):
            with Ctx(step, path) as ctx:
                assert fd.fd_attn_last_mode(ctx.h) == -1
                before = fd.fd_launch_count(ctx.h)
                got, status = gpu_attn(ctx, step, q, kv)
                assert status == 0 and fd.fd_attn_last_mode(ctx.h) == expect, (idx, path, fd.fd_attn_last_mode(ctx.h))
                assert fd.fd_launch_count(ctx.h) - before == (2 if expect == fd.FD_TC_PLANNED else 1)   # one launch unless planned
                assert_close(got.numpy(), ref, f"{step.name} path {path}")


EDGE = {
    # name: (Hq, Hkv, d, prefix_lens, q_lens, n_mask)
    "prefix0_and_single_row": (8, 2, 128, [0, 0, 1, 15], [1, 9, 1, 1], [0, 4, 0, 1]),
    "page_boundaries": (8, 2, 128, [16, 15, 17, 112, 127, 128, 129, 240], [16, 17, 15, 16, 1, 32, 31, 32],
                        [0, 1, 15, 16, 0, 16, 16, 16]),
    "mask_only_and_one_candidate": (8, 2, 128, [300, 77, 5], [16, 17, 4], [16, 16, 4]),
    "all_mask_counts": (4, 1, 128, [100 + 3 * m for m in range(17)], [16 + m for m in range(17)], list(range(17))),
    "empty_sequences_inside_batch": (8, 2, 128, [40, 90, 0, 260], [0, 5, 0, 32], [0, 2, 0, 16]),
    "head_dim64_gqa8": (16, 2, 64, [200, 31, 1000], [16, 3, 9], [8, 0, 4]),
    "mha_group1": (4, 4, 64, [130, 257], [32, 20], [16, 4]),
    "one_long_sequence_many_splits": (4, 1, 128, [20000], [32], [16]),
    "ragged_mix": (32, 8, 128, [5000, 13, 700, 2047, 2049, 129], [32, 1, 20, 9, 32, 16], [16, 0, 16, 0, 16, 8]),
    # many short segments per CTA range: every piece boundary, single-tile pieces, 1..3 active softmax warps
    "many_tiny_sequences": (32, 8, 128, [(7 * b) % 41 for b in range(150)], [1 + (5 * b) % 24 for b in range(150)],
                            [min(1 + (5 * b) % 24, (3 * b) % 17) for b in range(150)]),
    # one CTA range holds the tail of a long segment, whole short ones and the head of another long one
    "long_short_long": (32, 8, 128, [9000, 100, 37, 260, 12000, 5], [32, 4, 17, 32, 32, 9], [16, 0, 1, 16, 16, 0]),
    # group sizes that are not powers of two: the Q load boxes are 2, 1 and 1 block rows high
    "gqa3_up_to_32_rows": (6, 2, 128, [300, 1, 2500], [32, 31, 7], [16, 3, 0]),
    "gqa5_up_to_25_rows": (5, 1, 64, [700, 64], [25, 24], [9, 24]),
    "gqa6_up_to_21_rows": (12, 2, 128, [129, 4000, 0], [21, 20, 2], [5, 0, 1]),
    # a call small enough to leave most CTAs without a range, and one that fills exactly one tile
    "few_ranges": (8, 2, 128, [100, 40], [8, 3], [4, 0]),
    "exactly_one_tile": (4, 1, 128, [120], [8], [2]),
    # more row blocks than the plan kernel keeps in shared memory (its range search then probes global memory)
    "batch_1500": (8, 2, 128, [(11 * b) % 37 for b in range(1500)], [1 + b % 3 for b in range(1500)], [b % 2 for b in range(1500)]),
}


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name", sorted(EDGE))
def test_attention_edge_cases(name, path):
    Hq, Hkv, d, pl, ql, nm = EDGE[name]
    step = wl.make_step(name, wl.Shape(Hq, Hkv, d, 1000), pl, ql, nm, seed=zlib.crc32(name.encode()) % 10000, extra_table_cols=2)
    q, kv = wl.make_q(step), wl.make_kv(step, poison=float("nan"))     # NaN in every slot no token owns
    with Ctx(step, path, max_batch=len(pl)) as ctx:
        got, status = gpu_attn(ctx, step, q, kv)
        again, _ = gpu_attn(ctx, step, q, kv)
    assert status == 0
    assert_close(got.numpy(), oracle_attn(step, q, kv), name)
    assert torch.equal(got, again), "two runs on the same inputs differ bitwise"


@pytest.mark.parametrize("path", PATHS)
def test_attention_custom_scale_and_empty_batch(path):
    step = wl.make_step("scale", wl.Shape(8, 2, 128, 1000), [333, 40], [12, 32], [4, 16], seed=5)
    q, kv = wl.make_q(step), wl.make_kv(step)
    with Ctx(step, path, scale=0.05) as ctx:
        got, status = gpu_attn(ctx, step, q, kv)
        assert status == 0
        ref = oracle.attn(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, scale=0.05)
        assert_close(got.numpy(), ref, "scale")
        empty = torch.zeros((0,), dtype=torch.int32)
        code = fd.fd_attn_draft_verify(ctx.h, 0, 0, None, None, 0, None, None, None, None, None)
        assert code == fd.FD_OK and fd.fd_last_device_status(ctx.h) == 0


@pytest.mark.parametrize("path", PATHS)
def test_attention_device_detected_errors(path):
    step = wl.make_step("err", wl.Shape(8, 2, 128, 1000), [100, 200, 50], [8, 8, 8], [4, 4, 4], seed=6)
    q, kv = wl.make_q(step), wl.make_kv(step)
    ref = oracle_attn(step, q, kv)
    with Ctx(step, path) as ctx:
        bad = step.page_table.clone()
        bad[1, 3] = step.num_pages + 5                      # a page id outside the pool
        got, status = gpu_attn(ctx, step, q, kv, page_table=bad)
        assert status == fd.FD_DEV_BAD_PAGE
        assert_close(got[:8].numpy(), ref[:8], "seq0"); assert_close(got[16:].numpy(), ref[16:], "seq2")
        assert (got[8:16] == 0).all()
        for lens in [(step.prefix_lens, torch.tensor([8, 9, 8], dtype=torch.int32), step.n_mask),   # rows != T
                     (step.prefix_lens, step.q_lens, torch.tensor([4, 9, 4], dtype=torch.int32)),   # n_mask > q_len
                     (torch.tensor([100, -1, 50], dtype=torch.int32), step.q_lens, step.n_mask),
                     (torch.tensor([100, 10 ** 6, 50], dtype=torch.int32), step.q_lens, step.n_mask)]:
            got, status = gpu_attn(ctx, step, q, kv, lens=lens)
            assert status == fd.FD_DEV_BAD_LENGTHS and (got == 0).all()
        got, status = gpu_attn(ctx, step, q, kv)             # the context still works
        assert status == 0
        assert_close(got.numpy(), ref, "after errors")


def test_host_detected_errors_launch_nothing():
    step = wl.workload(0)
    with Ctx(step) as ctx:
        q = torch.zeros((9, 4, 64), dtype=torch.bfloat16, device="cuda")
        before = fd.fd_launch_count(ctx.h)
        assert fd.fd_attn_draft_verify(ctx.h, 1, 9, None, q, 4, q, q, q, q, q, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        assert fd.fd_attn_draft_verify(ctx.h, 2, 9, q, q, 4, q, q, q, q, q, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        assert fd.fd_verify_accept(ctx.h, 1, 5, None, q, q, q, q, q, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        assert fd.fd_kv_commit(ctx.h, 1, q, q, q, q, q, None, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        assert fd.fd_launch_count(ctx.h) == before
    with pytest.raises(fd.FlexDraftError):
        fd.fd_create(32, 8, 96, 1000, 1, 32, 8)             # head_dim 96
    with pytest.raises(fd.FlexDraftError):
        fd.fd_create(32, 8, 128, 1000, 1, 4097, 8)          # max_q_len beyond the supported 4096


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_accept_and_commit_workloads(idx):
    step = wl.workload(idx)
    logits, drafts, target = wl.make_logits(step)
    exp_acc, exp_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    with Ctx(step) as ctx:
        acc, bon, status = gpu_accept(ctx, step, logits, drafts)
        assert status == 0
        np.testing.assert_array_equal(acc, exp_acc)
        np.testing.assert_array_equal(bon, exp_bon)
        acc2, bon2, _ = gpu_accept(ctx, step, logits, drafts)      # scratch keys were re-zeroed
        np.testing.assert_array_equal(acc2, exp_acc); np.testing.assert_array_equal(bon2, exp_bon)
        pt, pl, freed, status = gpu_commit(ctx, step, acc)
        assert status == 0
    ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, exp_acc)
    np.testing.assert_array_equal(pt, ept)
    np.testing.assert_array_equal(pl, epl)
    np.testing.assert_array_equal(freed, efreed)


@pytest.mark.parametrize("V", [1, 3, 17, 1000, 4095, 4096, 4097, 8191, 8193, 151937, 200003])
def test_accept_vocab_sizes_ties_and_alignment(V):
    g = torch.Generator().manual_seed(V)
    ql = [1, 4, 16, 2, 7, 0, 16]
    nm = [0, 0, 0, 1, 3, 0, 16]
    step = wl.make_step("acc", wl.Shape(4, 2, 64, V), [5] * len(ql), ql, nm, seed=V, p_match=0.85)
    logits, drafts, _ = wl.make_logits(step)
    logits = torch.round(logits * 2) / 2                       # coarse grid: many exact ties, planted peak kept
    R = logits.shape[0]
    logits[0] = 0.25                                           # a flat row -> index 0
    if V > 2:
        logits[1, V - 1] = 9.0; logits[1, V // 2] = 9.0        # two-way tie for the maximum
        logits[2, :] = -float("inf"); logits[2, V - 2] = -3e38
        logits[3, 1] = float("inf"); logits[3, V - 1] = float("inf")
        logits[4, 0] = -0.0; logits[4, 1:] = -1.0; logits[4, V - 1] = 0.0   # -0.0 ties with +0.0
    exp_acc, exp_bon, exp_am = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    drafts2 = drafts.clone()                                   # make the drafts agree with the tied rows too
    r0 = 0
    for b, C in enumerate(step.cand_rows.tolist()):
        for j in range(C - 1):
            if (r0 + j) % 3 != 2:
                drafts2[r0 + j + 1] = int(exp_am[r0 + j])
        r0 += C
    with Ctx(step) as ctx:
        for d_ in (drafts, drafts2):
            e_acc, e_bon, _ = oracle.accept(logits, d_, step.q_lens, step.n_mask)
            acc, bon, status = gpu_accept(ctx, step, logits, d_)
            assert status == 0
            np.testing.assert_array_equal(acc, e_acc)
            np.testing.assert_array_equal(bon, e_bon)


@pytest.mark.parametrize("V,B", [(20004, 48), (8192, 96), (12292, 48)])
def test_accept_many_rows_ties_ragged_chunks_and_alignment(V, B):
    """Several hundred rows: last chunk of a row ragged (V % 4096 != 0) or full, ties across chunk boundaries, flat /
    -inf / +inf rows; the same logits one float off a 16-byte boundary (scalar head and tail around the vector loads)
    must give the same answer."""
    g = torch.Generator().manual_seed(V)
    ql = torch.randint(12, 17, (B,), generator=g).tolist()
    nm = [0] * B
    step = wl.make_step("acc", wl.Shape(4, 2, 64, V), [5] * B, ql, nm, seed=V, p_match=0.9)
    logits, drafts, _ = wl.make_logits(step)
    logits = torch.round(logits * 2) / 2                       # coarse grid: many exact ties, planted peak kept
    R = logits.shape[0]
    logits[0] = 0.25                                           # flat row -> index 0
    logits[1, V - 1] = 9.0; logits[1, 4096] = 9.0; logits[1, 4095] = 9.0   # tie across a chunk boundary -> 4095
    logits[2, :] = -float("inf"); logits[2, V - 2] = -3e38
    logits[3, 5000] = float("inf"); logits[3, V - 1] = float("inf")
    logits[4, :] = -float("inf")                               # nothing finite -> index 0
    logits[5, 0] = -0.0; logits[5, 1:] = -1.0; logits[5, V - 1] = 0.0      # -0.0 ties with +0.0
    logits[R - 1] = 1.5; logits[R - 1, V - 1] = 2.0            # the last chunk of the last row decides
    exp_acc, exp_bon, exp_am = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    assert exp_am[1] == 4095 and exp_am[4] == 0 and exp_am[R - 1] == V - 1
    with Ctx(step) as ctx:
        for _ in range(2):                                     # second call: keys and ticket were re-zeroed
            acc, bon, status = gpu_accept(ctx, step, logits, drafts)
            assert status == 0
            np.testing.assert_array_equal(acc, exp_acc); np.testing.assert_array_equal(bon, exp_bon)
        off = _one_float_off(logits)
        acc_t = torch.full((B,), -99, dtype=torch.int32, device="cuda"); bon_t = torch.full_like(acc_t, -99)
        fd.fd_verify_accept(ctx.h, B, R, off, dev(drafts), dev(step.q_lens), dev(step.n_mask), acc_t, bon_t)
        assert fd.fd_last_device_status(ctx.h) == 0
        np.testing.assert_array_equal(acc_t.cpu().numpy(), exp_acc); np.testing.assert_array_equal(bon_t.cpu().numpy(), exp_bon)


@pytest.mark.parametrize("seed", list(range(30)))
def test_accept_then_commit_random_batches(seed):
    """Thirty seeded random batches: vocabulary of any size (aligned or not, below and above one chunk), any mix of
    candidate and mask rows, sequences without candidates, coarse logits (ties); accept and the commit that follows
    it, bit-exact against the oracle, twice in a row on the same context."""
    g = torch.Generator().manual_seed(1000 + seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))
    V = [ri(1, 40), ri(41, 4096), ri(4097, 9000), 4096, 8192][seed % 5]
    B = ri(1, 40)
    ql, nm, pl = [], [], []
    for _ in range(B):
        L = 0 if ri(0, 9) == 0 else ri(1, 32)
        M = ri(0, L) if ri(0, 3) else 0
        ql.append(L); nm.append(M); pl.append(ri(0, 300))
    step = wl.make_step(f"ac{seed}", wl.Shape(4, 2, 64, V), pl, ql, nm, seed=2000 + seed, p_match=[0.5, 0.8, 0.95][seed % 3],
                        extra_table_cols=ri(0, 2))
    logits, drafts, _ = wl.make_logits(step)
    if seed % 2:
        logits = torch.round(logits * 2) / 2
    exp_acc, exp_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, exp_acc)
    with Ctx(step) as ctx:
        for _ in range(2):
            acc, bon, status = gpu_accept(ctx, step, logits, drafts)
            assert status == 0
            np.testing.assert_array_equal(acc, exp_acc); np.testing.assert_array_equal(bon, exp_bon)
            pt, pl2, freed, status = gpu_commit(ctx, step, acc)
            assert status == 0
            np.testing.assert_array_equal(pt, ept); np.testing.assert_array_equal(pl2, epl); np.testing.assert_array_equal(freed, efreed)


def test_sweeps_right_behind_an_attention_call():
    """With fd_calls_back_to_back on, a sweep launched right behind an attention call starts under that call's tail
    and writes its results after it: the greedy accept, the sampling accept and the draft tail must give exactly what
    they give on their own."""
    step = wl.workload(2)
    s = step.shape
    B, T, R, Rm = step.batch, step.total_q_rows, step.total_cand_rows, int(step.n_mask.sum())
    g = torch.Generator().manual_seed(31)
    q, kv = wl.make_q(step).cuda(), wl.make_kv(step).cuda()
    logits, drafts, _ = wl.make_logits(step)
    dlg = (logits + 0.5 * torch.randn(logits.shape, generator=g)).cuda()
    ua, ub = torch.rand((R,), generator=g).cuda(), torch.rand((B,), generator=g).cuda()
    ml, mb = torch.randn((Rm, s.vocab), generator=g).cuda(), torch.randn((Rm, s.vocab), generator=g).cuda()
    logits, drafts = logits.cuda(), drafts.cuda()
    with Ctx(step) as ctx:
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        out = torch.empty_like(q)
        attend = lambda: fd.fd_attn_draft_verify(ctx.h, B, T, q, kv, step.num_pages, dpt, dpl, dql, dnm, out)
        def accept():
            a = torch.full((B,), -9, dtype=torch.int32, device="cuda"); b = torch.full_like(a, -9)
            fd.fd_verify_accept(ctx.h, B, R, logits, drafts, dql, dnm, a, b)
            return a, b
        def sample():
            a = torch.full((B,), -9, dtype=torch.int32, device="cuda"); b = torch.full_like(a, -9)
            fd.fd_verify_accept_sample(ctx.h, B, R, logits, dlg, drafts, dql, dnm, 0.8, ua, ub, a, b)
            return a, b
        def tail():
            tok = torch.full((Rm,), -9, dtype=torch.int32, device="cuda"); pr = torch.zeros((Rm,), device="cuda")
            keep = torch.full((B, 1), -9, dtype=torch.int32, device="cuda")
            fd.fd_draft_select(ctx.h, B, Rm, 1, ml, mb, dnm, None, 0.3, tok, pr, keep)
            return tok, pr.view(torch.int32), keep
        alone = [f() for f in (accept, sample, tail)]
        torch.cuda.synchronize()
        fd.fd_calls_back_to_back(ctx.h, True)
        for rep in range(3):
            behind = []
            for f in (accept, sample, tail):
                attend()
                behind.append(f())
            torch.cuda.synchronize()
            assert fd.fd_last_device_status(ctx.h) == 0
            for x, y in zip(alone, behind):
                assert all(torch.equal(u, v) for u, v in zip(x, y))
        e_acc, e_bon, _ = oracle.accept(logits.cpu(), drafts.cpu(), step.q_lens, step.n_mask)
        np.testing.assert_array_equal(alone[0][0].cpu().numpy(), e_acc); np.testing.assert_array_equal(alone[0][1].cpu().numpy(), e_bon)


def test_accept_bad_lengths_and_no_candidates():
    step = wl.make_step("acc", wl.Shape(4, 2, 64, 500), [5, 5], [4, 16], [0, 16], seed=3)
    logits, drafts, _ = wl.make_logits(step)
    with Ctx(step) as ctx:
        acc, bon, status = gpu_accept(ctx, step, logits, drafts,
                                      lens=(torch.tensor([5, 16], dtype=torch.int32), step.n_mask))
        assert status == fd.FD_DEV_BAD_LENGTHS and (acc == -1).all() and (bon == -1).all()
        acc, bon, status = gpu_accept(ctx, step, logits, drafts)
        e_acc, e_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
        assert status == 0
        np.testing.assert_array_equal(acc, e_acc); np.testing.assert_array_equal(bon, e_bon)
        none = wl.make_step("none", wl.Shape(4, 2, 64, 500), [5, 5], [16, 16], [16, 16], seed=3)
        lg, dr, _ = wl.make_logits(none)
        acc, bon, status = gpu_accept(ctx, none, lg, dr)
        assert status == 0 and (acc == -1).all() and (bon == -1).all()


def test_commit_random_and_degenerate():
    g = torch.Generator().manual_seed(9)
    B = 1300                                                     # several 256-sequence chunks of the in-kernel scan
    n = torch.randint(0, 400, (B,), generator=g)
    C = torch.randint(0, 17, (B,), generator=g)
    M = torch.randint(0, 2, (B,), generator=g) * 16
    step = wl.make_step("commit", wl.Shape(4, 2, 64, 100), n.tolist(), (C + M).tolist(), M.tolist(), seed=10,
                        extra_table_cols=2)
    acc = np.array([int(torch.randint(0, int(c), (1,), generator=g)) if c > 0 else -1 for c in C], np.int32)
    with Ctx(step) as ctx:
        pt, pl, freed, status = gpu_commit(ctx, step, acc)
        assert status == 0
        ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, acc)
        np.testing.assert_array_equal(pt, ept); np.testing.assert_array_equal(pl, epl)
        np.testing.assert_array_equal(freed, efreed)
        bad = acc.copy()
        k = int(np.argmax(acc >= 0))
        bad[k] = int(step.q_lens[k])                            # accepted_len >= q_len: left unchanged, flagged
        pt, pl, freed, status = gpu_commit(ctx, step, bad)
        assert status == fd.FD_DEV_BAD_ACCEPT
        skip = acc.copy(); skip[k] = -1
        ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, skip)
        np.testing.assert_array_equal(pt, ept); np.testing.assert_array_equal(pl, epl)
        np.testing.assert_array_equal(freed, efreed)


_LONG_REF = {}   # layer -> oracle output of the whole layer, computed once and shared by both attention paths


def _long_context_reference(step, layer):
    if layer not in _LONG_REF:
        q, kv = wl.make_q(step, layer, device="cuda").cpu(), wl.make_kv(step, layer, device="cuda").cpu()
        _LONG_REF[layer] = oracle_attn(step, q, kv)
    return _LONG_REF[layer]


@pytest.mark.parametrize("path", PATHS)
def test_long_context_full_size_every_element(path):
    """Workload 5 at its full per-layer size (16 x 32 800 tokens, 2.15 GB of KV per layer, two layers with
    distinct pools), in the launch configuration the benchmark times (one pinned work list for all layers).
    Every output element of both layers is compared with the oracle.  At this length an output element is an
    average over 32 800 values and has a standard deviation near 0.009, so beside the elementwise bound every
    (row, head) vector must also agree to 2 % of its own length -- a lost tile or a wrong split weight shows there."""
    step = wl.workload(4, n_layers=2)
    dpt, dpl, dql, dnm = (t.cuda() for t in (step.page_table, step.prefix_lens, step.q_lens, step.n_mask))
    with Ctx(step, path) as ctx:
        # as the benchmark does for a multi-layer step: one work list, pinned, for every layer
        fd.fd_plan_pin(ctx.h, step.batch, step.total_q_rows, dpl, dql, dnm)
        for layer in range(2):
            q = wl.make_q(step, layer, device="cuda")
            kv = wl.make_kv(step, layer, device="cuda")
            out = torch.empty_like(q)
            fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, q, kv, step.num_pages, dpt, dpl, dql, dnm, out)
            assert fd.fd_last_device_status(ctx.h) == 0
            if layer == 0:          # 222 tiles per CTA, every split merged: the result must not depend on timing
                for _ in range(3):
                    again = torch.empty_like(q)
                    fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, q, kv, step.num_pages, dpt, dpl, dql, dnm, again)
                    assert torch.equal(out, again), "two runs on the same inputs differ bitwise"
                # without the pin the tensor-core kernel cuts the same ranges for itself (16 sequences): same bits
                fd.fd_plan_unpin(ctx.h)
                again.fill_(0)
                fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, q, kv, step.num_pages, dpt, dpl, dql, dnm, again)
                if path in (fd.FD_ATTN_AUTO, fd.FD_ATTN_TCGEN05_SELF_PLANNED):
                    assert fd.fd_attn_last_mode(ctx.h) == fd.FD_TC_SELF_PLANNED
                assert torch.equal(out, again), "planned and self-planned calls differ bitwise"
                fd.fd_plan_pin(ctx.h, step.batch, step.total_q_rows, dpl, dql, dnm)
                del again
            outc = out.float().cpu().numpy()
            del q, kv, out
            assert np.isfinite(outc).all()
            ref = _long_context_reference(step, layer)
            assert_close(outc, ref, f"layer {layer}")
            worst = worst_vector_error(outc, ref)
            assert worst <= 2e-2, f"layer {layer}: worst (row, head) vector off by {worst:.3e} of its length"


@pytest.mark.parametrize("append", [False, True])
def test_device_buffer_step_in_one_call(append):
    """fd_step_device: a 4-layer step -- (append,) attention per layer on one work list, accept, commit -- launched by
    one C call, against the oracle; twice on the same context."""
    shape = wl.Shape(32, 8, 128, 5000, n_layers=4)
    step = wl.make_step("dev", shape, [700, 130, 2049, 0, 31], [32, 9, 20, 16, 1], [16, 0, 8, 0, 0], seed=19, p_match=0.7, extra_table_cols=1)
    L, B, T, R = 4, step.batch, step.total_q_rows, step.total_cand_rows
    g = torch.Generator().manual_seed(23)
    qs = [wl.make_q(step, l) for l in range(L)]
    kvs = [wl.make_kv(step, l) for l in range(L)]
    kn = [torch.randn((T, 8, 128), generator=g).bfloat16() for _ in range(L)]
    vn = [torch.randn((T, 8, 128), generator=g).bfloat16() for _ in range(L)]
    logits, drafts, _ = wl.make_logits(step)
    refs, pools_ref = [], []
    for l in range(L):
        kv_l = kvs[l]
        if append:
            bits = oracle.kv_append(kn[l], vn[l], kvs[l], step.page_table, step.prefix_lens, step.q_lens)
            kv_l = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
            pools_ref.append(bits)
        refs.append(oracle.attn(qs[l], kv_l, step.page_table, step.prefix_lens, step.q_lens, step.n_mask))
    e_acc, e_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, e_acc)
    with Ctx(step) as ctx:
        dq = [t.cuda() for t in qs]; dk = [t.cuda() for t in kn]; dv = [t.cuda() for t in vn]
        pools = [t.cuda() for t in kvs]
        outs = [torch.full((T, 32, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
        dpt, dpl = step.page_table.cuda(), step.prefix_lens.cuda()
        dql, dnm = step.q_lens.cuda(), step.n_mask.cuda()
        acc = torch.full((B,), -9, dtype=torch.int32, device="cuda"); bon = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        freed = torch.full((B * 3,), -7, dtype=torch.int32, device="cuda"); nfr = torch.zeros(1, dtype=torch.int32, device="cuda")
        before = fd.fd_launch_count(ctx.h)
        fd.fd_step_device(ctx.h, B, T, R, dq, dk if append else None, dv if append else None, pools, outs, step.num_pages, dpt, dpl, dql, dnm,
                          None, logits.cuda(), drafts.cuda(), acc, bon, freed, nfr)
        assert fd.fd_last_device_status(ctx.h) == 0
        assert fd.fd_launch_count(ctx.h) - before == 1 + L * (2 if append else 1) + 2      # plan, (append,) attention per layer, accept, commit
        for l in range(L):
            assert_close(outs[l].float().cpu().numpy(), refs[l], f"layer {l}")
            if append:
                np.testing.assert_array_equal(pools[l].cpu().view(torch.int16).numpy().view(np.uint16), pools_ref[l])
        np.testing.assert_array_equal(acc.cpu().numpy(), e_acc); np.testing.assert_array_equal(bon.cpu().numpy(), e_bon)
        np.testing.assert_array_equal(dpt.cpu().numpy(), ept); np.testing.assert_array_equal(dpl.cpu().numpy(), epl)
        n = int(nfr.item())
        np.testing.assert_array_equal(freed[:n].cpu().numpy(), efreed)
        # the same step again on restored tables: same bits (plan pinned and dropped inside the call both times)
        dpt2, dpl2 = step.page_table.cuda(), step.prefix_lens.cuda()
        outs2 = [torch.empty_like(o) for o in outs]
        fd.fd_step_device(ctx.h, B, T, R, dq, dk if append else None, dv if append else None, pools, outs2, step.num_pages, dpt2, dpl2, dql,
                          dnm, None, logits.cuda(), drafts.cuda(), acc, bon, freed, nfr)
        assert fd.fd_last_device_status(ctx.h) == 0
        assert all(torch.equal(a, b) for a, b in zip(outs, outs2))
        np.testing.assert_array_equal(dpt2.cpu().numpy(), ept); np.testing.assert_array_equal(acc.cpu().numpy(), e_acc)


def test_host_buffer_step_matches_oracle():
    """fd_step_host: a whole 3-layer step from pinned host buffers (copies pipelined inside the library)."""
    shape = wl.Shape(32, 8, 128, 5000, n_layers=3)
    step = wl.make_step("host", shape, [700, 130, 2049, 0], [32, 9, 20, 16], [16, 0, 8, 0], seed=17, p_match=0.7,
                        extra_table_cols=1)
    L, B, T, R = 3, step.batch, step.total_q_rows, step.total_cand_rows
    qs = [wl.make_q(step, l) for l in range(L)]
    kvs = [wl.make_kv(step, l) for l in range(L)]
    logits, drafts, _ = wl.make_logits(step)
    pin = lambda t: t.contiguous().pin_memory()
    q_host = pin(torch.stack(qs)); out_host = pin(torch.zeros_like(q_host))
    h_logits, h_drafts = pin(logits), pin(drafts)
    h_pt, h_pl, h_ql, h_nm = pin(step.page_table.clone()), pin(step.prefix_lens.clone()), pin(step.q_lens), pin(step.n_mask)
    h_acc, h_bon = pin(torch.zeros(B, dtype=torch.int32)), pin(torch.zeros(B, dtype=torch.int32))
    h_freed, h_nf = pin(torch.full((B * 3,), -7, dtype=torch.int32)), pin(torch.zeros(1, dtype=torch.int32))
    dkv = [t.cuda() for t in kvs]
    with Ctx(step) as ctx:
        assert fd.fd_step_host(ctx.h, B, T, R, dkv, step.num_pages, q_host, out_host, h_logits, h_drafts, h_pt, h_pl, h_ql,
                               h_nm, h_acc, h_bon, h_freed, h_nf, raise_on_error=False) == fd.FD_ERR_INVALID_ARG  # not reserved
        fd.fd_host_reserve(ctx.h, T, R)
        for _ in range(2):                                   # twice: the second step reuses the staging buffers
            h_pt.copy_(step.page_table); h_pl.copy_(step.prefix_lens); out_host.zero_()
            fd.fd_step_host(ctx.h, B, T, R, dkv, step.num_pages, q_host, out_host, h_logits, h_drafts, h_pt, h_pl, h_ql,
                            h_nm, h_acc, h_bon, h_freed, h_nf)
            torch.cuda.current_stream().synchronize()
            assert fd.fd_last_device_status(ctx.h) == 0
            for l in range(L):
                ref = oracle.attn(qs[l], kvs[l], step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
                assert_close(out_host[l].float().numpy(), ref, f"layer {l}")
            e_acc, e_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
            np.testing.assert_array_equal(h_acc.numpy(), e_acc); np.testing.assert_array_equal(h_bon.numpy(), e_bon)
            ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, e_acc)
            np.testing.assert_array_equal(h_pt.numpy(), ept); np.testing.assert_array_equal(h_pl.numpy(), epl)
            assert int(h_nf) == len(efreed)
            np.testing.assert_array_equal(h_freed.numpy()[:len(efreed)], efreed)


def test_host_buffer_step_with_the_kv_append_inside():
    """fd_step_host_append: the caches start WITHOUT the query block's K/V (NaN there); the step writes them per layer
    and attends.  Outputs, accept and commit as the oracle on the complete caches; the caches end up bit-exact."""
    shape = wl.Shape(32, 8, 128, 5000, n_layers=3)
    step = wl.make_step("host_append", shape, [700, 130, 2049, 0], [32, 9, 20, 16], [16, 0, 8, 0], seed=19, p_match=0.7,
                        extra_table_cols=1)
    L, B, T, R = 3, step.batch, step.total_q_rows, step.total_cand_rows
    qs = [wl.make_q(step, l) for l in range(L)]
    kvs = [wl.make_kv(step, l) for l in range(L)]
    blocks = [wl.query_block_kv(step, kv) for kv in kvs]
    logits, drafts, _ = wl.make_logits(step)
    holes = []
    for kv in kvs:                                             # the same caches with the block's slots blanked
        h = kv.clone()
        for b in range(B):
            for j in range(int(step.prefix_lens[b]), int(step.kv_lens[b])):
                h[int(step.page_table[b, j // 16]), :, :, j % 16, :] = float("nan")
        holes.append(h.cuda())
    pin = lambda t: t.contiguous().pin_memory()
    q_host, out_host = pin(torch.stack(qs)), pin(torch.zeros((L, T, 32, 128), dtype=torch.bfloat16))
    k_host, v_host = pin(torch.stack([b_[0] for b_ in blocks])), pin(torch.stack([b_[1] for b_ in blocks]))
    h_logits, h_drafts = pin(logits), pin(drafts)
    h_pt, h_pl, h_ql, h_nm = pin(step.page_table.clone()), pin(step.prefix_lens.clone()), pin(step.q_lens), pin(step.n_mask)
    h_acc, h_bon = pin(torch.zeros(B, dtype=torch.int32)), pin(torch.zeros(B, dtype=torch.int32))
    h_freed, h_nf = pin(torch.full((B * 3,), -7, dtype=torch.int32)), pin(torch.zeros(1, dtype=torch.int32))
    with Ctx(step) as ctx:
        fd.fd_host_reserve(ctx.h, T, R)
        assert fd.fd_step_host_append(ctx.h, B, T, R, holes, step.num_pages, q_host, k_host, None, out_host, h_logits, h_drafts, h_pt,
                                      h_pl, h_ql, h_nm, h_acc, h_bon, h_freed, h_nf, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        fd.fd_step_host_append(ctx.h, B, T, R, holes, step.num_pages, q_host, k_host, v_host, out_host, h_logits, h_drafts, h_pt, h_pl,
                               h_ql, h_nm, h_acc, h_bon, h_freed, h_nf)
        torch.cuda.current_stream().synchronize()
        assert fd.fd_last_device_status(ctx.h) == 0
    for l in range(L):
        assert torch.equal(holes[l].cpu().view(torch.int16), kvs[l].view(torch.int16)), f"cache of layer {l}"
        ref = oracle.attn(qs[l], kvs[l], step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
        assert_close(out_host[l].float().numpy(), ref, f"layer {l}")
    e_acc, e_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    np.testing.assert_array_equal(h_acc.numpy(), e_acc); np.testing.assert_array_equal(h_bon.numpy(), e_bon)
    ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, e_acc)
    np.testing.assert_array_equal(h_pt.numpy(), ept); np.testing.assert_array_equal(h_pl.numpy(), epl)
    np.testing.assert_array_equal(h_freed.numpy()[:int(h_nf)], efreed)


def test_bounded_wait_times_out_cleanly_and_context_survives():
    """A device-side wait that nothing will ever satisfy gives up after its limit, raises FD_DEV_TIMEOUT and
    the kernel returns; the same context then computes a correct result."""
    import time
    step = wl.make_step("timeout", wl.Shape(8, 2, 128, 1000), [300], [12], [4], seed=2)
    q, kv = wl.make_q(step), wl.make_kv(step)
    with Ctx(step) as ctx:
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        fd.fd_selftest_wait_timeout(ctx.h, 50)
        assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_TIMEOUT          # synchronises
        dt = time.perf_counter() - t0
        assert 0.04 < dt < 2.0, dt
        assert fd.fd_last_device_status(ctx.h) == 0                           # read-and-clear
        got, status = gpu_attn(ctx, step, q, kv)
        assert status == 0
        assert_close(got.numpy(), oracle_attn(step, q, kv), "after timeout")


BLOCK_CASES = {
    # name: (Hq, Hkv, d, prefix_lens, C, M, n_blocks)
    "all_hypotheses": (32, 8, 128, [700, 130, 2049, 0, 5], [4, 8, 2, 4, 16], [28, 24, 30, 28, 16], [4, 8, 2, 4, 16]),
    "pruned_and_single": (32, 8, 128, [1000, 77, 300, 4000], [8, 6, 5, 16], [24, 12, 6, 0], [3, 1, 0, 0]),
    "block_straddles_tiles": (8, 2, 128, [120, 250, 383], [4, 4, 4], [28, 28, 28], [4, 2, 4]),
    "head_dim64": (16, 4, 64, [90, 513], [4, 8], [12, 24], [4, 8]),
    # query blocks longer than one 128-row tile holds (128 / G block rows): several row blocks per sequence.
    # First sequence = the paper's full parallel mode: bonus + 16 drafts and one 16-token branch per hypothesis.
    "long_blocks_all_17_hypotheses": (32, 8, 128, [300, 1000, 50, 700, 0], [17, 32, 16, 36, 40], [272, 8, 16, 64, 0], [17, 1, 1, 4, 0]),
    "long_blocks_gqa8_head_dim64": (16, 2, 64, [200, 31], [9, 20], [36, 30], [9, 2]),
}


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name", sorted(BLOCK_CASES))
def test_attention_mask_blocks(name, path):
    """Several next-draft branches per sequence (one mask block per hypothesis) against the oracle."""
    Hq, Hkv, d, pl, C, M, nb = BLOCK_CASES[name]
    step = wl.make_step(name, wl.Shape(Hq, Hkv, d, 1000), pl, [c + m for c, m in zip(C, M)], M,
                        seed=zlib.crc32(name.encode()) % 10000)
    q, kv = wl.make_q(step), wl.make_kv(step, poison=float("nan"))
    n_blocks = torch.tensor(nb, dtype=torch.int32)
    ref = oracle.attn_blocks(q, kv, step.page_table, step.prefix_lens, step.q_lens, step.n_mask, n_blocks)
    with Ctx(step, path, max_q_len=max(int(step.q_lens.max()), 1)) as ctx:
        dq, dkv = q.cuda(), kv.cuda()
        out = torch.full_like(dq, float("nan"))
        fd.fd_attn_draft_verify_blocks(ctx.h, step.batch, step.total_q_rows, dq, dkv, step.num_pages, step.page_table.cuda(),
                                       step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda(), n_blocks.cuda(), out)
        assert fd.fd_last_device_status(ctx.h) == 0
        assert_close(out.float().cpu().numpy(), ref, name)
        # broken block structure: not divisible / more blocks than hypotheses -> zeros and a status bit
        for bad in ([3 if m % 3 else 5 for m in M], [c + 1 for c in C]):
            if all(b_ <= 1 or (m % b_ == 0 and b_ <= c) for b_, m, c in zip(bad, M, C)):
                continue
            out.fill_(float("nan"))
            fd.fd_attn_draft_verify_blocks(ctx.h, step.batch, step.total_q_rows, dq, dkv, step.num_pages, step.page_table.cuda(),
                                           step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda(),
                                           torch.tensor(bad, dtype=torch.int32).cuda(), out)
            assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_BAD_LENGTHS and (out == 0).all()


def test_select_branch_matches_oracle():
    g = torch.Generator().manual_seed(4)
    B = 97
    C = torch.randint(1, 9, (B,), generator=g)
    nb = torch.tensor([int(torch.randint(0, int(c) + 1, (1,), generator=g)) for c in C])
    kb = torch.randint(1, 5, (B,), generator=g)
    M = torch.where(torch.rand(B, generator=g) < 0.15, torch.zeros_like(kb), kb * nb.clamp(min=1))
    step = wl.make_step("sel", wl.Shape(32, 8, 128, 1000), [3] * B, (C + M).tolist(), M.tolist(), seed=4)
    tokens = torch.randint(0, 1000, (int(M.sum()),), generator=g, dtype=torch.int32)
    acc = torch.tensor([int(torch.randint(-1, int(c), (1,), generator=g)) for c in C], dtype=torch.int32)
    exp_nd, exp_nl = oracle.select_branch(tokens, step.q_lens, step.n_mask, nb.int(), acc, max_kb=5)
    with Ctx(step) as ctx:
        nd = torch.full((B, 5), -9, dtype=torch.int32, device="cuda"); nl = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        fd.fd_select_branch(ctx.h, B, 5, tokens.cuda(), step.q_lens.cuda(), step.n_mask.cuda(), nb.int().cuda(), acc.cuda(), nd, nl)
        assert fd.fd_last_device_status(ctx.h) == 0
        np.testing.assert_array_equal(nd.cpu().numpy(), exp_nd); np.testing.assert_array_equal(nl.cpu().numpy(), exp_nl)
        fd.fd_select_branch(ctx.h, B, 2, tokens.cuda(), step.q_lens.cuda(), step.n_mask.cuda(), nb.int().cuda(), acc.cuda(),
                            nd[:, :2].contiguous(), nl)                       # blocks longer than the output rows
        assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_BAD_LENGTHS


@pytest.mark.parametrize("V,with_bias", [(151936, True), (151936, False), (4097, True), (1000, True), (37, False), (1, True)])
def test_draft_select_matches_oracle(V, with_bias):
    """Draft-side tail (Eq. 4 / Eq. 5) against the float64 oracle: tokens equal except where the oracle's margin
    between the two largest calibrated logits is below what a float32 sum can resolve (counted, bounded), confidences
    to 1e-4, verify lengths equal wherever the cumulative confidence is not within 1e-3 of the threshold (there the
    fp32 product may fall on either side)."""
    g = torch.Generator().manual_seed(V)
    M = [16, 0, 28, 6, 32, 12, 1]
    nb = [1, 1, 4, 0, 8, 3, 1]
    B, Rm = len(M), sum(M)
    logits = torch.randn((Rm, V), generator=g) * 2
    if V > 8:                                                   # confident drafts, as a trained drafter gives
        logits[torch.arange(Rm), torch.randint(0, V, (Rm,), generator=g)] += 9.0 * torch.rand((Rm,), generator=g) + 3.0
        logits[3, 5] = logits[3].max() + 1; logits[3, 2] = logits[3, 5]          # an exact tie: lowest index wins
    bias = torch.randn((Rm, V), generator=g) if with_bias else None
    n_mask, n_blocks = torch.tensor(M, dtype=torch.int32), torch.tensor(nb, dtype=torch.int32)
    step = wl.make_step("ds", wl.Shape(32, 8, 128, V), [5] * B, [32] * B, M, seed=1)
    with Ctx(step) as ctx:
        for thr in (0.5, 0.05):
            e_tok, e_pr, e_cum, e_keep, e_gap = oracle.draft_select(logits, bias, n_mask, n_blocks, thr, max_blocks=8, want_gap=True)
            tok = torch.full((Rm,), -9, dtype=torch.int32, device="cuda"); pr = torch.zeros((Rm,), device="cuda")
            keep = torch.full((B, 8), -9, dtype=torch.int32, device="cuda")
            fd.fd_draft_select(ctx.h, B, Rm, 8, logits.cuda(), None if bias is None else bias.cuda(), n_mask.cuda(), n_blocks.cuda(),
                               thr, tok, pr, keep)
            assert fd.fd_last_device_status(ctx.h) == 0
            # a float32 sum l + bias carries half an ulp of the sum per operand pair: two calibrated logits closer than
            # that may be ordered either way (or tie, lowest index first); anything wider must agree
            x_abs = float((logits.abs() + (bias.abs() if bias is not None else 0)).max())
            near = e_gap <= 2 * np.spacing(np.float32(x_abs))
            g_tok = tok.cpu().numpy()
            differ = g_tok != e_tok
            assert not (differ & ~near).any(), np.nonzero(differ & ~near)
            assert differ.sum() <= max(1, Rm // 20)
            same = ~differ
            np.testing.assert_allclose(pr.cpu().numpy()[same], e_pr[same], rtol=1e-4, atol=1e-30)
            got = keep.cpu().numpy()
            r0 = 0
            for b in range(B):
                n_b = max(nb[b], 1); kb = M[b] // n_b if M[b] else 0
                for gk in range(8):
                    c = e_cum[r0 + gk * kb:r0 + (gk + 1) * kb] if (M[b] and gk < n_b) else np.zeros(0)
                    if c.size and ((np.abs(c - thr) < 1e-3 * thr).any() or differ[r0 + gk * kb:r0 + (gk + 1) * kb].any()):
                        continue                                  # too close to call in fp32
                    assert got[b, gk] == e_keep[b, gk], (b, gk, got[b, gk], e_keep[b, gk])
                r0 += M[b]
            keep2 = torch.empty_like(keep); tok2 = torch.empty_like(tok); pr2 = torch.empty_like(pr)
            fd.fd_draft_select(ctx.h, B, Rm, 8, logits.cuda(), None if bias is None else bias.cuda(), n_mask.cuda(), n_blocks.cuda(),
                               thr, tok2, pr2, keep2)
            assert torch.equal(pr, pr2) and torch.equal(tok, tok2) and torch.equal(keep, keep2)      # bitwise repeatable
        bad = torch.tensor([16, 0, 28, 6, 32, 12, 2], dtype=torch.int32)                             # rows do not add up
        fd.fd_draft_select(ctx.h, B, Rm, 8, logits.cuda(), None, bad.cuda(), n_blocks.cuda(), 0.5, tok, pr, keep)
        assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_BAD_LENGTHS and (tok == -1).all() and (keep == 0).all()


@pytest.mark.parametrize("V,with_second,B", [(20004, True, 40), (20004, False, 40), (8192, True, 100), (12292, False, 48)])
def test_sweeps_aligned_and_one_float_off_agree_bit_for_bit(V, with_second, B):
    """Draft-side tail and sampling verification over several hundred rows, once on 16-byte aligned arrays (vector
    loads) and once on the same data one float off alignment (scalar loads): a chunk's partial and the order the
    partials are combined in do not depend on how the chunk was loaded, so every output must be identical -- tokens,
    confidences (bitwise), verify lengths, accepted lengths, bonus tokens -- and both must agree with the oracle.
    Row 7 has one finite logit, in the last chunk: every other chunk of it is -inf throughout."""
    g = torch.Generator().manual_seed(V + int(with_second))
    M = torch.randint(14, 17, (B,), generator=g).tolist()
    Rm = sum(M)
    logits = torch.randn((Rm, V), generator=g) * 2
    logits[torch.arange(Rm), torch.randint(0, V, (Rm,), generator=g)] += 9.0 * torch.rand((Rm,), generator=g) + 3.0
    logits[7, :] = -float("inf"); logits[7, V - 1] = 0.5        # one finite logit, in the ragged last chunk
    second = torch.randn((Rm, V), generator=g) if with_second else None
    n_mask = torch.tensor(M, dtype=torch.int32); n_blocks = torch.ones((B,), dtype=torch.int32)
    step = wl.make_step("ds", wl.Shape(32, 8, 128, V), [5] * B, [32] * B, M, seed=1)
    with Ctx(step) as ctx:
        res = []
        for mk in (lambda t: t.cuda(), _one_float_off):
            tok = torch.full((Rm,), -9, dtype=torch.int32, device="cuda"); pr = torch.zeros((Rm,), device="cuda")
            keep = torch.full((B, 2), -9, dtype=torch.int32, device="cuda")
            fd.fd_draft_select(ctx.h, B, Rm, 2, mk(logits), None if second is None else mk(second), n_mask.cuda(), n_blocks.cuda(),
                               0.3, tok, pr, keep)
            assert fd.fd_last_device_status(ctx.h) == 0
            res.append((tok.cpu(), pr.cpu(), keep.cpu()))
        assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][2], res[1][2])
        assert torch.equal(res[0][1].view(torch.int32), res[1][1].view(torch.int32))
        e_tok, e_pr, _, _, e_gap = oracle.draft_select(logits, second, n_mask, n_blocks, 0.3, max_blocks=2, want_gap=True)
        x_abs = float((logits[torch.isfinite(logits)].abs().max() + (second.abs().max() if second is not None else 0)))
        same = res[0][0].numpy() == e_tok
        assert (same | (e_gap <= 2 * np.spacing(np.float32(x_abs)))).all()
        np.testing.assert_allclose(res[0][1].numpy()[same], e_pr[same], rtol=1e-4, atol=1e-30)

        # sampling verification over the same rows taken as candidate rows (draft logits = `second`)
        ql = torch.tensor(M, dtype=torch.int32); nm0 = torch.zeros((B,), dtype=torch.int32)
        drafts = torch.randint(0, V, (Rm,), generator=g, dtype=torch.int32)
        am = logits.argmax(dim=1).to(torch.int32)
        drafts[1:] = torch.where(torch.rand((Rm - 1,), generator=g) < 0.8, am[:-1], drafts[1:])
        ua = torch.rand((Rm,), generator=g); ub = torch.rand((B,), generator=g)
        out = []
        for mk in (lambda t: t.cuda(), _one_float_off):
            acc = torch.full((B,), -7, dtype=torch.int32, device="cuda"); bon = torch.full((B,), -7, dtype=torch.int32, device="cuda")
            for _ in range(2):                                  # twice: the counters must come back to zero
                fd.fd_verify_accept_sample(ctx.h, B, Rm, mk(logits), None if second is None else mk(second), drafts.cuda(), ql.cuda(),
                                           nm0.cuda(), 0.7, ua.cuda(), ub.cuda(), acc, bon)
                assert fd.fd_last_device_status(ctx.h) == 0
            out.append((acc.cpu(), bon.cpu()))
        assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1])
        acc_ref, _, ratio = oracle.accept_stochastic(logits.numpy(), None if second is None else second.numpy(), drafts.numpy(),
                                                     ql.numpy(), nm0.numpy(), 0.7, ua.numpy(), ub.numpy())
        differ = int((out[0][0].numpy() != acc_ref).sum())
        assert differ <= max(1, B // 10), differ                # fp32 probabilities: only near-ties may part


def test_kv_append_matches_oracle_and_feeds_the_attention():
    """fd_kv_append bit-exact against the oracle (every byte of the pool), then attention over the appended cache."""
    shape = wl.Shape(32, 8, 128, 1000)
    step = wl.make_step("append", shape, [0, 15, 16, 700, 2047], [32, 3, 17, 1, 20], [16, 0, 9, 0, 8], seed=33, extra_table_cols=1)
    kv = wl.make_kv(step, poison=None)
    g = torch.Generator().manual_seed(3)
    T = step.total_q_rows
    k_new = torch.randn((T, 8, 128), generator=g).bfloat16(); v_new = torch.randn((T, 8, 128), generator=g).bfloat16()
    exp_bits = oracle.kv_append(k_new, v_new, kv, step.page_table, step.prefix_lens, step.q_lens)
    q = wl.make_q(step)
    with Ctx(step) as ctx:
        dkv = kv.cuda()
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        fd.fd_kv_append(ctx.h, step.batch, T, k_new.cuda(), v_new.cuda(), dkv, step.num_pages, dpt, dpl, dql)
        assert fd.fd_last_device_status(ctx.h) == 0
        got_bits = dkv.cpu().view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(got_bits, exp_bits)
        out = torch.empty((T, 32, 128), dtype=torch.bfloat16, device="cuda")
        fd.fd_attn_draft_verify(ctx.h, step.batch, T, q.cuda(), dkv, step.num_pages, dpt, dpl, dql, dnm, out)
        kv_ref = torch.from_numpy(exp_bits.view(np.int16)).view(torch.bfloat16)
        assert_close(out.float().cpu().numpy(), oracle.attn(q, kv_ref, step.page_table, step.prefix_lens, step.q_lens, step.n_mask), "append+attend")
        bad = step.page_table.clone(); bad[2, 1] = -1                       # a page of the block is not allocated
        dkv2 = kv.cuda()
        fd.fd_kv_append(ctx.h, step.batch, T, k_new.cuda(), v_new.cuda(), dkv2, step.num_pages, bad.cuda(), dpl, dql)
        assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_BAD_PAGE
        fd.fd_kv_append(ctx.h, step.batch, T - 1, k_new.cuda(), v_new.cuda(), dkv2, step.num_pages, dpt, dpl, dql)
        assert fd.fd_last_device_status(ctx.h) == fd.FD_DEV_BAD_LENGTHS


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_chain_of_calls_whose_output_is_the_next_query(idx):
    """Under a pinned plan consecutive attention calls overlap: a call may read its q and its cache while the call
    before it is still running, unless that call writes them.  Here every call's q IS the previous call's out (the
    buffers start as NaN), interleaved with calls on buffers of their own: reading ahead must happen only where it is
    safe, so every result has to match the oracle applied layer by layer."""
    step = wl.workload(idx)
    s = step.shape
    L = 6
    kvs = [wl.make_kv(step, l) for l in range(L)]
    q0 = wl.make_q(step)
    with Ctx(step) as ctx:
        fd.fd_calls_back_to_back(ctx.h, True)                      # nothing but the library's launches between the calls below
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        dkv = [k.cuda() for k in kvs]
        dq0 = q0.cuda()
        for rep in range(2):
            outs = [torch.full_like(dq0, float("nan")) for _ in range(L)]
            fd.fd_plan_pin(ctx.h, step.batch, step.total_q_rows, dpl, dql, dnm)
            q = dq0
            for l in range(L):
                fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, q, dkv[l], step.num_pages, dpt, dpl, dql, dnm, outs[l])
                q = outs[l] if l % 2 == 0 else dq0                               # odd layers feed on the even layer's output
            fd.fd_plan_unpin(ctx.h)
            assert fd.fd_last_device_status(ctx.h) == 0
            # the reference of a layer that feeds on an output is computed from what the kernel produced there
            for l in range(L):
                fed = q0 if l % 2 == 0 else outs[l - 1].cpu()
                ref = oracle.attn(fed, kvs[l], step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
                assert_close(outs[l].float().cpu().numpy(), ref, f"{step.name} layer {l} rep {rep}")


def test_chained_append_whose_input_is_the_previous_output():
    """Under a pinned plan the append of layer l + 1 runs while the attention call of layer l is finishing, unless it
    reads what that call writes.  Layer 1's k_new here IS (a part of) layer 0's out, NaN beforehand; layers 2 and 3 have
    inputs of their own.  Every cache must end up as the oracle's append of what the inputs finally held, every output
    as the oracle's attention over that cache."""
    step = wl.workload(2)
    s = step.shape
    T, L = step.total_q_rows, 4
    g = torch.Generator().manual_seed(21)
    kvs = [wl.make_kv(step, l) for l in range(L)]
    qs = [wl.make_q(step, l) for l in range(L)]
    kn = [torch.randn((T, s.n_kv_heads, s.head_dim), generator=g).bfloat16() for _ in range(L)]
    vn = [torch.randn((T, s.n_kv_heads, s.head_dim), generator=g).bfloat16() for _ in range(L)]
    with Ctx(step) as ctx:
        fd.fd_calls_back_to_back(ctx.h, True)                      # nothing but the library's launches between the calls below
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        for rep in range(2):
            pools = [k.cuda() for k in kvs]
            outs = [torch.full((T, s.n_q_heads, s.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
            dkn = [k.cuda() for k in kn]; dvn = [v.cuda() for v in vn]
            dkn[1] = outs[0].view(-1)[: T * s.n_kv_heads * s.head_dim].view(T, s.n_kv_heads, s.head_dim)   # aliases out of layer 0
            fd.fd_plan_pin(ctx.h, step.batch, T, dpl, dql, dnm)
            for l in range(L):
                fd.fd_kv_append(ctx.h, step.batch, T, dkn[l], dvn[l], pools[l], step.num_pages, dpt, dpl, dql)
                fd.fd_attn_draft_verify(ctx.h, step.batch, T, qs[l].cuda(), pools[l], step.num_pages, dpt, dpl, dql, dnm, outs[l])
            fd.fd_plan_unpin(ctx.h)
            assert fd.fd_last_device_status(ctx.h) == 0
            for l in range(L):
                exp_bits = oracle.kv_append(dkn[l].cpu(), dvn[l].cpu(), kvs[l], step.page_table, step.prefix_lens, step.q_lens)
                np.testing.assert_array_equal(pools[l].cpu().view(torch.int16).numpy().view(np.uint16), exp_bits)
                kv_ref = torch.from_numpy(exp_bits.view(np.int16)).view(torch.bfloat16)
                ref = oracle.attn(qs[l], kv_ref, step.page_table, step.prefix_lens, step.q_lens, step.n_mask)
                assert_close(outs[l].float().cpu().numpy(), ref, f"layer {l} rep {rep}")


@pytest.mark.parametrize("seed", list(range(100, 130)))
def test_random_chains_against_the_oracle(seed):
    """Thirty seeded random batches (1 to 60 sequences, any head layout) through three layers under one pinned plan --
    with or without the append of the block's own K/V before each attention call, with or without the caller's promise
    that lets consecutive launches overlap -- three times over: every cache bit for bit, every output element within
    tolerance, NaN in the output buffers beforehand."""
    g = torch.Generator().manual_seed(seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))
    G = [1, 2, 4, 8][ri(0, 3)]
    Hkv = [1, 2, 4, 8][ri(0, 3)]
    while G * Hkv > 32:
        Hkv //= 2
    d = [64, 128][ri(0, 1)]
    B = [ri(1, 3), ri(4, 12), ri(13, 60)][ri(0, 2)]
    max_rows = min(32, 128 // G)
    pl = [[0, ri(1, 40), ri(100, 140), ri(0, 1200), ri(0, 1200)][ri(0, 4)] for _ in range(B)]
    ql = [0 if ri(0, 11) == 0 else ri(1, max_rows) for _ in range(B)]
    nm = [ri(0, L) for L in ql]
    overlap, with_append = bool(ri(0, 1)), bool(ri(0, 1))
    step = wl.make_step(f"chain{seed}", wl.Shape(G * Hkv, Hkv, d, 1000), pl, ql, nm, seed=seed, extra_table_cols=ri(0, 2))
    T, s, L = step.total_q_rows, step.shape, 3
    if T == 0:
        pytest.skip("all blocks empty")
    qs = [wl.make_q(step, l) for l in range(L)]
    kvs = [wl.make_kv(step, l) for l in range(L)]
    kn = [torch.randn((T, Hkv, d), generator=g).bfloat16() for _ in range(L)]
    vn = [torch.randn((T, Hkv, d), generator=g).bfloat16() for _ in range(L)]
    caches, refs = [], []
    for l in range(L):
        bits = oracle.kv_append(kn[l], vn[l], kvs[l], step.page_table, step.prefix_lens, step.q_lens) if with_append else \
            kvs[l].view(torch.int16).numpy().view(np.uint16)
        caches.append(bits)
        refs.append(oracle_attn(step, qs[l], torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)))
    with Ctx(step) as ctx:
        fd.fd_calls_back_to_back(ctx.h, overlap)
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        dq, dkn, dvn = [q.cuda() for q in qs], [k.cuda() for k in kn], [v.cuda() for v in vn]
        for rep in range(3):
            pools = [k.cuda() for k in kvs]
            outs = [torch.full((T, s.n_q_heads, d), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
            fd.fd_plan_pin(ctx.h, B, T, dpl, dql, dnm)
            for l in range(L):
                if with_append:
                    fd.fd_kv_append(ctx.h, B, T, dkn[l], dvn[l], pools[l], step.num_pages, dpt, dpl, dql)
                fd.fd_attn_draft_verify(ctx.h, B, T, dq[l], pools[l], step.num_pages, dpt, dpl, dql, dnm, outs[l])
            fd.fd_plan_unpin(ctx.h)
            assert fd.fd_last_device_status(ctx.h) == 0
            for l in range(L):
                np.testing.assert_array_equal(pools[l].cpu().view(torch.int16).numpy().view(np.uint16), caches[l])
                assert_close(outs[l].float().cpu().numpy(), refs[l], f"{step.name} layer {l} rep {rep} overlap {overlap} append {with_append}")


def test_pinned_plan_serves_every_layer_and_is_dropped_on_other_lengths():
    """fd_plan_pin: several attention calls reuse one work list; a call with other lengths recomputes it."""
    step = wl.workload(2)
    step2 = wl.make_step("other", step.shape, [300, 500], [20, 7], [16, 0], seed=77)
    wide = torch.full((2, step.max_pages_per_seq), -1, dtype=torch.int32)   # the context fixes the table width
    wide[:, :step2.max_pages_per_seq] = step2.page_table
    step2.page_table = wide
    with Ctx(step) as ctx:
        dev = {k: getattr(step, k).cuda() for k in ("page_table", "prefix_lens", "q_lens", "n_mask")}
        fd.fd_plan_pin(ctx.h, step.batch, step.total_q_rows, dev["prefix_lens"], dev["q_lens"], dev["n_mask"])
        before = fd.fd_launch_count(ctx.h)
        for layer in range(3):
            q, kv = wl.make_q(step, layer), wl.make_kv(step, layer)
            out = torch.empty(q.shape, dtype=torch.bfloat16, device="cuda")
            fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, q.cuda(), kv.cuda(), step.num_pages, dev["page_table"],
                                    dev["prefix_lens"], dev["q_lens"], dev["n_mask"], out)
            assert fd.fd_last_device_status(ctx.h) == 0
            assert_close(out.float().cpu().numpy(), oracle_attn(step, q, kv), f"pinned layer {layer}")
        assert fd.fd_launch_count(ctx.h) - before == 3          # one kernel per call: no plan launches
        q2, kv2 = wl.make_q(step2), wl.make_kv(step2)
        got, status = gpu_attn(ctx, step2, q2, kv2)             # other lengths: the pin is dropped, a new plan is made
        assert status == 0
        assert_close(got.numpy(), oracle_attn(step2, q2, kv2), "after the pin")
        fd.fd_plan_unpin(ctx.h)


def test_commit_drops_the_pinned_plan():
    """pin, attend, accept-less commit, attend again on the same length arrays without pinning again: the commit has
    rewritten prefix_lens in place, so the second call must plan for the new lengths, not reuse the old work list."""
    shape = wl.Shape(32, 8, 128, 1000)
    step = wl.make_step("pin_commit", shape, [700, 200, 3000], [20, 8, 32], [4, 4, 16], seed=41, extra_table_cols=3)
    q, kv = wl.make_q(step), wl.make_kv(step, poison=None)           # every page holds data: pages get reassigned below
    with Ctx(step) as ctx:
        dq, dkv = q.cuda(), kv.cuda()
        dpt, dpl, dql, dnm = step.page_table.cuda(), step.prefix_lens.cuda(), step.q_lens.cuda(), step.n_mask.cuda()
        out = torch.empty_like(dq)
        fd.fd_plan_pin(ctx.h, step.batch, step.total_q_rows, dpl, dql, dnm)
        fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, dq, dkv, step.num_pages, dpt, dpl, dql, dnm, out)
        assert_close(out.float().cpu().numpy(), oracle_attn(step, q, kv), "pinned")
        acc = torch.tensor([15, 0, 7], dtype=torch.int32)
        freed = torch.empty((64,), dtype=torch.int32, device="cuda"); nf = torch.zeros((1,), dtype=torch.int32, device="cuda")
        fd.fd_kv_commit(ctx.h, step.batch, dpt, dpl, dql, acc.cuda(), freed, nf)
        ept, epl, efreed = oracle.commit(step.page_table, step.prefix_lens, step.q_lens, acc)
        np.testing.assert_array_equal(dpl.cpu().numpy(), epl)
        # the host hands pages back for the next block (same device arrays, new contents)
        pool = efreed.tolist() + step.spare_pages.tolist()
        npt = ept.copy()
        for b in range(step.batch):
            for pg in range(-(-(int(epl[b]) + int(step.q_lens[b])) // 16)):
                if npt[b, pg] < 0:
                    npt[b, pg] = pool.pop()
        dpt.copy_(torch.from_numpy(npt))
        before = fd.fd_launch_count(ctx.h)
        fd.fd_attn_draft_verify(ctx.h, step.batch, step.total_q_rows, dq, dkv, step.num_pages, dpt, dpl, dql, dnm, out)
        assert fd.fd_last_device_status(ctx.h) == 0
        assert fd.fd_launch_count(ctx.h) - before >= 1
        ref = oracle.attn(q, kv, npt, epl, step.q_lens, step.n_mask)
        assert_close(out.float().cpu().numpy(), ref, "after the commit")


def _stochastic_case(seed, V, B, T, with_q, max_c=8):
    rng = np.random.default_rng(seed)
    C = rng.integers(0, max_c + 1, size=B); C[0] = max_c; C[-1] = 1
    M = rng.integers(0, 4, size=B)
    R = int(C.sum())
    logits = (rng.normal(size=(R, V)) * 2.0).astype(np.float32)
    dlog = (logits + rng.normal(size=(R, V)).astype(np.float32) * 0.7).astype(np.float32)
    drafts = rng.integers(0, V, size=R).astype(np.int32)
    for r in range(R - 1):                                   # proposals drawn from q (or its argmax): mostly accepted
        z = (dlog[r].astype(np.float64) - dlog[r].max()) / T
        if with_q:
            pr = np.exp(z); pr /= pr.sum()
            drafts[r + 1] = rng.choice(V, p=pr)
        else:
            drafts[r + 1] = int(np.argmax(logits[r])) if rng.random() < 0.7 else int(rng.integers(0, V))
    ua = rng.random(R, dtype=np.float32); ub = rng.random(B, dtype=np.float32)
    return (C + M).astype(np.int32), M.astype(np.int32), logits, (dlog if with_q else None), drafts, ua, ub


@pytest.mark.parametrize("V,B,T,with_q", [(1000, 33, 1.0, True), (5000, 16, 0.6, True), (5000, 16, 0.3, False),
                                         (151936, 6, 0.6, True), (151936, 6, 1.0, False)])
def test_stochastic_verification_matches_oracle(V, B, T, with_q):
    """fd_verify_accept_sample against the speculative-sampling oracle on the same uniforms.  A decision is compared
    exactly unless the oracle shows that it sits on a rounding boundary (the kernel forms probabilities in fp32)."""
    ql, nm, logits, dlog, drafts, ua, ub = _stochastic_case(1234 + V + B, V, B, T, with_q)
    R = logits.shape[0]
    acc_ref, bon_ref, ratio, w = oracle.accept_stochastic(logits, dlog, drafts, ql, nm, T, ua, ub, want_weights=True)
    h = fd.fd_create(32, 8, 128, V, B, 16, 8)
    try:
        t = lambda a: torch.from_numpy(a).cuda()
        acc = torch.full((B,), -7, dtype=torch.int32, device="cuda"); bon = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        for _ in range(2):                                   # twice: the scratch counters must come back to zero
            fd.fd_verify_accept_sample(h, B, R, t(logits), None if dlog is None else t(dlog), t(drafts), t(ql), t(nm), T, t(ua), t(ub),
                                       acc, bon)
            assert fd.fd_last_device_status(h) == 0
        acc, bon = acc.cpu().numpy(), bon.cpu().numpy()
    finally:
        fd.fd_destroy(h)
    C = ql - nm
    r0, boundary = 0, 0
    for b in range(B):
        if C[b] == 0:
            assert acc[b] == -1 and bon[b] == -1
            continue
        tested = np.arange(r0, r0 + C[b] - 1)
        near = np.abs(ua[tested] - np.minimum(1.0, ratio[tested])) < 2e-5 + 1e-4 * ratio[tested]
        if acc[b] != acc_ref[b]:                             # allowed only where the test they part at is a near-tie
            d = min(int(acc[b]), int(acc_ref[b]))
            assert 0 <= d < len(tested) and near[d], (b, acc[b], acc_ref[b])
            boundary += 1
        else:
            cdf = np.cumsum(w[b]); tot = cdf[-1]
            tk = int(bon[b])
            assert 0 <= tk < V
            if tk != bon_ref[b]:
                lo = (cdf[tk - 1] if tk > 0 else 0.0) / tot; hi = cdf[tk] / tot
                assert w[b][tk] > 0 and lo - 1e-5 <= float(ub[b]) <= hi + 1e-5, (b, tk, bon_ref[b], lo, hi, ub[b])
                boundary += 1
        r0 += C[b]
    assert boundary <= max(1, B // 10), boundary


def test_stochastic_verification_errors():
    h = fd.fd_create(32, 8, 128, 1000, 4, 16, 8)
    try:
        z = torch.zeros((8, 1000), dtype=torch.float32, device="cuda"); i4 = torch.zeros((8,), dtype=torch.int32, device="cuda")
        u = torch.zeros((8,), dtype=torch.float32, device="cuda")
        assert fd.fd_verify_accept_sample(h, 2, 4, z, None, i4, i4, i4, 0.0, u, u, i4, i4, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        assert fd.fd_verify_accept_sample(h, 2, 4, None, None, i4, i4, i4, 1.0, u, u, i4, i4, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
        ql = torch.tensor([3, 2], dtype=torch.int32, device="cuda"); nm = torch.zeros((2,), dtype=torch.int32, device="cuda")
        acc = torch.full((2,), 7, dtype=torch.int32, device="cuda"); bon = torch.full((2,), 7, dtype=torch.int32, device="cuda")
        fd.fd_verify_accept_sample(h, 2, 4, z, None, i4, ql, nm, 1.0, u, u, acc, bon)             # 5 rows claimed, 4 given
        assert fd.fd_last_device_status(h) == fd.FD_DEV_BAD_LENGTHS
        assert (acc == -1).all() and (bon == -1).all()           # the convention of every call: -1 for all sequences
        ql = torch.tensor([3, 1], dtype=torch.int32, device="cuda")
        fd.fd_verify_accept_sample(h, 2, 4, z, None, i4, ql, nm, 1.0, u, u, acc, bon)             # the context still works
        assert fd.fd_last_device_status(h) == 0 and (acc >= 0).all() and (bon >= 0).all()
    finally:
        fd.fd_destroy(h)


def test_multi_step_decode_loop_append_attend_accept_commit():
    """Twelve decode steps of a toy target through the C ABI -- KV append, attention, greedy accept, commit with
    rollback, pages handed back and reused -- against the same loop run on the oracle; both must stay in lockstep
    (bit-exact lengths, tokens and page tables; attention within tolerance; the cache bit-exact) and commit exactly
    the greedy sequence of the toy target."""
    V, B, k, M, steps, P, W = 50, 3, 5, 4, 12, 16, 16
    Hq, Hkv, d = 8, 2, 128
    rng = np.random.default_rng(21)
    table = rng.standard_normal((V, V)).astype(np.float32)
    nxt = np.argmax(table, axis=1)
    g = torch.Generator().manual_seed(5)
    emb_k = torch.randn((V + 1, Hkv, d), generator=g).bfloat16(); emb_v = torch.randn((V + 1, Hkv, d), generator=g).bfloat16()
    num_pages = 64
    kv_ref = torch.zeros((num_pages, 2, Hkv, P, d), dtype=torch.bfloat16)          # oracle side cache
    kv_gpu = kv_ref.clone().cuda()
    pt = np.full((B, W), -1, np.int32); pl = np.zeros((B,), np.int32)
    free = list(range(num_pages - 1, -1, -1))
    bonus = [3, 11, 29]
    committed = [[] for _ in range(B)]
    h = fd.fd_create(Hq, Hkv, d, V, B, 16, W)
    try:
        for step_i in range(steps):
            fed_all, ql, nm = [], [], []
            for b in range(B):
                drafts, prev = [], bonus[b]
                for _ in range(k if b != 1 else 2):                                  # ragged: sequence 1 drafts less
                    t = int(nxt[prev]) if rng.random() < 0.7 else int(rng.integers(V))
                    drafts.append(t); prev = t
                fed = [bonus[b]] + drafts
                m_b = M if b != 2 else 0                                             # sequence 2 runs without mask tokens
                need = -(-(int(pl[b]) + len(fed) + m_b) // P)
                for pg in range(need):
                    if pt[b, pg] < 0:
                        pt[b, pg] = free.pop()
                fed_all.append(fed); ql.append(len(fed) + m_b); nm.append(m_b)
            ql_a, nm_a = np.array(ql, np.int32), np.array(nm, np.int32)
            tok_rows = [t for b in range(B) for t in fed_all[b] + [V] * nm[b]]      # mask token = extra embedding row V
            k_new, v_new = emb_k[tok_rows], emb_v[tok_rows]
            T = len(tok_rows)
            q = torch.randn((T, Hq, d), generator=g).bfloat16()
            cand_tok = np.array([t for b in range(B) for t in fed_all[b]], np.int32)
            logits = table[cand_tok]
            # oracle side
            bits = oracle.kv_append(k_new, v_new, kv_ref, pt, pl, ql_a)
            kv_ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
            ref_out = oracle.attn(q, kv_ref, pt, pl, ql_a, nm_a)
            acc_r, bon_r, _ = oracle.accept(logits, cand_tok, ql_a, nm_a)
            pt_r, pl_r, freed_r = oracle.commit(pt, pl, ql_a, acc_r)
            # GPU side
            t32 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
            dpt, dpl, dql, dnm = t32(pt), t32(pl), t32(ql_a), t32(nm_a)
            fd.fd_kv_append(h, B, T, k_new.cuda(), v_new.cuda(), kv_gpu, num_pages, dpt, dpl, dql)
            out = torch.empty((T, Hq, d), dtype=torch.bfloat16, device="cuda")
            fd.fd_attn_draft_verify(h, B, T, q.cuda(), kv_gpu, num_pages, dpt, dpl, dql, dnm, out)
            acc = torch.empty((B,), dtype=torch.int32, device="cuda"); bon = torch.empty_like(acc)
            fd.fd_verify_accept(h, B, len(cand_tok), t32(logits), t32(cand_tok), dql, dnm, acc, bon)
            freed = torch.full((B * W,), -7, dtype=torch.int32, device="cuda"); nf = torch.zeros((1,), dtype=torch.int32, device="cuda")
            fd.fd_kv_commit(h, B, dpt, dpl, dql, acc, freed, nf)
            assert fd.fd_last_device_status(h) == 0
            assert torch.equal(kv_gpu.cpu().view(torch.int16), kv_ref.view(torch.int16)), f"cache, step {step_i}"
            assert_close(out.float().cpu().numpy(), ref_out, f"attention, step {step_i}")
            np.testing.assert_array_equal(acc.cpu().numpy(), acc_r); np.testing.assert_array_equal(bon.cpu().numpy(), bon_r)
            np.testing.assert_array_equal(dpt.cpu().numpy(), pt_r); np.testing.assert_array_equal(dpl.cpu().numpy(), pl_r)
            n = int(nf.item())
            np.testing.assert_array_equal(freed.cpu().numpy()[:n], freed_r)
            for b in range(B):
                committed[b] += fed_all[b][:int(acc_r[b]) + 1]
                bonus[b] = int(bon_r[b])
            free += freed_r.tolist()[::-1]
            pt, pl = pt_r, pl_r
            assert [len(c) for c in committed] == pl.tolist()
    finally:
        fd.fd_destroy(h)
    for b, start in enumerate([3, 11, 29]):                                          # lossless: plain greedy decoding
        greedy = [start]
        for _ in range(len(committed[b])):
            greedy.append(int(nxt[greedy[-1]]))
        assert committed[b] == greedy[:len(committed[b])] and bonus[b] == greedy[len(committed[b])]
    assert sorted(free + pt[pt >= 0].tolist()) == list(range(num_pages))


def test_stochastic_verification_is_lossless_on_the_gpu():
    """The defining property, measured on the kernel itself: whatever the drafter proposes, the token committed at
    the first position is distributed as the target distribution p_0 (98 304 draws, small vocabulary)."""
    rng = np.random.default_rng(8)
    V, B, calls, T = 11, 4096, 24, 0.8
    lp = (rng.normal(size=(2, V)) * 1.5).astype(np.float32)
    ld = (lp + rng.normal(size=(2, V))).astype(np.float32)
    sm = lambda x: np.exp((x.astype(np.float64) - x.max()) / T) / np.exp((x.astype(np.float64) - x.max()) / T).sum()
    p0, q0 = sm(lp[0]), sm(ld[0])
    logits = torch.from_numpy(np.tile(lp, (B, 1))).cuda(); dlog = torch.from_numpy(np.tile(ld, (B, 1))).cuda()
    ql = torch.full((B,), 2, dtype=torch.int32, device="cuda"); nm = torch.zeros((B,), dtype=torch.int32, device="cuda")
    acc = torch.empty((B,), dtype=torch.int32, device="cuda"); bon = torch.empty_like(acc)
    counts = np.zeros((V,), np.int64); accepted = 0
    h = fd.fd_create(32, 8, 128, V, B, 16, 8)
    try:
        for _ in range(calls):
            x = rng.choice(V, size=B, p=q0).astype(np.int32)
            drafts = np.zeros((2 * B,), np.int32); drafts[1::2] = x
            ua = torch.from_numpy(rng.random(2 * B, dtype=np.float32)).cuda(); ub = torch.from_numpy(rng.random(B, dtype=np.float32)).cuda()
            fd.fd_verify_accept_sample(h, B, 2 * B, logits, dlog, torch.from_numpy(drafts).cuda(), ql, nm, T, ua, ub, acc, bon)
            a, bo = acc.cpu().numpy(), bon.cpu().numpy()
            assert set(np.unique(a)) <= {0, 1}
            counts += np.bincount(np.where(a == 1, x, bo), minlength=V)
            accepted += int((a == 1).sum())
        assert fd.fd_last_device_status(h) == 0
    finally:
        fd.fd_destroy(h)
    n = B * calls
    freq = counts / n
    assert np.all(np.abs(freq - p0) < 4.5 * np.sqrt(p0 * (1 - p0) / n) + 1e-9), (freq, p0)
    assert abs(accepted / n - np.minimum(p0, q0).sum()) < 5e-3
