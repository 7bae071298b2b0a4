"""fd_verify_accept_static -- the verification step for callers that cannot allocate device memory
(a plugin inside a serving process whose pool owns the whole GPU, code running next to a stream
capture, a worker that starts on a full device).  It keeps its scratch in an array compiled into
the library, so every call in the process shares that array and its contents survive from call to
call.  The checks: through the C ABI, its results equal those of fd_verify_accept (bit-exact, the
bar of every accept test here) on two different calls in a row -- the second would be wrong if the
first left anything behind -- and an oversized request is refused without a launch.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_20022_b200 as fd
from paper_2605_20022_b200 import workload as wl

pytestmark = pytest.mark.gpu


def run_both(step, seed_shift):
    step.seed += seed_shift
    logits, drafts, _ = wl.make_logits(step)
    B, R, V = step.batch, step.total_cand_rows, step.shape.vocab
    d = lambda t: t.cuda()
    dl, dd, dq, dm = d(logits), d(drafts), d(step.q_lens), d(step.n_mask)
    ctx = fd.fd_create(step.shape.n_q_heads, step.shape.n_kv_heads, step.shape.head_dim, V, B, 32, 8)
    try:
        acc0 = torch.full((B,), -5, dtype=torch.int32, device="cuda"); bon0 = acc0.clone()
        fd.fd_verify_accept(ctx, B, R, dl, dd, dq, dm, acc0, bon0)
    finally:
        fd.fd_destroy(ctx)
    acc1 = torch.full((B,), -6, dtype=torch.int32, device="cuda"); bon1 = acc1.clone()
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fd.fd_verify_accept_static(V, B, R, dl, dd, dq, dm, acc1, bon1, status)
    torch.cuda.synchronize()
    assert int(status) == 0
    assert torch.equal(acc0, acc1) and torch.equal(bon0, bon1)
    e_acc, e_bon, _ = oracle.accept(logits, drafts, step.q_lens, step.n_mask)
    np.testing.assert_array_equal(acc1.cpu().numpy(), e_acc)
    np.testing.assert_array_equal(bon1.cpu().numpy(), e_bon)
    return acc1.cpu().numpy()


def test_static_scratch_accept_matches_context_accept_twice_in_a_row():
    big = wl.make_step("a", wl.Shape(32, 8, 128, 151936), [7] * 6, [16, 32, 5, 16, 1, 20], [0, 16, 0, 16, 0, 8], seed=41, p_match=0.8)
    small = wl.make_step("b", wl.Shape(32, 8, 128, 9001), [7] * 9, [3, 16, 16, 32, 2, 9, 16, 1, 12], [0, 0, 16, 16, 1, 3, 0, 0, 4], seed=42, p_match=0.6)
    a = run_both(big, 0)
    b = run_both(small, 0)          # fewer rows than the call before it: stale keys beyond its rows are never read
    c = run_both(big, 1)            # more rows again, different logits
    assert (a >= -1).all() and (b >= -1).all() and (c >= -1).all()


def test_static_scratch_limits_and_status_word():
    z = torch.zeros((4,), dtype=torch.int32, device="cuda")
    f = torch.zeros((4, 16), dtype=torch.float32, device="cuda")
    too_many = fd.FD_STATIC_MAX_ROWS + 1
    assert fd.fd_verify_accept_static(16, 1, too_many, f, z, z, z, z, z, None, raise_on_error=False) == fd.FD_ERR_STATIC_LIMIT
    assert fd.fd_verify_accept_static(16, fd.FD_STATIC_MAX_BATCH + 1, 4, f, z, z, z, z, z, None, raise_on_error=False) == fd.FD_ERR_STATIC_LIMIT
    assert fd.fd_verify_accept_static(16, 1, 4, None, z, z, z, z, z, None, raise_on_error=False) == fd.FD_ERR_INVALID_ARG
    assert fd.status_string(fd.FD_ERR_STATIC_LIMIT) == "FD_ERR_STATIC_LIMIT"
    # lengths that do not add up to the row count: flagged through the caller's status word, outputs -1
    ql = torch.tensor([3], dtype=torch.int32, device="cuda"); nm = torch.zeros_like(ql)
    acc = torch.zeros((1,), dtype=torch.int32, device="cuda"); bon = acc.clone()
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fd.fd_verify_accept_static(16, 1, 4, f, z, ql, nm, acc, bon, status)
    torch.cuda.synchronize()
    assert int(status) == fd.FD_DEV_BAD_LENGTHS and int(acc) == -1 and int(bon) == -1
    # and the next, well-formed call is unaffected by what that one left in the array
    ql4 = torch.tensor([4], dtype=torch.int32, device="cuda")
    f[2, 5] = 3.0
    fd.fd_verify_accept_static(16, 1, 4, f, z, ql4, nm, acc, bon, None)
    torch.cuda.synchronize()
    assert int(acc) == 2 and int(bon) == 5             # rows 0, 1: argmax 0 == next draft; row 2: argmax 5 != draft 0
