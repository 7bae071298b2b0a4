"""Shared plumbing of the GPU parity tests: move a seeded step to the device, call the
C ABI through the binding, bring results back."""
import numpy as np
import torch

import paper_2605_20022_b200 as fd

ATOL, RTOL = 2e-2, 2e-2      # bf16 attention outputs: |gpu - ref| <= 2e-2 + 2e-2 |ref|


class Ctx:
    """fd_create / fd_destroy as a context manager, sized for one Step."""

    def __init__(self, step, attn_path=fd.FD_ATTN_AUTO, max_batch=None, max_q_len=None, scale=0.0):
        s = step.shape
        G = s.n_q_heads // s.n_kv_heads
        self.step = step
        self.h = fd.fd_create(s.n_q_heads, s.n_kv_heads, s.head_dim, s.vocab,
                              max_batch or max(step.batch, 1), max_q_len or min(128 // G, 32),
                              step.max_pages_per_seq, s.page_size, scale, attn_path)

    def __enter__(self):
        return self

    def __exit__(self, *a):
        fd.fd_destroy(self.h)


def dev(t):
    return t.cuda()


def gpu_attn(ctx, step, q, kv, page_table=None, lens=None):
    """Returns out [T,Hq,d] as a float32 CPU tensor and the device status word."""
    pl, ql, nm = lens if lens is not None else (step.prefix_lens, step.q_lens, step.n_mask)
    pt = step.page_table if page_table is None else page_table
    dq, dkv, dpt, dpl, dql, dnm = dev(q), dev(kv), dev(pt), dev(pl), dev(ql), dev(nm)
    out = torch.full_like(dq, float("nan"))
    fd.fd_attn_draft_verify(ctx.h, int(pl.numel()), int(q.shape[0]), dq, dkv, int(kv.shape[0]), dpt, dpl, dql, dnm, out)
    status = fd.fd_last_device_status(ctx.h)
    return out.float().cpu(), status


def assert_close(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    bound = ATOL + RTOL * np.abs(ref)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    worst = float((err - bound).max()) if err.size else -1.0
    assert worst <= 0, f"{what}: max |err| {err.max():.4g}, worst excess over tolerance {worst:.4g}"


def worst_vector_error(got, ref):
    """Largest error of a (row, head) output vector relative to the vector's own length.  At long contexts an output
    element averages tens of thousands of values and is small against the elementwise tolerance, which a lost tile would
    pass; the vector's relative error shows it (tests/test_comparison_bounds.py measures both)."""
    got = np.asarray(got, dtype=np.float64)
    return float((np.linalg.norm(got - ref, axis=-1) / np.linalg.norm(ref, axis=-1)).max())


def gpu_accept(ctx, step, logits, drafts, lens=None):
    ql, nm = lens if lens is not None else (step.q_lens, step.n_mask)
    B = int(ql.numel())
    acc = torch.full((max(B, 1),), -99, dtype=torch.int32, device="cuda")
    bon = torch.full((max(B, 1),), -99, dtype=torch.int32, device="cuda")
    fd.fd_verify_accept(ctx.h, B, int(logits.shape[0]), dev(logits), dev(drafts), dev(ql), dev(nm), acc, bon)
    status = fd.fd_last_device_status(ctx.h)
    return acc[:B].cpu().numpy(), bon[:B].cpu().numpy(), status


def gpu_commit(ctx, step, accepted, page_table=None, prefix_lens=None, q_lens=None):
    pt = dev((step.page_table if page_table is None else page_table).clone())
    pl = dev((step.prefix_lens if prefix_lens is None else prefix_lens).clone())
    ql = dev(step.q_lens if q_lens is None else q_lens)
    B = int(pl.numel())
    freed = torch.full((B * 4 + 8,), -7, dtype=torch.int32, device="cuda")
    n_freed = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    fd.fd_kv_commit(ctx.h, B, pt, pl, ql, dev(torch.as_tensor(accepted, dtype=torch.int32)), freed, n_freed)
    status = fd.fd_last_device_status(ctx.h)
    n = int(n_freed.item())
    return pt.cpu().numpy(), pl.cpu().numpy(), freed[:n].cpu().numpy(), status
