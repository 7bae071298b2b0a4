"""Seeded synthetic inputs for the draft-verify decode step.

This module only *draws* inputs (lengths, page tables, bf16 Q/K/V, fp32 logits,
draft tokens); it contains none of the method's arithmetic, and both the CUDA
path and the CPU checker are handed the very same tensors.  The shapes are the
five benchmark workloads (Qwen3-8B attention shape, 16-token bf16 KV pages,
vocab 151 936); the values are iid N(0,1).  They stand in for the paper's real
workloads (Qwen3 checkpoints decoding benchmark prompts), which need trained
weights and datasets.

Recipe
------
* base seed 20022; workload ``c`` (0-based) uses ``20022 + 1000*(c+1)``, layer
  ``l`` adds ``l``; lengths come from a CPU generator, so they do not depend on
  the device the tensors are drawn on.
* page pool = sum_b ceil(kv_len_b/16) + 64 spare pages; physical ids are a seeded
  random permutation (a shuffled page table); entries beyond a sequence's
  allocation are -1.
* every KV slot that no valid token owns (spare pages, the tail of each last
  page) is overwritten with a poison value (1e30, or NaN on request) so that a
  kernel reading past ``kv_len`` shows up in the output.
* logits are N(0,1) fp32 with ONE planted peak per candidate row (value in
  [6, 7), far above the N(0,1) maximum over the vocabulary), so the target token
  of every row is known by construction.  Drafts equal the target token of the
  previous row with probability ``p_match``; otherwise they are a different
  token drawn uniformly.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

BASE_SEED = 20022
PAGE = 16


@dataclass(frozen=True)
class Shape:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    n_layers: int = 1
    page_size: int = PAGE


QWEN3_8B = Shape(32, 8, 128, 151936, 1)
TINY = Shape(4, 1, 64, 1000, 1)

WORKLOAD_NAMES = [
    "tiny_b1_prefix128_c5_m4",
    "qwen3_8b_b1_prefix2048_c16_m16",
    "qwen3_8b_b8_parallel_ragged",
    "qwen3_8b_b64_sequential_ragged",
    "qwen3_8b_b16_prefix32768_36layers",
    "qwen3_8b_b8_all_hypotheses_c4_4x7",
    "qwen3_8b_b64_sequential_draft_pass",
    "qwen3_8b_b4_all_17_hypotheses_k16",
]


@dataclass
class Step:
    """Lengths + page table of one decode step (CPU int32 tensors)."""
    name: str
    shape: Shape
    seed: int
    p_match: float
    prefix_lens: torch.Tensor
    q_lens: torch.Tensor
    n_mask: torch.Tensor
    page_table: torch.Tensor          # [B, max_pages_per_seq], -1 = unallocated
    num_pages: int
    spare_pages: torch.Tensor = field(default=None)  # physical ids owned by no sequence
    n_blocks: Optional[torch.Tensor] = None          # [B] mask blocks per sequence (None = one block each)

    @property
    def batch(self) -> int:
        return int(self.prefix_lens.numel())

    @property
    def total_q_rows(self) -> int:
        return int(self.q_lens.sum())

    @property
    def cand_rows(self) -> torch.Tensor:
        return (self.q_lens - self.n_mask).clamp(min=0)

    @property
    def total_cand_rows(self) -> int:
        return int(self.cand_rows.sum())

    @property
    def kv_lens(self) -> torch.Tensor:
        return self.prefix_lens + self.q_lens

    @property
    def max_pages_per_seq(self) -> int:
        return int(self.page_table.shape[1])

    def attn_bytes(self) -> int:
        """Algorithmic bytes of one attention call: every valid KV token once + Q + O."""
        s = self.shape
        kv = int(self.kv_lens.sum()) * 2 * s.n_kv_heads * s.head_dim * 2
        qo = 2 * self.total_q_rows * s.n_q_heads * s.head_dim * 2
        return kv + qo

    def logits_bytes(self) -> int:
        return self.total_cand_rows * self.shape.vocab * 4


def _cpu_gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def _randint(g, lo: int, hi: int, n: int) -> torch.Tensor:
    """n integers uniform in [lo, hi] (inclusive)."""
    return torch.randint(lo, hi + 1, (n,), generator=g, dtype=torch.int64).to(torch.int32)


def make_step(name: str, shape: Shape, prefix_lens: Sequence[int], q_lens: Sequence[int],
              n_mask: Sequence[int], seed: int, p_match: float = 0.8, spare: int = 64,
              extra_table_cols: int = 0, shuffle: bool = True) -> Step:
    """Build the page table for given lengths: a seeded permutation of the pool."""
    pl = torch.as_tensor(list(prefix_lens), dtype=torch.int32)
    ql = torch.as_tensor(list(q_lens), dtype=torch.int32)
    nm = torch.as_tensor(list(n_mask), dtype=torch.int32)
    P = shape.page_size
    need = ((pl + ql + P - 1) // P).to(torch.int64)
    num_pages = int(need.sum()) + spare
    g = _cpu_gen(seed + 7)
    ids = torch.randperm(num_pages, generator=g) if shuffle else torch.arange(num_pages)
    max_pages = int(need.max()) + extra_table_cols if need.numel() else 1
    max_pages = max(max_pages, 1)
    table = torch.full((pl.numel(), max_pages), -1, dtype=torch.int32)
    off = 0
    for b in range(pl.numel()):
        nb = int(need[b])
        table[b, :nb] = ids[off:off + nb].to(torch.int32)
        off += nb
    return Step(name, shape, seed, p_match, pl, ql, nm, table, num_pages, ids[off:].to(torch.int64))


def workload(idx: int, n_layers: Optional[int] = None) -> Step:
    """The benchmark workload ``idx`` (0..4), or one of the extra ones (5, 6, 7)."""
    seed = BASE_SEED + 1000 * (idx + 1)
    g = _cpu_gen(seed)
    if idx == 0:
        return make_step(WORKLOAD_NAMES[0], TINY, [128], [9], [4], seed, p_match=0.7)
    if idx == 1:
        return make_step(WORKLOAD_NAMES[1], QWEN3_8B, [2048], [32], [16], seed, p_match=0.8)
    if idx == 2:
        B = 8
        n = _randint(g, 512, 8192, B)
        c = _randint(g, 4, 16, B)            # confidence-truncated verify length, bonus row included
        m = torch.full((B,), 16, dtype=torch.int32)
        return make_step(WORKLOAD_NAMES[2], QWEN3_8B, n.tolist(), (c + m).tolist(), m.tolist(), seed, 0.8)
    if idx == 3:
        B = 64
        n = _randint(g, 1024, 4096, B)
        c = _randint(g, 1, 16, B)
        m = torch.zeros((B,), dtype=torch.int32)
        return make_step(WORKLOAD_NAMES[3], QWEN3_8B, n.tolist(), c.tolist(), m.tolist(), seed, 0.75)
    if idx == 4:
        B = 16
        shape = Shape(32, 8, 128, 151936, 36 if n_layers is None else n_layers)
        return make_step(WORKLOAD_NAMES[4], shape, [32768] * B, [32] * B, [16] * B, seed, 0.8)
    if idx == 5:
        # beyond the five benchmark configurations: the all-hypotheses form of parallel drafting at the size one
        # M = 128 tile allows: bonus + 3 drafts, and one 7-token next-draft branch per hypothesis r = 0..3
        B = 8
        n = _randint(g, 512, 8192, B)
        st = make_step(WORKLOAD_NAMES[5], QWEN3_8B, n.tolist(), [32] * B, [28] * B, seed, 0.8)
        st.n_blocks = torch.full((B,), 4, dtype=torch.int32)
        return st
    if idx == 6:
        # beyond the five benchmark configurations: the draft pass of sequential mode on its own -- the resolved
        # bonus token and 16 mask tokens against the committed KV of the batch-64 workload (one candidate row,
        # so the accept call that follows only turns that row's argmax into the next bonus token)
        B = 64
        n = _randint(g, 1024, 4096, B)
        return make_step(WORKLOAD_NAMES[6], QWEN3_8B, n.tolist(), [17] * B, [16] * B, seed, 0.75)
    if idx == 7:
        # beyond the five benchmark configurations: the paper's parallel mode in full -- bonus + 16 drafts, and one
        # 16-token next-draft branch for every hypothesis r = 0..16 (Eq. 2): 289 query rows per sequence, which the
        # kernels process as ten row blocks of 32 block rows, each streaming the sequence's KV
        B = 4
        n = _randint(g, 512, 8192, B)
        st = make_step(WORKLOAD_NAMES[7], QWEN3_8B, n.tolist(), [289] * B, [272] * B, seed, 0.8)
        st.n_blocks = torch.full((B,), 17, dtype=torch.int32)
        return st
    raise ValueError(f"no workload {idx}")


def _dev_gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_q(step: Step, layer: int = 0, device="cpu") -> torch.Tensor:
    """q [T, Hq, d] bf16, iid N(0,1)."""
    s = step.shape
    g = _dev_gen(device, step.seed + 100_000 + layer)
    return torch.randn((step.total_q_rows, s.n_q_heads, s.head_dim), generator=g, device=device,
                       dtype=torch.float32).to(torch.bfloat16)


def make_kv(step: Step, layer: int = 0, device="cpu", poison: float = 1e30) -> torch.Tensor:
    """kv_cache [num_pages, 2, Hkv, 16, d] bf16, iid N(0,1); unowned slots poisoned."""
    s = step.shape
    g = _dev_gen(device, step.seed + 200_000 + layer)
    kv = torch.empty((step.num_pages, 2, s.n_kv_heads, s.page_size, s.head_dim), device=device,
                     dtype=torch.bfloat16)
    chunk = 4096                                    # pages per draw keeps the fp32 temporary small
    for p0 in range(0, step.num_pages, chunk):
        p1 = min(step.num_pages, p0 + chunk)
        kv[p0:p1] = torch.randn((p1 - p0,) + tuple(kv.shape[1:]), generator=g, device=device,
                                dtype=torch.float32).to(torch.bfloat16)
    if poison is not None:
        if step.spare_pages is not None and step.spare_pages.numel():
            kv[step.spare_pages.to(device)] = poison
        P = s.page_size
        for b in range(step.batch):
            L = int(step.kv_lens[b])
            if L % P:
                kv[int(step.page_table[b, L // P]), :, :, L % P:, :] = poison
    return kv


def make_logits(step: Step, device="cpu"):
    """(logits [R,V] fp32, draft_tokens [R] i32, target [R] i32).

    ``target[r]`` is the index of the planted peak of row r (the row's argmax by
    construction).  ``draft_tokens[r]`` is the token fed at candidate row r: row 0
    of a sequence is the previous bonus token (any token), row j+1 repeats
    ``target`` of row j with probability ``p_match``.
    """
    s = step.shape
    R, V = step.total_cand_rows, s.vocab
    g = _dev_gen(device, step.seed + 300_000)
    logits = torch.empty((R, V), device=device, dtype=torch.float32)
    for r0 in range(0, R, 64):
        r1 = min(R, r0 + 64)
        logits[r0:r1] = torch.randn((r1 - r0, V), generator=g, device=device, dtype=torch.float32)
    gc = _cpu_gen(step.seed + 300_001)
    target = torch.randint(0, V, (R,), generator=gc, dtype=torch.int64)
    peak = 6.0 + torch.rand((R,), generator=gc, dtype=torch.float32)
    if R:
        logits[torch.arange(R, device=device), target.to(device)] = peak.to(device)
    match = torch.rand((R,), generator=gc) < step.p_match
    other = (target + 1 + torch.randint(0, max(V - 1, 1), (R,), generator=gc, dtype=torch.int64)) % V
    drafts = torch.empty((R,), dtype=torch.int64)
    r = 0
    for b in range(step.batch):
        C = int(step.cand_rows[b])
        if C == 0:
            continue
        drafts[r] = int(torch.randint(0, V, (1,), generator=gc))
        for j in range(C - 1):
            drafts[r + j + 1] = target[r + j] if bool(match[r + j]) else other[r + j]
        r += C
    return logits, drafts.to(torch.int32), target.to(torch.int32)


def query_block_kv(step: Step, kv: torch.Tensor):
    """(k_new, v_new) [T, Hkv, d]: the K/V rows of every sequence's query block, read out of a cache that already
    holds them (positions n_b .. n_b + Lq_b - 1, through the page table) -- what the projections of the step would hand
    to the KV append.  Pure indexing; `kv` may live on any device."""
    seq = torch.repeat_interleave(torch.arange(step.batch), step.q_lens.long())
    start = torch.cumsum(step.q_lens.long(), 0) - step.q_lens.long()
    pos = step.prefix_lens.long()[seq] + (torch.arange(step.total_q_rows) - start[seq])
    pages = step.page_table.long()[seq, pos // step.shape.page_size].to(kv.device)
    slots = (pos % step.shape.page_size).to(kv.device)
    return kv[pages, 0, :, slots, :].contiguous(), kv[pages, 1, :, slots, :].contiguous()
