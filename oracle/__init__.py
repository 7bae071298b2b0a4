"""CPU oracle for the FlexDraft decode-step hot path (test infrastructure only).

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product path never does.  The arithmetic lives in
``fd_oracle.c`` (plain float64 C, OpenMP over independent output rows); this file
only compiles it with gcc and marshals numpy / torch CPU arrays into it.

Functions
---------
attn(...)        full attention under the hybrid mask (Sec. 4.1), float64 output
attn_row(...)    one output row of the same definition (sampled checks)
attn_blocks(...) the same with several mask blocks per sequence (all hypotheses, Eq. 2)
select_branch(...) pick the prepared next-draft branch of the accepted length
kv_append(...)   write the query block's K/V into its pages (append, then attend)
draft_select(...) draft-side tail: calibrated argmax, confidence, Eq. 5 verify length
accept_stochastic(...) verification by speculative sampling at temperature > 0 (Sec. 3)
accept(...)      greedy verification: argmax, accepted length, bonus token (Sec. 3)
commit(...)      KV commit / rollback by page-table truncation
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# FD_ORACLE_SRC: a test hook.  tests/test_oracle_mutants.py points it at a copy of the source with one mistake planted
# in it and checks that the pins notice; nothing else sets it.
_SRC = os.environ.get("FD_ORACLE_SRC") or os.path.join(_HERE, "fd_oracle.c")
_SO = (_SRC + ".so") if os.environ.get("FD_ORACLE_SRC") else os.path.join(_HERE, "libfd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile fd_oracle.c with gcc (-O2, OpenMP).  Returns the path of the library."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.fdo_num_threads.restype = ctypes.c_int
        _lib.fdo_commit.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().fdo_num_threads())


def _bits(t) -> np.ndarray:
    """bf16 torch CPU tensor (or uint16 numpy array) -> contiguous uint16 bit pattern."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy().view(np.uint16))


def _i32(t) -> np.ndarray:
    if not isinstance(t, np.ndarray):
        t = t.cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.int32)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def attn(q, kv_cache, page_table, prefix_lens, q_lens, n_mask, scale=None) -> np.ndarray:
    """q [T,Hq,d] bf16, kv_cache [pages,2,Hkv,P,d] bf16 -> out [T,Hq,d] float64."""
    qb, kvb = _bits(q), _bits(kv_cache)
    T, Hq, d = qb.shape
    _, two, Hkv, P, d2 = kvb.shape
    assert two == 2 and d2 == d
    pt, pl, ql, nm = _i32(page_table), _i32(prefix_lens), _i32(q_lens), _i32(n_mask)
    B = pl.shape[0]
    assert int(ql.sum()) == T
    out = np.zeros((T, Hq, d), dtype=np.float64)
    s = float(scale) if scale else 1.0 / float(np.sqrt(d))
    _load().fdo_attn(ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
                     ctypes.c_int(P), ctypes.c_int(pt.shape[1]), _p(qb), _p(kvb), _p(pt), _p(pl), _p(ql),
                     _p(nm), ctypes.c_double(s), _p(out))
    return out


def attn_blocks(q, kv_cache, page_table, prefix_lens, q_lens, n_mask, n_blocks, scale=None) -> np.ndarray:
    """Attention with several mask blocks per sequence (all-hypotheses parallel drafting, Eq. 2)."""
    qb, kvb = _bits(q), _bits(kv_cache)
    T, Hq, d = qb.shape
    _, two, Hkv, P, d2 = kvb.shape
    pt, pl, ql, nm, nb = _i32(page_table), _i32(prefix_lens), _i32(q_lens), _i32(n_mask), _i32(n_blocks)
    B = pl.shape[0]
    assert int(ql.sum()) == T
    out = np.zeros((T, Hq, d), dtype=np.float64)
    s = float(scale) if scale else 1.0 / float(np.sqrt(d))
    _load().fdo_attn_blocks(ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(P),
                            ctypes.c_int(pt.shape[1]), _p(qb), _p(kvb), _p(pt), _p(pl), _p(ql), _p(nm), _p(nb),
                            ctypes.c_double(s), _p(out))
    return out


def select_branch(mask_tokens, q_lens, n_mask, n_blocks, accepted_len, max_kb):
    """Returns (next_draft [B, max_kb] padded with -1, next_len [B])."""
    mt, ql, nm, nb, acc = _i32(mask_tokens), _i32(q_lens), _i32(n_mask), _i32(n_blocks), _i32(accepted_len)
    B = ql.shape[0]
    nd = np.zeros((B, max_kb), np.int32)
    nl = np.zeros((B,), np.int32)
    _load().fdo_select_branch(ctypes.c_int(B), ctypes.c_int(max_kb), _p(mt), _p(ql), _p(nm), _p(nb), _p(acc), _p(nd), _p(nl))
    return nd, nl


def attn_row(q, kv_cache, page_table, prefix_lens, q_lens, n_mask, b, i, h, scale=None) -> np.ndarray:
    """One output row out[d] (sequence b, block row i, q-head h) of the same definition."""
    qb, kvb = _bits(q), _bits(kv_cache)
    T, Hq, d = qb.shape
    _, two, Hkv, P, _ = kvb.shape
    pt, pl, ql, nm = _i32(page_table), _i32(prefix_lens), _i32(q_lens), _i32(n_mask)
    out = np.zeros((d,), dtype=np.float64)
    s = float(scale) if scale else 1.0 / float(np.sqrt(d))
    _load().fdo_attn_row(ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(P),
                         ctypes.c_int(pt.shape[1]), _p(qb), _p(kvb), _p(pt), _p(pl), _p(ql), _p(nm),
                         ctypes.c_double(s), ctypes.c_int(b), ctypes.c_int(i), ctypes.c_int(h), _p(out))
    return out


def accept(logits, draft_tokens, q_lens, n_mask):
    """logits [R,V] fp32 -> (accepted_len [B], bonus_token [B], argmax [R]) int32."""
    lg = logits if isinstance(logits, np.ndarray) else logits.cpu().numpy()
    lg = np.ascontiguousarray(lg, dtype=np.float32)
    R, V = lg.shape
    dt, ql, nm = _i32(draft_tokens), _i32(q_lens), _i32(n_mask)
    B = ql.shape[0]
    assert int(np.maximum(ql - nm, 0).sum()) == R and dt.shape[0] == R
    acc = np.zeros((B,), np.int32)
    bon = np.zeros((B,), np.int32)
    am = np.zeros((max(R, 1),), np.int32)
    _load().fdo_accept(ctypes.c_int(B), ctypes.c_int(V), _p(lg), _p(dt), _p(ql), _p(nm), _p(acc), _p(bon), _p(am))
    return acc, bon, am[:R]


def accept_stochastic(logits, draft_logits, draft_tokens, q_lens, n_mask, temperature, u_accept, u_bonus, want_weights=False):
    """Speculative sampling (Sec. 3).  Returns (accepted_len [B], bonus_token [B], ratio [R] f64[, weights [B,V] f64])."""
    lg = np.ascontiguousarray(logits if isinstance(logits, np.ndarray) else logits.cpu().numpy(), dtype=np.float32)
    dl = None if draft_logits is None else np.ascontiguousarray(
        draft_logits if isinstance(draft_logits, np.ndarray) else draft_logits.cpu().numpy(), dtype=np.float32)
    R, V = lg.shape
    dt, ql, nm = _i32(draft_tokens), _i32(q_lens), _i32(n_mask)
    ua = np.ascontiguousarray(u_accept if isinstance(u_accept, np.ndarray) else u_accept.cpu().numpy(), dtype=np.float32)
    ub = np.ascontiguousarray(u_bonus if isinstance(u_bonus, np.ndarray) else u_bonus.cpu().numpy(), dtype=np.float32)
    B = ql.shape[0]
    assert int(np.maximum(ql - nm, 0).sum()) == R and dt.shape[0] == R and ua.shape[0] == R and ub.shape[0] == B
    assert dl is None or dl.shape == lg.shape
    acc = np.zeros((B,), np.int32); bon = np.zeros((B,), np.int32)
    ratio = np.zeros((max(R, 1),), np.float64)
    w = np.zeros((B, V), np.float64) if want_weights else None
    _load().fdo_accept_stochastic(ctypes.c_int(B), ctypes.c_int(V), _p(lg), None if dl is None else _p(dl), _p(dt), _p(ql), _p(nm),
                                  ctypes.c_double(temperature), _p(ua), _p(ub), _p(acc), _p(bon), _p(ratio),
                                  None if w is None else _p(w))
    return (acc, bon, ratio[:R], w) if want_weights else (acc, bon, ratio[:R])


def draft_select(logits, bias, n_mask, n_blocks, threshold, max_blocks, want_gap=False):
    """Draft-side tail (Eq. 4 + Eq. 5): returns (tokens [Rm] i32, probs [Rm] f64, cum [Rm] f64, keep_len [B, max_blocks] i32),
    and with want_gap also the margin [Rm] f64 by which each row's winning calibrated logit beats the best other one."""
    lg = np.ascontiguousarray(logits if isinstance(logits, np.ndarray) else logits.cpu().numpy(), dtype=np.float32)
    bs = None if bias is None else np.ascontiguousarray(bias if isinstance(bias, np.ndarray) else bias.cpu().numpy(), dtype=np.float32)
    Rm, V = lg.shape
    nm = _i32(n_mask)
    nb = None if n_blocks is None else _i32(n_blocks)
    B = nm.shape[0]
    assert int(np.maximum(nm, 0).sum()) == Rm
    tok = np.zeros((max(Rm, 1),), np.int32); pr = np.zeros((max(Rm, 1),), np.float64); cum = np.zeros((max(Rm, 1),), np.float64)
    gap = np.zeros((max(Rm, 1),), np.float64)
    keep = np.zeros((B, max_blocks), np.int32)
    _load().fdo_draft_select(ctypes.c_int(B), ctypes.c_int(V), ctypes.c_int(max_blocks), _p(lg), None if bs is None else _p(bs), _p(nm),
                             None if nb is None else _p(nb), ctypes.c_double(threshold), _p(tok), _p(pr), _p(cum), _p(keep), _p(gap))
    if want_gap:
        return tok[:Rm], pr[:Rm], cum[:Rm], keep, gap[:Rm]
    return tok[:Rm], pr[:Rm], cum[:Rm], keep


def kv_append(k_new, v_new, kv_cache, page_table, prefix_lens, q_lens):
    """Returns a copy of kv_cache (uint16 bit pattern, same shape) with the query block's K/V written in."""
    kb, vb = _bits(k_new), _bits(v_new)
    kv = _bits(kv_cache).copy()
    T, Hkv, d = kb.shape
    P = kv.shape[3]
    pt, pl, ql = _i32(page_table), _i32(prefix_lens), _i32(q_lens)
    assert int(ql.sum()) == T and vb.shape == kb.shape
    _load().fdo_kv_append(ctypes.c_int(pl.shape[0]), ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(P), ctypes.c_int(pt.shape[1]),
                          _p(kb), _p(vb), _p(kv), _p(pt), _p(pl), _p(ql))
    return kv


def commit(page_table, prefix_lens, q_lens, accepted_len, page_size=16):
    """Returns (new_page_table, new_prefix_lens, freed_pages[0:n_freed]); inputs untouched."""
    pt = _i32(page_table).copy()
    pl = _i32(prefix_lens).copy()
    ql, acc = _i32(q_lens), _i32(accepted_len)
    B, maxp = pt.shape
    freed = np.full((B * maxp + 1,), -7, np.int32)
    n = _load().fdo_commit(ctypes.c_int(B), ctypes.c_int(page_size), ctypes.c_int(maxp), _p(pt), _p(pl), _p(ql),
                           _p(acc), _p(freed))
    return pt, pl, freed[:n].copy()
