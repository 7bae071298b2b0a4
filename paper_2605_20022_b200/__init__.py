"""Python binding of libflexdraft (argument marshalling only).

Every function has the name and the argument order of its C entry point in
``include/flexdraft.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is
handed through unchanged.  All arithmetic runs inside the library's CUDA kernels.
If the library has not been built, or no CUDA device is present, the calls raise:
there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

from . import _build

FD_OK = 0
FD_ERR_INVALID_ARG, FD_ERR_UNSUPPORTED, FD_ERR_WORKSPACE, FD_ERR_CUDA, FD_ERR_DEVICE_STATUS = 1, 2, 3, 4, 5
FD_ERR_STATIC_LIMIT = 6
FD_STATIC_MAX_ROWS, FD_STATIC_MAX_BATCH = 4096, 4096
FD_DEV_BAD_LENGTHS, FD_DEV_BAD_PAGE, FD_DEV_TIMEOUT, FD_DEV_BAD_ACCEPT = 1, 2, 4, 8
FD_ATTN_AUTO, FD_ATTN_SIMT, FD_ATTN_TCGEN05 = 0, 1, 2
FD_ATTN_TCGEN05_PLANNED, FD_ATTN_TCGEN05_SELF_PLANNED = 3, 4
FD_TC_PLANNED, FD_TC_SELF_PLANNED, FD_TC_CLUSTER = 0, 1, 2

EXPORTS = ["fd_create", "fd_destroy", "fd_attn_draft_verify", "fd_verify_accept", "fd_kv_commit",
           "fd_last_device_status", "fd_attn_path", "fd_attn_last_mode", "fd_launch_count", "fd_status_string",
           "fd_verify_accept_static", "fd_host_reserve", "fd_step_host", "fd_step_host_append", "fd_step_device", "fd_selftest_wait_timeout", "fd_attn_draft_verify_blocks", "fd_select_branch", "fd_draft_select", "fd_kv_append", "fd_plan_pin", "fd_plan_unpin", "fd_calls_back_to_back", "fd_verify_accept_sample", "fd_plan_ranges_host"]


class fd_config(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
                ("page_size", ctypes.c_int), ("vocab", ctypes.c_int), ("max_batch", ctypes.c_int),
                ("max_q_len", ctypes.c_int), ("max_pages_per_seq", ctypes.c_int),
                ("softmax_scale", ctypes.c_float), ("attn_path", ctypes.c_int)]


class FlexDraftError(RuntimeError):
    def __init__(self, where: str, code: int):
        super().__init__(f"{where}: {status_string(code)} ({code})")
        self.code = code


_lib = None


def library_path() -> str:
    return _build.SO


def load() -> ctypes.CDLL:
    """dlopen libflexdraft.so (built in-tree by ``_build.build()``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.SO):
            raise FileNotFoundError(f"{_build.SO} is not built: run `python -m paper_2605_20022_b200._build`")
        lib = ctypes.CDLL(_build.SO)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.fd_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(fd_config)]
        lib.fd_destroy.argtypes = [vp]
        lib.fd_attn_draft_verify.argtypes = [vp, ci, ci, vp, vp, ci, vp, vp, vp, vp, vp, vp]
        lib.fd_verify_accept.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, vp, vp]
        lib.fd_kv_commit.argtypes = [vp, ci, vp, vp, vp, vp, vp, vp, vp]
        lib.fd_verify_accept_static.argtypes = [ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.fd_host_reserve.argtypes = [vp, ci, ci]
        lib.fd_selftest_wait_timeout.argtypes = [vp, ci, vp]
        lib.fd_attn_draft_verify_blocks.argtypes = [vp, ci, ci, vp, vp, ci, vp, vp, vp, vp, vp, vp, vp]
        lib.fd_select_branch.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.fd_verify_accept_sample.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
        lib.fd_plan_ranges_host.argtypes = [ci, ci, vp, vp, ci, vp]
        lib.fd_plan_pin.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp]
        lib.fd_plan_unpin.argtypes = [vp]
        lib.fd_calls_back_to_back.argtypes = [vp, ci]
        lib.fd_step_device.argtypes = [vp, ci, ci, ci, ci] + [ctypes.POINTER(vp)] * 5 + [ci] + [vp] * 12
        lib.fd_kv_append.argtypes = [vp, ci, ci, vp, vp, vp, ci, vp, vp, vp, vp]
        lib.fd_draft_select.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
        lib.fd_step_host.argtypes = [vp, ci, ci, ci, ci, ctypes.POINTER(vp), ci] + [vp] * 14
        lib.fd_step_host_append.argtypes = [vp, ci, ci, ci, ci, ctypes.POINTER(vp), ci] + [vp] * 16
        lib.fd_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
        lib.fd_attn_path.argtypes = [vp]
        lib.fd_attn_last_mode.argtypes = [vp]
        lib.fd_launch_count.argtypes = [vp]
        lib.fd_launch_count.restype = ctypes.c_int64
        lib.fd_status_string.argtypes = [ci]
        lib.fd_status_string.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().fd_status_string(int(code)).decode()


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(where: str, code: int, raise_on_error: bool) -> int:
    if code != FD_OK and raise_on_error:
        raise FlexDraftError(where, code)
    return code


def fd_create(n_q_heads: int, n_kv_heads: int, head_dim: int, vocab: int, max_batch: int, max_q_len: int,
              max_pages_per_seq: int, page_size: int = 16, softmax_scale: float = 0.0,
              attn_path: int = FD_ATTN_AUTO) -> int:
    """Returns the opaque context handle (an integer address)."""
    cfg = fd_config(n_q_heads, n_kv_heads, head_dim, page_size, vocab, max_batch, max_q_len, max_pages_per_seq,
                    softmax_scale, attn_path)
    ctx = ctypes.c_void_p()
    code = load().fd_create(ctypes.byref(ctx), ctypes.byref(cfg))
    _check("fd_create", code, True)
    return ctx.value


def fd_destroy(ctx: int) -> None:
    load().fd_destroy(ctx)


def fd_attn_draft_verify(ctx, batch, total_q_rows, q, kv_cache, num_pages, page_table, prefix_lens, q_lens, n_mask,
                         out, stream=None, raise_on_error=True) -> int:
    code = load().fd_attn_draft_verify(ctx, batch, total_q_rows, _ptr(q), _ptr(kv_cache), num_pages,
                                       _ptr(page_table), _ptr(prefix_lens), _ptr(q_lens), _ptr(n_mask), _ptr(out),
                                       _stream(stream))
    return _check("fd_attn_draft_verify", code, raise_on_error)


def fd_attn_draft_verify_blocks(ctx, batch, total_q_rows, q, kv_cache, num_pages, page_table, prefix_lens, q_lens, n_mask,
                                n_blocks, out, stream=None, raise_on_error=True) -> int:
    code = load().fd_attn_draft_verify_blocks(ctx, batch, total_q_rows, _ptr(q), _ptr(kv_cache), num_pages,
                                              _ptr(page_table), _ptr(prefix_lens), _ptr(q_lens), _ptr(n_mask),
                                              _ptr(n_blocks), _ptr(out), _stream(stream))
    return _check("fd_attn_draft_verify_blocks", code, raise_on_error)


def fd_verify_accept_sample(ctx, batch, total_cand_rows, logits, draft_logits, draft_tokens, q_lens, n_mask, temperature,
                            u_accept, u_bonus, accepted_len, bonus_token, stream=None, raise_on_error=True) -> int:
    code = load().fd_verify_accept_sample(ctx, batch, total_cand_rows, _ptr(logits), _ptr(draft_logits), _ptr(draft_tokens),
                                          _ptr(q_lens), _ptr(n_mask), float(temperature), _ptr(u_accept), _ptr(u_bonus),
                                          _ptr(accepted_len), _ptr(bonus_token), _stream(stream))
    return _check("fd_verify_accept_sample", code, raise_on_error)


def fd_plan_ranges_host(prefix_lens, q_lens, n_kv_heads: int, n_ranges: int):
    """Host-only: the first tile of each of the n_ranges ranges (+ the total), as a list of ints."""
    import numpy as np
    pl = np.ascontiguousarray(np.asarray(prefix_lens), dtype=np.int32); ql = np.ascontiguousarray(np.asarray(q_lens), dtype=np.int32)
    out = np.zeros((n_ranges + 1,), np.int32)
    code = load().fd_plan_ranges_host(int(pl.shape[0]), n_kv_heads, pl.ctypes.data, ql.ctypes.data, n_ranges, out.ctypes.data)
    _check("fd_plan_ranges_host", code, True)
    return out.tolist()


def fd_plan_pin(ctx, batch, total_q_rows, prefix_lens, q_lens, n_mask, n_blocks=None, stream=None, raise_on_error=True) -> int:
    code = load().fd_plan_pin(ctx, batch, total_q_rows, _ptr(prefix_lens), _ptr(q_lens), _ptr(n_mask), _ptr(n_blocks), _stream(stream))
    return _check("fd_plan_pin", code, raise_on_error)


def fd_plan_unpin(ctx, raise_on_error=True) -> int:
    return _check("fd_plan_unpin", load().fd_plan_unpin(ctx), raise_on_error)


def fd_kv_append(ctx, batch, total_q_rows, k_new, v_new, kv_cache, num_pages, page_table, prefix_lens, q_lens, stream=None,
                 raise_on_error=True) -> int:
    code = load().fd_kv_append(ctx, batch, total_q_rows, _ptr(k_new), _ptr(v_new), _ptr(kv_cache), num_pages,
                               _ptr(page_table), _ptr(prefix_lens), _ptr(q_lens), _stream(stream))
    return _check("fd_kv_append", code, raise_on_error)


def fd_draft_select(ctx, batch, total_mask_rows, max_blocks, draft_logits, bias, n_mask, n_blocks, threshold, mask_tokens,
                    mask_probs, keep_len, stream=None, raise_on_error=True) -> int:
    code = load().fd_draft_select(ctx, batch, total_mask_rows, max_blocks, _ptr(draft_logits), _ptr(bias), _ptr(n_mask),
                                  _ptr(n_blocks), float(threshold), _ptr(mask_tokens), _ptr(mask_probs), _ptr(keep_len),
                                  _stream(stream))
    return _check("fd_draft_select", code, raise_on_error)


def fd_select_branch(ctx, batch, max_block_len, mask_tokens, q_lens, n_mask, n_blocks, accepted_len, next_draft, next_len,
                     stream=None, raise_on_error=True) -> int:
    code = load().fd_select_branch(ctx, batch, max_block_len, _ptr(mask_tokens), _ptr(q_lens), _ptr(n_mask),
                                   _ptr(n_blocks), _ptr(accepted_len), _ptr(next_draft), _ptr(next_len), _stream(stream))
    return _check("fd_select_branch", code, raise_on_error)


def fd_verify_accept(ctx, batch, total_cand_rows, logits, draft_tokens, q_lens, n_mask, accepted_len, bonus_token,
                     stream=None, raise_on_error=True) -> int:
    code = load().fd_verify_accept(ctx, batch, total_cand_rows, _ptr(logits), _ptr(draft_tokens), _ptr(q_lens),
                                   _ptr(n_mask), _ptr(accepted_len), _ptr(bonus_token), _stream(stream))
    return _check("fd_verify_accept", code, raise_on_error)


def fd_verify_accept_static(vocab, batch, total_cand_rows, logits, draft_tokens, q_lens, n_mask, accepted_len,
                            bonus_token, device_status=None, stream=None, raise_on_error=True) -> int:
    """fd_verify_accept for callers that may not allocate: no context, scratch inside the library
    (at most FD_STATIC_MAX_ROWS candidate rows).  Calls sharing a device must not overlap on the GPU."""
    code = load().fd_verify_accept_static(vocab, batch, total_cand_rows, _ptr(logits), _ptr(draft_tokens), _ptr(q_lens),
                                          _ptr(n_mask), _ptr(accepted_len), _ptr(bonus_token), _ptr(device_status),
                                          _stream(stream))
    return _check("fd_verify_accept_static", code, raise_on_error)


def fd_kv_commit(ctx, batch, page_table, prefix_lens, q_lens, accepted_len, freed_pages, n_freed, stream=None,
                 raise_on_error=True) -> int:
    code = load().fd_kv_commit(ctx, batch, _ptr(page_table), _ptr(prefix_lens), _ptr(q_lens), _ptr(accepted_len),
                               _ptr(freed_pages), _ptr(n_freed), _stream(stream))
    return _check("fd_kv_commit", code, raise_on_error)


def fd_host_reserve(ctx, max_total_q_rows, max_total_cand_rows) -> None:
    _check("fd_host_reserve", load().fd_host_reserve(ctx, max_total_q_rows, max_total_cand_rows), True)


def fd_step_host(ctx, batch, total_q_rows, total_cand_rows, kv_caches, num_pages, q_host, out_host, logits_host,
                 draft_tokens_host, page_table_host, prefix_lens_host, q_lens_host, n_mask_host, accepted_len_host,
                 bonus_token_host, freed_pages_host, n_freed_host, stream=None, raise_on_error=True,
                 n_blocks_host=None) -> int:
    """One whole step from host (CPU, ideally pinned) tensors; `kv_caches` is a list of device tensors, one per
    layer.  `q_host` / `out_host` are [n_layers, T, Hq, d] CPU tensors."""
    n_layers = len(kv_caches)
    arr = (ctypes.c_void_p * n_layers)(*[_ptr(t) for t in kv_caches])
    code = load().fd_step_host(ctx, batch, total_q_rows, total_cand_rows, n_layers, arr, num_pages, _ptr(q_host),
                               _ptr(out_host), _ptr(logits_host), _ptr(draft_tokens_host), _ptr(page_table_host),
                               _ptr(prefix_lens_host), _ptr(q_lens_host), _ptr(n_mask_host), _ptr(n_blocks_host),
                               _ptr(accepted_len_host),
                               _ptr(bonus_token_host), _ptr(freed_pages_host), _ptr(n_freed_host), _stream(stream))
    return _check("fd_step_host", code, raise_on_error)


def fd_step_host_append(ctx, batch, total_q_rows, total_cand_rows, kv_caches, num_pages, q_host, k_new_host, v_new_host, out_host,
                        logits_host, draft_tokens_host, page_table_host, prefix_lens_host, q_lens_host, n_mask_host,
                        accepted_len_host, bonus_token_host, freed_pages_host, n_freed_host, stream=None, raise_on_error=True,
                        n_blocks_host=None) -> int:
    """fd_step_host with the KV append inside: `k_new_host` / `v_new_host` are [n_layers, T, Hkv, d] CPU tensors."""
    n_layers = len(kv_caches)
    arr = (ctypes.c_void_p * n_layers)(*[_ptr(t) for t in kv_caches])
    code = load().fd_step_host_append(ctx, batch, total_q_rows, total_cand_rows, n_layers, arr, num_pages, _ptr(q_host),
                                      _ptr(k_new_host), _ptr(v_new_host), _ptr(out_host), _ptr(logits_host),
                                      _ptr(draft_tokens_host), _ptr(page_table_host), _ptr(prefix_lens_host),
                                      _ptr(q_lens_host), _ptr(n_mask_host), _ptr(n_blocks_host), _ptr(accepted_len_host),
                                      _ptr(bonus_token_host), _ptr(freed_pages_host), _ptr(n_freed_host), _stream(stream))
    return _check("fd_step_host_append", code, raise_on_error)


def fd_ptr_array(tensors):
    """A host array of the device addresses of `tensors` (for fd_step_device: build once, pass every step)."""
    return (ctypes.c_void_p * len(tensors))(*[_ptr(t) for t in tensors])


def fd_step_device(ctx, batch, total_q_rows, total_cand_rows, q, k_new, v_new, kv_caches, out, num_pages, page_table, prefix_lens,
                   q_lens, n_mask, n_blocks, logits, draft_tokens, accepted_len, bonus_token, freed_pages, n_freed, stream=None,
                   raise_on_error=True) -> int:
    """One step on device buffers.  q, k_new, v_new, kv_caches, out: lists of per-layer tensors, or arrays from fd_ptr_array."""
    arr = lambda x: None if x is None else (x if isinstance(x, ctypes.Array) else fd_ptr_array(x))
    qa, ka, va, kva, oa = arr(q), arr(k_new), arr(v_new), arr(kv_caches), arr(out)
    code = load().fd_step_device(ctx, batch, total_q_rows, total_cand_rows, len(kva), qa, ka, va, kva, oa, num_pages, _ptr(page_table),
                                 _ptr(prefix_lens), _ptr(q_lens), _ptr(n_mask), _ptr(n_blocks), _ptr(logits), _ptr(draft_tokens),
                                 _ptr(accepted_len), _ptr(bonus_token), _ptr(freed_pages), _ptr(n_freed), _stream(stream))
    return _check("fd_step_device", code, raise_on_error)


def fd_selftest_wait_timeout(ctx, limit_ms, stream=None) -> None:
    _check("fd_selftest_wait_timeout", load().fd_selftest_wait_timeout(ctx, limit_ms, _stream(stream)), True)


def fd_last_device_status(ctx, stream=None) -> int:
    code = ctypes.c_int32(0)
    _check("fd_last_device_status", load().fd_last_device_status(ctx, ctypes.byref(code), _stream(stream)), True)
    return code.value


def fd_calls_back_to_back(ctx, on=True) -> int:
    return _check("fd_calls_back_to_back", load().fd_calls_back_to_back(ctx, 1 if on else 0), True)


def fd_attn_path(ctx) -> int:
    return load().fd_attn_path(ctx)


def fd_attn_last_mode(ctx) -> int:
    return load().fd_attn_last_mode(ctx)


def fd_launch_count(ctx) -> int:
    return int(load().fd_launch_count(ctx))
