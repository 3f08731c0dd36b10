"""ctypes binding of ``include/spf.h``: argument marshalling only.

The functions named ``spf_*`` mirror the C entry points one to one and take torch CUDA tensors
(used here as device buffers) instead of raw pointers.  ``Selector`` chains the four calls for one
prompt and owns the scratch buffers a serving loop would reuse.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import List, Optional, Sequence

import torch

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG_DIR, "libspf.so")


class SpfError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where}: status {status} ({detail})")
        self.status = status


class _Shape(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("n_lookahead", ctypes.c_int32), ("softmax_scale", ctypes.c_float)]


class _Prompt(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int64), ("k_layers", ctypes.POINTER(ctypes.c_void_p)),
                ("k_stride_head", ctypes.c_int64), ("k_stride_tok", ctypes.c_int64), ("q", ctypes.c_void_p),
                ("importance", ctypes.c_void_p), ("lse", ctypes.c_void_p)]


class _Fp8Prompt(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int64), ("k_layers", ctypes.POINTER(ctypes.c_void_p)),
                ("k_stride_head", ctypes.c_int64), ("k_stride_tok", ctypes.c_int64), ("k_scale", ctypes.c_void_p),
                ("q", ctypes.c_void_p), ("importance", ctypes.c_void_p), ("lse", ctypes.c_void_p)]


class _PoolItem(ctypes.Structure):
    _fields_ = [("importance", ctypes.c_void_p), ("n_tokens", ctypes.c_int64), ("chunk_scores", ctypes.c_void_p)]


class _TopkItem(ctypes.Structure):
    _fields_ = [("chunk_scores", ctypes.c_void_p), ("n_chunks", ctypes.c_int64), ("k", ctypes.c_int64),
                ("kept_chunks", ctypes.c_void_p)]


class _CompactItem(ctypes.Structure):
    _fields_ = [("kept_chunks", ctypes.c_void_p), ("k", ctypes.c_int64), ("n_tokens", ctypes.c_int64),
                ("token_ids", ctypes.c_void_p), ("char_start", ctypes.c_void_p), ("char_end", ctypes.c_void_p),
                ("out_ids", ctypes.c_void_p), ("out_pos", ctypes.c_void_p), ("out_tok_spans", ctypes.c_void_p),
                ("out_char_spans", ctypes.c_void_p), ("out_counts", ctypes.c_void_p)]


class _SelectParams(ctypes.Structure):
    _fields_ = [("chunk", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("keep_ratio", ctypes.c_double)]


class _PagedPrompt(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int64), ("k_pools", ctypes.POINTER(ctypes.c_void_p)),
                ("n_pool_blocks", ctypes.c_int64), ("block_tokens", ctypes.c_int32), ("block_table", ctypes.c_void_p),
                ("q", ctypes.c_void_p), ("importance", ctypes.c_void_p), ("lse", ctypes.c_void_p)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_02631_b200.build` "
                          "(there is no fallback path)")
    dll = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    dll.spf_score_workspace_bytes.restype = ctypes.c_size_t
    dll.spf_score_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), i32]
    dll.spf_score.restype = i32
    dll.spf_score.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), i32, vp, ctypes.c_size_t, vp, vp]
    dll.spf_score_extra.restype = i32
    dll.spf_score_extra.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), i32, vp, vp, ctypes.c_size_t, vp, vp]
    dll.spf_score_paged_workspace_bytes.restype = ctypes.c_size_t
    dll.spf_score_paged_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_PagedPrompt), i32]
    dll.spf_score_paged.restype = i32
    dll.spf_score_paged.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_PagedPrompt), i32, vp, ctypes.c_size_t, vp, vp]
    dll.spf_score_fp8_workspace_bytes.restype = ctypes.c_size_t
    dll.spf_score_fp8_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Fp8Prompt), i32]
    dll.spf_score_fp8.restype = i32
    dll.spf_score_fp8.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Fp8Prompt), i32, vp, ctypes.c_size_t, vp, vp]
    dll.spf_score_shard_lse.restype = i32
    dll.spf_score_shard_lse.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), vp, ctypes.c_size_t, vp]
    dll.spf_score_shard_apply.restype = i32
    dll.spf_score_shard_apply.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), vp, vp, ctypes.c_size_t, vp]
    dll.spf_score_shard_lse_ex.restype = i32
    dll.spf_score_shard_lse_ex.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), vp, ctypes.c_size_t, vp, vp]
    dll.spf_score_shard_apply_ex.restype = i32
    dll.spf_score_shard_apply_ex.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), vp, vp, ctypes.c_size_t, vp, vp]
    dll.spf_selftest_bounded_wait.restype = i32
    dll.spf_selftest_bounded_wait.argtypes = [vp, vp]
    dll.spf_set_score_path.restype = i32
    dll.spf_set_score_path.argtypes = [i32]
    dll.spf_score_static.restype = i32
    dll.spf_score_static.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Prompt), i32, vp]
    dll.spf_chunk_pool.restype = i32
    dll.spf_chunk_pool.argtypes = [vp, i64, i32, i32, vp, vp]
    dll.spf_select_topk.restype = i32
    dll.spf_select_topk.argtypes = [vp, i64, i64, vp, vp]
    dll.spf_chunk_pool_edge.restype = i32
    dll.spf_chunk_pool_edge.argtypes = [vp, i64, i32, i32, i32, vp, vp]
    dll.spf_select_topk_forced.restype = i32
    dll.spf_select_topk_forced.argtypes = [vp, i64, i64, i32, i32, vp, vp]
    dll.spf_compact_spans.restype = i32
    dll.spf_compact_spans.argtypes = [vp, i64, i32, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    dll.spf_compress_host_arena_bytes.restype = ctypes.c_size_t
    dll.spf_compress_host_arena_bytes.argtypes = [ctypes.POINTER(_Shape), i64, ctypes.POINTER(_SelectParams)]
    dll.spf_compress_host.restype = i32
    dll.spf_compress_host.argtypes = [ctypes.POINTER(_Shape), i64, ctypes.POINTER(ctypes.c_void_p), vp, vp, vp, vp,
                                      ctypes.POINTER(_SelectParams), vp, ctypes.c_size_t, vp, vp, vp, vp, vp, vp]
    dll.spf_select_compact.restype = i32
    dll.spf_select_compact.argtypes = [vp, i64, i64, i32, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    dll.spf_chunk_pool_batch.restype = i32
    dll.spf_chunk_pool_batch.argtypes = [ctypes.POINTER(_PoolItem), i32, i32, i32, vp]
    dll.spf_select_topk_batch.restype = i32
    dll.spf_select_topk_batch.argtypes = [ctypes.POINTER(_TopkItem), i32, vp]
    dll.spf_compact_spans_batch.restype = i32
    dll.spf_compact_spans_batch.argtypes = [ctypes.POINTER(_CompactItem), i32, i32, vp]
    dll.spf_keep_count.restype = i64
    dll.spf_keep_count.argtypes = [i64, ctypes.c_double]
    dll.spf_keep_rate.restype = ctypes.c_double
    dll.spf_keep_rate.argtypes = [i64, i64]
    dll.spf_snap_budget.restype = i64
    dll.spf_snap_budget.argtypes = [i64, i64]
    dll.spf_concat_with_delim.restype = i64
    dll.spf_concat_with_delim.argtypes = [ctypes.c_char_p, i64, vp, i64, ctypes.c_char_p, i64, vp, i64]
    dll.spf_status_string.restype = ctypes.c_char_p
    dll.spf_status_string.argtypes = [i32]
    dll.spf_last_error.restype = ctypes.c_char_p
    dll.spf_last_error.argtypes = []
    dll.spf_version.restype = ctypes.c_char_p
    dll.spf_version.argtypes = []
    return dll


lib = _load()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise SpfError(status, where, (lib.spf_last_error() or b"").decode() or
                       (lib.spf_status_string(status) or b"").decode())


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"{name} must be a CUDA tensor of dtype {dtype}")
    return t


def spf_version() -> str:
    return lib.spf_version().decode()


def spf_status_string(status: int) -> str:
    return lib.spf_status_string(status).decode()


def spf_last_error() -> str:
    return lib.spf_last_error().decode()


def spf_keep_count(n_chunks: int, keep_ratio: float) -> int:
    return int(lib.spf_keep_count(n_chunks, keep_ratio))


def spf_keep_rate(target_tokens: int, budget_tokens: int) -> float:
    return float(lib.spf_keep_rate(target_tokens, budget_tokens))


def spf_snap_budget(desired_tokens: int, block_tokens: int = 4096) -> int:
    return int(lib.spf_snap_budget(desired_tokens, block_tokens))


def spf_concat_with_delim(text: str, char_spans, delim: str) -> str:
    """Compressed prompt text from character spans (host routine of the library; spans as [n, 2] integers)."""
    import numpy as np
    raw, d = text.encode("utf-8"), delim.encode("utf-8")
    spans = np.ascontiguousarray(np.asarray(char_spans, dtype=np.int32).reshape(-1, 2))
    need = int(lib.spf_concat_with_delim(raw, len(raw), spans.ctypes.data, len(spans), d, len(d), None, 0))
    if need < 0:
        _check(need, "spf_concat_with_delim")
    out = ctypes.create_string_buffer(max(need, 1))
    got = int(lib.spf_concat_with_delim(raw, len(raw), spans.ctypes.data, len(spans), d, len(d), out, need))
    if got != need:
        _check(got if got < 0 else -1, "spf_concat_with_delim")
    return out.raw[:need].decode("utf-8")


@dataclasses.dataclass
class PromptBuffers:
    """Device buffers of one prompt, as spf_score reads and writes them."""
    q: torch.Tensor                      # bf16 [L, Hq, m, d]
    k_layers: Sequence[torch.Tensor]     # L tensors bf16 [Hkv, N, d]; last dim contiguous
    importance: torch.Tensor             # fp32 [N] (out)
    lse: Optional[torch.Tensor] = None   # fp32 [L, Hq, m] (out)


def _marshal(prompts: Sequence[PromptBuffers], softmax_scale: float):
    first = prompts[0]
    L, Hq, m, d = first.q.shape
    Hkv = first.k_layers[0].shape[0]
    shape = _Shape(L, Hq, Hkv, d, m, float(softmax_scale))
    arr = (_Prompt * len(prompts))()
    keep = []
    for i, p in enumerate(prompts):
        _dev(p.q, torch.bfloat16, "q")
        if tuple(p.q.shape) != (L, Hq, m, d) or not p.q.is_contiguous():
            raise ValueError("q must be contiguous [L, Hq, m, d], the same shape for all prompts")
        if len(p.k_layers) != L:
            raise ValueError("k_layers must hold one tensor per layer")
        k0 = p.k_layers[0]
        n = k0.shape[1]
        for kl in p.k_layers:
            _dev(kl, torch.bfloat16, "k_layers[l]")
            if tuple(kl.shape) != (Hkv, n, d) or kl.stride(2) != 1 or kl.stride() != k0.stride():
                raise ValueError("every k_layers[l] must be [Hkv, N, d] with a contiguous last dim and equal strides")
        _dev(p.importance, torch.float32, "importance")
        if p.importance.numel() != n or not p.importance.is_contiguous():
            raise ValueError("importance must be contiguous fp32 [N]")
        if p.lse is not None:
            _dev(p.lse, torch.float32, "lse")
            if p.lse.numel() != L * Hq * m or not p.lse.is_contiguous():
                raise ValueError("lse must be contiguous fp32 [L, Hq, m]")
        ptrs = (ctypes.c_void_p * L)(*[kl.data_ptr() for kl in p.k_layers])
        keep.append(ptrs)
        arr[i] = _Prompt(n, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), k0.stride(0), k0.stride(1),
                         p.q.data_ptr(), p.importance.data_ptr(), _ptr(p.lse))
    return shape, arr, keep


def spf_score_workspace_bytes(prompts: Sequence[PromptBuffers], softmax_scale: float = 0.0) -> int:
    shape, arr, _keep = _marshal(prompts, softmax_scale)
    n = int(lib.spf_score_workspace_bytes(ctypes.byref(shape), arr, len(prompts)))
    if n == 0:
        raise SpfError(-1, "spf_score_workspace_bytes", spf_last_error())
    return n


def spf_score(prompts: Sequence[PromptBuffers], workspace: torch.Tensor, softmax_scale: float = 0.0,
              dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> None:
    shape, arr, _keep = _marshal(prompts, softmax_scale)
    if not workspace.is_cuda:
        raise TypeError("workspace must be a CUDA tensor")
    _check(lib.spf_score(ctypes.byref(shape), arr, len(prompts), workspace.data_ptr(),
                         workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream_ptr(stream)),
           "spf_score")


def spf_score_extra(prompts: Sequence[PromptBuffers], extra_lse: Sequence[Optional[torch.Tensor]], workspace: torch.Tensor,
                    softmax_scale: float = 0.0, dev_status: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_score with a per-row extra term in the softmax denominator: extra_lse[p] is fp32 [L, Hq, m] or None."""
    shape, arr, _keep = _marshal(prompts, softmax_scale)
    if len(extra_lse) != len(prompts):
        raise ValueError("one extra_lse entry per prompt")
    L, Hq, m, _ = prompts[0].q.shape
    for e in extra_lse:
        if e is not None:
            _dev(e, torch.float32, "extra_lse")
            if e.numel() != L * Hq * m or not e.is_contiguous():
                raise ValueError("extra_lse must be contiguous fp32 [L, Hq, m]")
    ptrs = (ctypes.c_void_p * len(prompts))(*[None if e is None else e.data_ptr() for e in extra_lse])
    _check(lib.spf_score_extra(ctypes.byref(shape), arr, len(prompts), ptrs, workspace.data_ptr(),
                               workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream_ptr(stream)),
           "spf_score_extra")


@dataclasses.dataclass
class PagedPromptBuffers:
    """Device buffers of one prompt whose keys sit in a block pool (see spf_paged_prompt in include/spf.h)."""
    q: torch.Tensor                      # bf16 [L, Hq, m, d]
    k_pools: Sequence[torch.Tensor]      # L tensors bf16 [n_pool_blocks, Hkv, block_tokens, d], contiguous
    block_table: torch.Tensor            # int32 [ceil(N / block_tokens)]
    n_tokens: int
    importance: torch.Tensor             # fp32 [N] (out)
    lse: Optional[torch.Tensor] = None   # fp32 [L, Hq, m] (out)


def _marshal_paged(prompts: Sequence[PagedPromptBuffers], softmax_scale: float):
    L, Hq, m, d = prompts[0].q.shape
    Hkv = prompts[0].k_pools[0].shape[1]
    shape = _Shape(L, Hq, Hkv, d, m, float(softmax_scale))
    arr = (_PagedPrompt * len(prompts))()
    keep = []
    for i, p in enumerate(prompts):
        _dev(p.q, torch.bfloat16, "q")
        _dev(p.block_table, torch.int32, "block_table")
        _dev(p.importance, torch.float32, "importance")
        if len(p.k_pools) != L or not p.q.is_contiguous() or not p.block_table.is_contiguous():
            raise ValueError("one contiguous pool per layer, contiguous q and block_table")
        nb, hk, bt, dd = p.k_pools[0].shape
        for pool in p.k_pools:
            _dev(pool, torch.bfloat16, "k_pools[l]")
            if tuple(pool.shape) != (nb, hk, bt, dd) or not pool.is_contiguous() or hk != Hkv or dd != d:
                raise ValueError("every pool must be contiguous bf16 [n_pool_blocks, Hkv, block_tokens, d]")
        if p.block_table.numel() < (p.n_tokens + bt - 1) // bt or p.importance.numel() != p.n_tokens:
            raise ValueError("block_table or importance has the wrong size")
        ptrs = (ctypes.c_void_p * L)(*[pool.data_ptr() for pool in p.k_pools])
        keep.append(ptrs)
        arr[i] = _PagedPrompt(p.n_tokens, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), nb, bt, p.block_table.data_ptr(),
                              p.q.data_ptr(), p.importance.data_ptr(), _ptr(p.lse))
    return shape, arr, keep


def spf_score_paged_workspace_bytes(prompts: Sequence[PagedPromptBuffers], softmax_scale: float = 0.0) -> int:
    shape, arr, _keep = _marshal_paged(prompts, softmax_scale)
    n = int(lib.spf_score_paged_workspace_bytes(ctypes.byref(shape), arr, len(prompts)))
    if n == 0:
        raise SpfError(-1, "spf_score_paged_workspace_bytes", spf_last_error())
    return n


def spf_score_paged(prompts: Sequence[PagedPromptBuffers], workspace: torch.Tensor, softmax_scale: float = 0.0,
                    dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> None:
    shape, arr, _keep = _marshal_paged(prompts, softmax_scale)
    _check(lib.spf_score_paged(ctypes.byref(shape), arr, len(prompts), workspace.data_ptr(),
                               workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream_ptr(stream)),
           "spf_score_paged")


@dataclasses.dataclass
class Fp8PromptBuffers:
    """Device buffers of one prompt whose key cache is held in 8 bits (see spf_fp8_prompt in include/spf.h)."""
    q: torch.Tensor                      # bf16 [L, Hq, m, d]
    k_layers: Sequence[torch.Tensor]     # L tensors uint8 [Hkv, N, d] (E4M3 bytes); last dim contiguous
    k_scale: torch.Tensor                # fp32 [L, Hkv]
    importance: torch.Tensor             # fp32 [N] (out)
    lse: Optional[torch.Tensor] = None   # fp32 [L, Hq, m] (out)


def _marshal_fp8(prompts: Sequence[Fp8PromptBuffers], softmax_scale: float):
    L, Hq, m, d = prompts[0].q.shape
    Hkv = prompts[0].k_layers[0].shape[0]
    shape = _Shape(L, Hq, Hkv, d, m, float(softmax_scale))
    arr = (_Fp8Prompt * len(prompts))()
    keep = []
    for i, p in enumerate(prompts):
        _dev(p.q, torch.bfloat16, "q")
        _dev(p.k_scale, torch.float32, "k_scale")
        _dev(p.importance, torch.float32, "importance")
        k0 = p.k_layers[0]
        n = k0.shape[1]
        if len(p.k_layers) != L or not p.q.is_contiguous() or tuple(p.q.shape) != (L, Hq, m, d):
            raise ValueError("one key tensor per layer and a contiguous q of the batch's shape")
        for kl in p.k_layers:
            _dev(kl, torch.uint8, "k_layers[l]")
            if tuple(kl.shape) != (Hkv, n, d) or kl.stride(2) != 1 or kl.stride() != k0.stride():
                raise ValueError("every k_layers[l] must be uint8 [Hkv, N, d] with a contiguous last dim and equal strides")
        if p.k_scale.numel() != L * Hkv or not p.k_scale.is_contiguous() or p.importance.numel() != n:
            raise ValueError("k_scale must be contiguous fp32 [L, Hkv] and importance fp32 [N]")
        if p.lse is not None:
            _dev(p.lse, torch.float32, "lse")
        ptrs = (ctypes.c_void_p * L)(*[kl.data_ptr() for kl in p.k_layers])
        keep.append(ptrs)
        arr[i] = _Fp8Prompt(n, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), k0.stride(0), k0.stride(1),
                            p.k_scale.data_ptr(), p.q.data_ptr(), p.importance.data_ptr(), _ptr(p.lse))
    return shape, arr, keep


def spf_score_fp8_workspace_bytes(prompts: Sequence[Fp8PromptBuffers], softmax_scale: float = 0.0) -> int:
    shape, arr, _keep = _marshal_fp8(prompts, softmax_scale)
    n = int(lib.spf_score_fp8_workspace_bytes(ctypes.byref(shape), arr, len(prompts)))
    if n == 0:
        raise SpfError(-1, "spf_score_fp8_workspace_bytes", spf_last_error())
    return n


def spf_score_fp8(prompts: Sequence[Fp8PromptBuffers], workspace: torch.Tensor, softmax_scale: float = 0.0,
                  dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_score for key caches held as E4M3 bytes with one fp32 scale per (layer, kv-head)."""
    shape, arr, _keep = _marshal_fp8(prompts, softmax_scale)
    _check(lib.spf_score_fp8(ctypes.byref(shape), arr, len(prompts), workspace.data_ptr(),
                             workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream_ptr(stream)),
           "spf_score_fp8")


def spf_score_shard_lse(prompt: PromptBuffers, workspace: torch.Tensor, softmax_scale: float = 0.0,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """Row log-sum-exps over this shard's keys only, written to prompt.lse (see spf_score_shard_lse in include/spf.h)."""
    if prompt.lse is None:
        raise ValueError("prompt.lse receives the result")
    shape, arr, _keep = _marshal([prompt], softmax_scale)
    _check(lib.spf_score_shard_lse(ctypes.byref(shape), arr, workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                   _stream_ptr(stream)), "spf_score_shard_lse")


def spf_score_shard_apply(prompt: PromptBuffers, lse_all: torch.Tensor, workspace: torch.Tensor, softmax_scale: float = 0.0,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    """Importance of this shard's keys given the whole prompt's row log-sum-exps (fp32 [L, Hq, m])."""
    _dev(lse_all, torch.float32, "lse_all")
    shape, arr, _keep = _marshal([prompt], softmax_scale)
    L, Hq, m, _ = prompt.q.shape
    if lse_all.numel() != L * Hq * m or not lse_all.is_contiguous():
        raise ValueError("lse_all must be contiguous fp32 [L, Hq, m]")
    _check(lib.spf_score_shard_apply(ctypes.byref(shape), arr, lse_all.data_ptr(), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "spf_score_shard_apply")


def spf_score_shard_lse_ex(prompt: PromptBuffers, workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                           softmax_scale: float = 0.0, stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_score_shard_lse on the kernels spf_score would pick (the fused kernel's first visit where the shape allows)."""
    if prompt.lse is None:
        raise ValueError("prompt.lse receives the result")
    shape, arr, _keep = _marshal([prompt], softmax_scale)
    _check(lib.spf_score_shard_lse_ex(ctypes.byref(shape), arr, workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                      _ptr(dev_status), _stream_ptr(stream)), "spf_score_shard_lse_ex")


def spf_score_shard_apply_ex(prompt: PromptBuffers, lse_all: torch.Tensor, workspace: torch.Tensor,
                             dev_status: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                             stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_score_shard_apply on the kernels spf_score would pick (the fused kernel's second visit where the shape allows)."""
    _dev(lse_all, torch.float32, "lse_all")
    shape, arr, _keep = _marshal([prompt], softmax_scale)
    L, Hq, m, _ = prompt.q.shape
    if lse_all.numel() != L * Hq * m or not lse_all.is_contiguous():
        raise ValueError("lse_all must be contiguous fp32 [L, Hq, m]")
    _check(lib.spf_score_shard_apply_ex(ctypes.byref(shape), arr, lse_all.data_ptr(), workspace.data_ptr(),
                                        workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream_ptr(stream)),
           "spf_score_shard_apply_ex")


def spf_selftest_bounded_wait(dev_status: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Enqueues the bounded-wait self-test; dev_status (int32, zeroed) reads SPF_ERR_TIMEOUT (-5) afterwards."""
    _dev(dev_status, torch.int32, "dev_status")
    _check(lib.spf_selftest_bounded_wait(dev_status.data_ptr(), _stream_ptr(stream)), "spf_selftest_bounded_wait")


def spf_set_score_path(path: int) -> int:
    """0 automatic, 1 general two-sweep path, 2 fused path; returns the previous setting."""
    return int(lib.spf_set_score_path(path))


def spf_score_static(prompts: Sequence[PromptBuffers], softmax_scale: float = 0.0,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_score for callers that cannot allocate: the library's built-in scratch array replaces the workspace.

    Calls that overlap on the GPU share that array and race; keep them ordered on one stream.
    """
    shape, arr, _keep = _marshal(prompts, softmax_scale)
    _check(lib.spf_score_static(ctypes.byref(shape), arr, len(prompts), _stream_ptr(stream)), "spf_score_static")


def spf_chunk_pool(importance: torch.Tensor, pool_kernel: int, chunk: int, chunk_scores: torch.Tensor,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
    _dev(importance, torch.float32, "importance")
    _dev(chunk_scores, torch.float32, "chunk_scores")
    n = importance.numel()
    if chunk >= 1 and chunk_scores.numel() < (n + chunk - 1) // chunk:
        raise ValueError("chunk_scores is too small")
    _check(lib.spf_chunk_pool(importance.data_ptr(), n, pool_kernel, chunk, chunk_scores.data_ptr(),
                              _stream_ptr(stream)), "spf_chunk_pool")


def spf_chunk_pool_edge(importance: torch.Tensor, pool_kernel: int, chunk: int, edge_rule: int, chunk_scores: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_chunk_pool with the pooling edge rule as an argument (0: divide by the kernel, 1: by the tokens covered)."""
    _dev(importance, torch.float32, "importance")
    _dev(chunk_scores, torch.float32, "chunk_scores")
    n = importance.numel()
    if chunk >= 1 and chunk_scores.numel() < (n + chunk - 1) // chunk:
        raise ValueError("chunk_scores is too small")
    _check(lib.spf_chunk_pool_edge(importance.data_ptr(), n, pool_kernel, chunk, edge_rule, chunk_scores.data_ptr(),
                                   _stream_ptr(stream)), "spf_chunk_pool_edge")


def spf_select_topk_forced(chunk_scores: torch.Tensor, n_chunks: int, k: int, force_first: bool, force_last: bool,
                           kept_chunks: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_select_topk that always keeps the first and / or the last chunk (they count towards k)."""
    _dev(chunk_scores, torch.float32, "chunk_scores")
    _dev(kept_chunks, torch.int32, "kept_chunks")
    if chunk_scores.numel() < n_chunks or kept_chunks.numel() < k:
        raise ValueError("chunk_scores or kept_chunks is too small")
    _check(lib.spf_select_topk_forced(chunk_scores.data_ptr(), n_chunks, k, int(bool(force_first)), int(bool(force_last)),
                                      kept_chunks.data_ptr(), _stream_ptr(stream)), "spf_select_topk_forced")


def spf_select_topk(chunk_scores: torch.Tensor, n_chunks: int, k: int, kept_chunks: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
    _dev(chunk_scores, torch.float32, "chunk_scores")
    _dev(kept_chunks, torch.int32, "kept_chunks")
    if chunk_scores.numel() < n_chunks or kept_chunks.numel() < k:
        raise ValueError("chunk_scores or kept_chunks is too small")
    _check(lib.spf_select_topk(chunk_scores.data_ptr(), n_chunks, k, kept_chunks.data_ptr(), _stream_ptr(stream)),
           "spf_select_topk")


def spf_compact_spans(kept_chunks: torch.Tensor, k: int, chunk: int, n_tokens: int, token_ids: torch.Tensor,
                      char_start: torch.Tensor, char_end: torch.Tensor, out_ids: torch.Tensor,
                      out_pos: Optional[torch.Tensor], out_tok_spans: torch.Tensor, out_char_spans: torch.Tensor,
                      out_counts: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    for name, t in (("kept_chunks", kept_chunks), ("token_ids", token_ids), ("char_start", char_start),
                    ("char_end", char_end), ("out_ids", out_ids), ("out_tok_spans", out_tok_spans),
                    ("out_char_spans", out_char_spans)):
        _dev(t, torch.int32, name)
    if out_pos is not None:
        _dev(out_pos, torch.int32, "out_pos")
    _dev(out_counts, torch.int64, "out_counts")
    need = min(max(k, 0) * max(chunk, 0), n_tokens)
    if out_ids.numel() < need or (out_pos is not None and out_pos.numel() < need) or \
            out_tok_spans.numel() < 2 * k or out_char_spans.numel() < 2 * k or out_counts.numel() < 2 or \
            min(token_ids.numel(), char_start.numel(), char_end.numel()) < n_tokens or kept_chunks.numel() < k:
        raise ValueError("a buffer is smaller than include/spf.h requires")
    _check(lib.spf_compact_spans(kept_chunks.data_ptr(), k, chunk, n_tokens, token_ids.data_ptr(),
                                 char_start.data_ptr(), char_end.data_ptr(), out_ids.data_ptr(), _ptr(out_pos),
                                 out_tok_spans.data_ptr(), out_char_spans.data_ptr(), out_counts.data_ptr(),
                                 _stream_ptr(stream)), "spf_compact_spans")


def spf_select_compact(chunk_scores: torch.Tensor, n_chunks: int, k: int, chunk: int, n_tokens: int, token_ids: torch.Tensor,
                       char_start: torch.Tensor, char_end: torch.Tensor, kept_chunks: torch.Tensor, out_ids: torch.Tensor,
                       out_pos: Optional[torch.Tensor], out_tok_spans: torch.Tensor, out_char_spans: torch.Tensor,
                       out_counts: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_select_topk + spf_compact_spans in one launch (same buffers and sizes as the two calls)."""
    _dev(chunk_scores, torch.float32, "chunk_scores")
    for name, t in (("kept_chunks", kept_chunks), ("token_ids", token_ids), ("char_start", char_start),
                    ("char_end", char_end), ("out_ids", out_ids), ("out_tok_spans", out_tok_spans),
                    ("out_char_spans", out_char_spans)):
        _dev(t, torch.int32, name)
    if out_pos is not None:
        _dev(out_pos, torch.int32, "out_pos")
    _dev(out_counts, torch.int64, "out_counts")
    need = min(max(k, 0) * max(chunk, 0), n_tokens)
    if chunk_scores.numel() < n_chunks or kept_chunks.numel() < k or out_ids.numel() < need or \
            (out_pos is not None and out_pos.numel() < need) or out_tok_spans.numel() < 2 * k or \
            out_char_spans.numel() < 2 * k or out_counts.numel() < 2 or \
            min(token_ids.numel(), char_start.numel(), char_end.numel()) < n_tokens:
        raise ValueError("a buffer is smaller than include/spf.h requires")
    _check(lib.spf_select_compact(chunk_scores.data_ptr(), n_chunks, k, chunk, n_tokens, token_ids.data_ptr(),
                                  char_start.data_ptr(), char_end.data_ptr(), kept_chunks.data_ptr(), out_ids.data_ptr(),
                                  _ptr(out_pos), out_tok_spans.data_ptr(), out_char_spans.data_ptr(), out_counts.data_ptr(),
                                  _stream_ptr(stream)), "spf_select_compact")


def spf_chunk_pool_batch(importances: Sequence[torch.Tensor], pool_kernel: int, chunk: int,
                         chunk_scores: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_chunk_pool for several prompts in one launch: importances[p] fp32 [N_p] -> chunk_scores[p] fp32 [ceil(N_p / chunk)]."""
    items = (_PoolItem * len(importances))()
    for i, (imp, cs) in enumerate(zip(importances, chunk_scores)):
        _dev(imp, torch.float32, "importance")
        _dev(cs, torch.float32, "chunk_scores")
        if chunk >= 1 and cs.numel() < (imp.numel() + chunk - 1) // chunk:
            raise ValueError("chunk_scores is too small")
        items[i] = _PoolItem(imp.data_ptr(), imp.numel(), cs.data_ptr())
    _check(lib.spf_chunk_pool_batch(items, len(importances), pool_kernel, chunk, _stream_ptr(stream)), "spf_chunk_pool_batch")


def spf_select_topk_batch(chunk_scores: Sequence[torch.Tensor], n_chunks: Sequence[int], ks: Sequence[int],
                          kept_chunks: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_select_topk for several prompts in one launch (one CTA per prompt)."""
    items = (_TopkItem * len(chunk_scores))()
    for i, (cs, n, k, kept) in enumerate(zip(chunk_scores, n_chunks, ks, kept_chunks)):
        _dev(cs, torch.float32, "chunk_scores")
        _dev(kept, torch.int32, "kept_chunks")
        if cs.numel() < n or kept.numel() < k:
            raise ValueError("chunk_scores or kept_chunks is too small")
        items[i] = _TopkItem(cs.data_ptr(), n, k, kept.data_ptr())
    _check(lib.spf_select_topk_batch(items, len(chunk_scores), _stream_ptr(stream)), "spf_select_topk_batch")


def spf_compact_spans_batch(kept_chunks: Sequence[torch.Tensor], ks: Sequence[int], chunk: int, n_tokens: Sequence[int],
                            token_ids: Sequence[torch.Tensor], char_start: Sequence[torch.Tensor],
                            char_end: Sequence[torch.Tensor], out_ids: Sequence[torch.Tensor],
                            out_pos: Sequence[Optional[torch.Tensor]], out_tok_spans: Sequence[torch.Tensor],
                            out_char_spans: Sequence[torch.Tensor], out_counts: Sequence[torch.Tensor],
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """spf_compact_spans for several prompts in one launch; buffer sizes per prompt as for the single call."""
    n_items = len(kept_chunks)
    items = (_CompactItem * n_items)()
    for i in range(n_items):
        k, n = ks[i], n_tokens[i]
        for name, t in (("kept_chunks", kept_chunks[i]), ("token_ids", token_ids[i]), ("char_start", char_start[i]),
                        ("char_end", char_end[i]), ("out_ids", out_ids[i]), ("out_tok_spans", out_tok_spans[i]),
                        ("out_char_spans", out_char_spans[i])):
            _dev(t, torch.int32, name)
        _dev(out_counts[i], torch.int64, "out_counts")
        need = min(max(k, 0) * max(chunk, 0), n)
        if out_ids[i].numel() < need or (out_pos[i] is not None and out_pos[i].numel() < need) or \
                out_tok_spans[i].numel() < 2 * k or out_char_spans[i].numel() < 2 * k or out_counts[i].numel() < 2 or \
                min(token_ids[i].numel(), char_start[i].numel(), char_end[i].numel()) < n or kept_chunks[i].numel() < k:
            raise ValueError("a buffer is smaller than include/spf.h requires")
        items[i] = _CompactItem(kept_chunks[i].data_ptr(), k, n, token_ids[i].data_ptr(), char_start[i].data_ptr(),
                                char_end[i].data_ptr(), out_ids[i].data_ptr(), _ptr(out_pos[i]), out_tok_spans[i].data_ptr(),
                                out_char_spans[i].data_ptr(), out_counts[i].data_ptr())
    _check(lib.spf_compact_spans_batch(items, n_items, chunk, _stream_ptr(stream)), "spf_compact_spans_batch")


def _host(t: torch.Tensor, dtype: torch.dtype, name: str) -> torch.Tensor:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous host tensor of dtype {dtype}")
    return t


def spf_compress_host_arena_bytes(n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_lookahead: int,
                                  n_tokens: int, chunk: int, pool_kernel: int, keep: float, softmax_scale: float = 0.0) -> int:
    shape = _Shape(n_layers, n_q_heads, n_kv_heads, head_dim, n_lookahead, float(softmax_scale))
    prm = _SelectParams(chunk, pool_kernel, float(keep))
    n = int(lib.spf_compress_host_arena_bytes(ctypes.byref(shape), n_tokens, ctypes.byref(prm)))
    if n == 0:
        raise SpfError(-1, "spf_compress_host_arena_bytes", spf_last_error())
    return n


def spf_compress_host(q: torch.Tensor, k_layers: Sequence[torch.Tensor], token_ids: torch.Tensor, char_start: torch.Tensor,
                      char_end: torch.Tensor, chunk: int, pool_kernel: int, keep: float, arena: torch.Tensor,
                      out_ids: torch.Tensor, out_pos: Optional[torch.Tensor], out_tok_spans: torch.Tensor,
                      out_char_spans: torch.Tensor, out_counts: torch.Tensor, softmax_scale: float = 0.0,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
    """The whole path for one prompt in HOST tensors (inputs and outputs); ``arena`` is device scratch.  Synchronises the
    stream.  See spf_compress_host in include/spf.h for sizes."""
    L, Hq, m, d = q.shape
    Hkv, n, _ = k_layers[0].shape
    _host(q, torch.bfloat16, "q")
    for kl in k_layers:
        _host(kl, torch.bfloat16, "k_layers[l]")
        if tuple(kl.shape) != (Hkv, n, d):
            raise ValueError("every k_layers[l] must be [Hkv, N, d]")
    for name, t in (("token_ids", token_ids), ("char_start", char_start), ("char_end", char_end), ("out_ids", out_ids),
                    ("out_tok_spans", out_tok_spans), ("out_char_spans", out_char_spans)):
        _host(t, torch.int32, name)
    if out_pos is not None:
        _host(out_pos, torch.int32, "out_pos")
    _host(out_counts, torch.int64, "out_counts")
    if not arena.is_cuda:
        raise TypeError("arena must be a CUDA tensor")
    k = spf_keep_count((n + chunk - 1) // chunk, keep)
    need = min(k * chunk, n)
    if len(k_layers) != L or min(token_ids.numel(), char_start.numel(), char_end.numel()) < n or out_ids.numel() < need or \
            (out_pos is not None and out_pos.numel() < need) or out_tok_spans.numel() < 2 * k or \
            out_char_spans.numel() < 2 * k or out_counts.numel() < 2:
        raise ValueError("a buffer is smaller than include/spf.h requires")
    shape = _Shape(L, Hq, Hkv, d, m, float(softmax_scale))
    prm = _SelectParams(chunk, pool_kernel, float(keep))
    ptrs = (ctypes.c_void_p * L)(*[kl.data_ptr() for kl in k_layers])
    _check(lib.spf_compress_host(ctypes.byref(shape), n, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), q.data_ptr(),
                                 token_ids.data_ptr(), char_start.data_ptr(), char_end.data_ptr(), ctypes.byref(prm),
                                 arena.data_ptr(), arena.numel() * arena.element_size(), out_ids.data_ptr(), _ptr(out_pos),
                                 out_tok_spans.data_ptr(), out_char_spans.data_ptr(), out_counts.data_ptr(),
                                 _stream_ptr(stream)), "spf_compress_host")


@dataclasses.dataclass
class Selection:
    """Device-side result of one prompt; ``n_kept`` / ``n_spans`` are read from ``counts`` on demand."""
    importance: torch.Tensor
    lse: torch.Tensor
    chunk_scores: torch.Tensor
    k: int
    kept_chunks: torch.Tensor
    out_ids: torch.Tensor
    out_pos: torch.Tensor
    tok_spans: torch.Tensor
    char_spans: torch.Tensor
    counts: torch.Tensor

    def host(self):
        """Copies the result to the host (synchronises) and trims it to the valid rows."""
        counts = self.counts.cpu()
        n_kept, n_spans = int(counts[0]), int(counts[1])
        return dict(importance=self.importance.cpu().numpy(), lse=self.lse.cpu().numpy(),
                    chunk_scores=self.chunk_scores.cpu().numpy(), k=self.k,
                    kept=self.kept_chunks[:self.k].cpu().numpy(), ids=self.out_ids[:n_kept].cpu().numpy(),
                    pos=self.out_pos[:n_kept].cpu().numpy(), tok_spans=self.tok_spans[:n_spans].cpu().numpy(),
                    char_spans=self.char_spans[:n_spans].cpu().numpy())


class Selector:
    """Chains spf_score -> spf_chunk_pool -> spf_select_topk -> spf_compact_spans for prompts of one geometry.

    Buffers are allocated once for ``max_tokens`` and reused, so that a call enqueues kernels only.
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_lookahead: int,
                 max_tokens: int, chunk: int = 32, pool_kernel: int = 13, softmax_scale: float = 0.0,
                 device: str = "cuda", pool_edge_rule: int = 0, force_first: bool = False, force_last: bool = False):
        self.geom = (n_layers, n_q_heads, n_kv_heads, head_dim, n_lookahead)
        self.chunk, self.pool_kernel, self.softmax_scale = chunk, pool_kernel, softmax_scale
        # switches for points the paper leaves open (defaults: the readings the library takes)
        self.pool_edge_rule, self.force_first, self.force_last = pool_edge_rule, force_first, force_last
        self.max_tokens = max_tokens
        self.device = torch.device(device)
        max_chunks = (max_tokens + chunk - 1) // chunk
        dev = self.device
        self.importance = torch.empty(max_tokens, dtype=torch.float32, device=dev)
        self.lse = torch.empty(n_layers * n_q_heads * n_lookahead, dtype=torch.float32, device=dev)
        self.chunk_scores = torch.empty(max_chunks, dtype=torch.float32, device=dev)
        self.kept = torch.empty(max_chunks, dtype=torch.int32, device=dev)
        self.out_ids = torch.empty(max_tokens, dtype=torch.int32, device=dev)
        self.out_pos = torch.empty(max_tokens, dtype=torch.int32, device=dev)
        self.tok_spans = torch.empty((max_chunks, 2), dtype=torch.int32, device=dev)
        self.char_spans = torch.empty((max_chunks, 2), dtype=torch.int32, device=dev)
        self.counts = torch.zeros(2, dtype=torch.int64, device=dev)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.workspace: Optional[torch.Tensor] = None

    def _workspace(self, bufs: PromptBuffers) -> torch.Tensor:
        need = spf_score_workspace_bytes([bufs], self.softmax_scale)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self.workspace

    def run(self, q: torch.Tensor, k_layers: Sequence[torch.Tensor], token_ids: torch.Tensor,
            char_start: torch.Tensor, char_end: torch.Tensor, keep: float,
            stream: Optional[torch.cuda.Stream] = None) -> Selection:
        """Enqueues the whole path for one prompt whose tensors are already on the device.  Nothing is synchronised:
        device-side conditions (see spf_score) accumulate in ``self.dev_status``, which the caller zeroes and reads
        (run_checked does both)."""
        n = k_layers[0].shape[1]
        if n > self.max_tokens:
            raise ValueError(f"prompt has {n} tokens, selector was sized for {self.max_tokens}")
        bufs = PromptBuffers(q, k_layers, self.importance[:n], self.lse)
        spf_score([bufs], self._workspace(bufs), self.softmax_scale, self.dev_status, stream)
        return self._select(n, token_ids, char_start, char_end, keep, stream)

    def run_paged(self, q: torch.Tensor, k_pools: Sequence[torch.Tensor], block_table: torch.Tensor, n_tokens: int,
                  token_ids: torch.Tensor, char_start: torch.Tensor, char_end: torch.Tensor, keep: float,
                  stream: Optional[torch.cuda.Stream] = None) -> Selection:
        """run() for a prompt whose keys sit in a block pool (see PagedPromptBuffers)."""
        n = n_tokens
        if n > self.max_tokens:
            raise ValueError(f"prompt has {n} tokens, selector was sized for {self.max_tokens}")
        bufs = PagedPromptBuffers(q, k_pools, block_table, n, self.importance[:n], self.lse)
        need = spf_score_paged_workspace_bytes([bufs], self.softmax_scale)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        spf_score_paged([bufs], self.workspace, self.softmax_scale, self.dev_status, stream)
        return self._select(n, token_ids, char_start, char_end, keep, stream)

    def run_fp8(self, q: torch.Tensor, k_layers: Sequence[torch.Tensor], k_scale: torch.Tensor, token_ids: torch.Tensor,
                char_start: torch.Tensor, char_end: torch.Tensor, keep: float,
                stream: Optional[torch.cuda.Stream] = None) -> Selection:
        """run() for a prompt whose key cache is held as E4M3 bytes (see Fp8PromptBuffers)."""
        n = k_layers[0].shape[1]
        if n > self.max_tokens:
            raise ValueError(f"prompt has {n} tokens, selector was sized for {self.max_tokens}")
        bufs = Fp8PromptBuffers(q, k_layers, k_scale, self.importance[:n], self.lse)
        need = spf_score_fp8_workspace_bytes([bufs], self.softmax_scale)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        spf_score_fp8([bufs], self.workspace, self.softmax_scale, self.dev_status, stream)
        return self._select(n, token_ids, char_start, char_end, keep, stream)

    def _select(self, n: int, token_ids: torch.Tensor, char_start: torch.Tensor, char_end: torch.Tensor, keep: float,
                stream: Optional[torch.cuda.Stream]) -> Selection:
        """Pooling, top-k and compaction on the importance scores already in self.importance[:n]."""
        n_chunks = (n + self.chunk - 1) // self.chunk
        k = spf_keep_count(n_chunks, keep)
        if self.pool_edge_rule:
            spf_chunk_pool_edge(self.importance[:n], self.pool_kernel, self.chunk, self.pool_edge_rule,
                                self.chunk_scores[:n_chunks], stream)
        else:
            spf_chunk_pool(self.importance[:n], self.pool_kernel, self.chunk, self.chunk_scores[:n_chunks], stream)
        if self.force_first or self.force_last:
            k = max(k, len({0} if self.force_first else set()) + (1 if self.force_last and (n_chunks > 1 or not self.force_first) else 0))
            spf_select_topk_forced(self.chunk_scores, n_chunks, k, self.force_first, self.force_last, self.kept, stream)
            spf_compact_spans(self.kept, k, self.chunk, n, token_ids, char_start, char_end, self.out_ids, self.out_pos,
                              self.tok_spans, self.char_spans, self.counts, stream)
        else:
            # top-k and compaction chained in one launch
            spf_select_compact(self.chunk_scores, n_chunks, k, self.chunk, n, token_ids, char_start, char_end, self.kept,
                               self.out_ids, self.out_pos, self.tok_spans, self.char_spans, self.counts, stream)
        L, Hq, _, _, m = self.geom
        return Selection(self.importance[:n], self.lse.view(L, Hq, m), self.chunk_scores[:n_chunks], k, self.kept,
                         self.out_ids, self.out_pos, self.tok_spans, self.char_spans, self.counts)

    # device conditions after which the general path is tried: a row sum beyond fp32 (-6), a bounded wait that ran
    # out (-5); and the host refusal of a grid that cannot be co-resident (-2, raised as SpfError)
    _RETRY_ON = (-5, -6)

    def run_checked(self, q: torch.Tensor, k_layers: Sequence[torch.Tensor], token_ids: torch.Tensor,
                    char_start: torch.Tensor, char_end: torch.Tensor, keep: float,
                    stream: Optional[torch.cuda.Stream] = None) -> Selection:
        """Like run(), but synchronises and reads the device status.  If the fused scoring kernel reported
        SPF_ERR_RANGE (a row sum beyond fp32) or SPF_ERR_TIMEOUT (a bounded wait ran out, e.g. because its CTAs
        could not all run at once), or refused the launch as unsupported, the prompt is scored again on the
        general path, which has neither limit.  Any other status raises."""
        s = stream or torch.cuda.current_stream()
        self.dev_status.zero_()
        try:
            sel = self.run(q, k_layers, token_ids, char_start, char_end, keep, stream)
            s.synchronize()
            status = int(self.dev_status.item())
        except SpfError as err:
            if err.status != -2:
                raise
            status = -2
        if status in self._RETRY_ON or status == -2:
            previous = spf_set_score_path(1)
            try:
                self.dev_status.zero_()
                sel = self.run(q, k_layers, token_ids, char_start, char_end, keep, stream)
                s.synchronize()
                status = int(self.dev_status.item())
            finally:
                spf_set_score_path(previous)
        if status != 0:
            raise SpfError(status, "Selector.run_checked", spf_status_string(status))
        return sel

    def run_host(self, q: torch.Tensor, k_layers: Sequence[torch.Tensor], token_ids: torch.Tensor,
                 char_start: torch.Tensor, char_end: torch.Tensor, keep: float):
        """Same path for HOST tensors (ideally pinned) through spf_compress_host: one C call that copies in, runs and
        copies the selection back.  The device arena and the pinned result buffers are kept between calls.

        Returns host NumPy arrays: kept ids, positions, token spans, character spans.
        """
        L, Hq, Hkv, d, m = self.geom
        n = k_layers[0].shape[1]
        need = spf_compress_host_arena_bytes(L, Hq, Hkv, d, m, n, self.chunk, self.pool_kernel, keep, self.softmax_scale)
        if getattr(self, "_arena", None) is None or self._arena.numel() < need:
            self._arena = torch.empty(need, dtype=torch.uint8, device=self.device)
        k = spf_keep_count((n + self.chunk - 1) // self.chunk, keep)
        rows = min(k * self.chunk, n)
        host = getattr(self, "_host_out", None)
        if host is None or host[0].numel() < rows or host[2].numel() < 2 * k:
            host = [torch.empty(rows, dtype=torch.int32).pin_memory(), torch.empty(rows, dtype=torch.int32).pin_memory(),
                    torch.empty((k, 2), dtype=torch.int32).pin_memory(), torch.empty((k, 2), dtype=torch.int32).pin_memory(),
                    torch.empty(2, dtype=torch.int64).pin_memory()]
            self._host_out = host
        ids, pos, tok, ch, counts = host
        with torch.cuda.device(self.device):
            spf_compress_host(q, k_layers, token_ids, char_start, char_end, self.chunk, self.pool_kernel, keep, self._arena,
                              ids, pos, tok, ch, counts, self.softmax_scale)
        n_kept, n_spans = int(counts[0]), int(counts[1])
        return dict(ids=ids[:n_kept].numpy().copy(), pos=pos[:n_kept].numpy().copy(), tok_spans=tok[:n_spans].numpy().copy(),
                    char_spans=ch[:n_spans].numpy().copy())


class BatchSelector:
    """The path for a batch of prompts of one geometry: one spf_score call for the batch, then ONE launch each of
    pooling, top-k and compaction for all prompts (the batched calls).  Buffers are allocated once per prompt slot."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_lookahead: int,
                 max_tokens: Sequence[int], chunk: int = 32, pool_kernel: int = 13, softmax_scale: float = 0.0,
                 device: str = "cuda"):
        self.geom = (n_layers, n_q_heads, n_kv_heads, head_dim, n_lookahead)
        self.chunk, self.pool_kernel, self.softmax_scale = chunk, pool_kernel, softmax_scale
        self.device = torch.device(device)
        self.slots = [Selector(n_layers, n_q_heads, n_kv_heads, head_dim, n_lookahead, n, chunk=chunk,
                               pool_kernel=pool_kernel, softmax_scale=softmax_scale, device=device) for n in max_tokens]
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.workspace: Optional[torch.Tensor] = None

    def run(self, prompts, keep: float, stream: Optional[torch.cuda.Stream] = None):
        """prompts: objects with q, k (list), token_ids, char_start, char_end, n_tokens (device tensors).  Returns one
        Selection per prompt; nothing is synchronised."""
        if len(prompts) > len(self.slots):
            raise ValueError("more prompts than slots")
        slots = self.slots[:len(prompts)]
        bufs = [PromptBuffers(p.q, p.k, s.importance[:p.n_tokens], s.lse) for p, s in zip(prompts, slots)]
        need = spf_score_workspace_bytes(bufs, self.softmax_scale)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        spf_score(bufs, self.workspace, self.softmax_scale, self.dev_status, stream)
        ns = [p.n_tokens for p in prompts]
        ncs = [(n + self.chunk - 1) // self.chunk for n in ns]
        ks = [spf_keep_count(c, keep) for c in ncs]
        spf_chunk_pool_batch([s.importance[:n] for s, n in zip(slots, ns)], self.pool_kernel, self.chunk,
                             [s.chunk_scores[:c] for s, c in zip(slots, ncs)], stream)
        spf_select_topk_batch([s.chunk_scores for s in slots], ncs, ks, [s.kept for s in slots], stream)
        spf_compact_spans_batch([s.kept for s in slots], ks, self.chunk, ns, [p.token_ids for p in prompts],
                                [p.char_start for p in prompts], [p.char_end for p in prompts], [s.out_ids for s in slots],
                                [s.out_pos for s in slots], [s.tok_spans for s in slots], [s.char_spans for s in slots],
                                [s.counts for s in slots], stream)
        L, Hq, _, _, m = self.geom
        return [Selection(s.importance[:n], s.lse.view(L, Hq, m), s.chunk_scores[:c], k, s.kept, s.out_ids, s.out_pos,
                          s.tok_spans, s.char_spans, s.counts) for s, n, c, k in zip(slots, ns, ncs, ks)]
