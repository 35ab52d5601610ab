"""ctypes binding of libloma (declared in ``include/loma.h``).

Argument marshalling only: every function here has the name of the C entry
point it calls, takes torch tensors (device memory) or plain ints, pulls out
pointers, shapes and strides, and raises :class:`LomaError` on a negative
status.  No arithmetic of the method happens in Python, and there is no
fallback: if the library has not been built, loading fails with an error.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

LOMA_F32 = 0
LOMA_BF16 = 1
LOMA_FLAG_MEM_SEES_PRIOR_MEM = 1
LOMA_FLAG_NO_REP_ZONE = 2
LOMA_FLAG_FORCE_GENERIC = 1 << 8

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libloma.so")
_lib = None

_i, _i64, _f, _u, _p, _sz = (ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_uint, ctypes.c_void_p,
                             ctypes.c_size_t)

# name -> (restype, argtypes); mirrors include/loma.h
SIGNATURES = {
    "loma_layout_index": (_i, [_i, _i, _i, _i, _u, _p, _p, _p, _p, _p, _i, _p]),
    "loma_prefill_cache": (_i, [_p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _i64, _i64, _i64, _i, _u, _p, _p]),
    "loma_generation_index": (_i, [_i, _i, _i, _p, _p, _p, _i, _p]),
    "loma_masked_attn_fwd": (_i, [_p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i64, _i64, _i64, _i, _f,
                                  _u, _p]),
    "loma_masked_attn_bwd": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i64, _i64, _i64, _i,
                                  _f, _u, _p, _sz, _p]),
    "loma_masked_attn_bwd_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i, _u]),
    "loma_rope_apply": (_i, [_p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i64, _i64, _i64, _i, _f, _i, _u, _p]),
    "loma_masked_attn_plan_coverage": (_i, [_i, _i, _i, _i, _u, _p]),
    "loma_masked_attn_bwd_plan_coverage": (_i, [_i, _i, _i, _i, _u, _p]),
    "loma_prefill_attn": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _f, _u, _p]),
    "loma_prefill_attn_ragged": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _p, _i, _i, _f, _u, _p]),
    "loma_prefill_attn_paged": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _p, _i, _i, _f, _u, _p]),
    "loma_prefill_attn_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _f, _i, _f, _u, _p]),
    "loma_prefill_attn_ragged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _p, _i, _p, _f, _i, _f, _u, _p]),
    "loma_prefill_attn_paged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _p, _i, _p, _f, _i, _f,
                                          _u, _p]),
    "loma_prefill_attn_plan_coverage": (_i, [_i, _i, _p]),
    "loma_decode_attn": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _f, _u, _p, _sz, _p]),
    "loma_decode_attn_layers": (_i, [_i, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _f, _u, _p, _sz, _p]),
    "loma_compress_step_layers": (_i, [_i, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _f, _u, _p, _sz,
                                       _p]),
    "loma_decode_attn_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _f, _i, _f, _u, _p, _sz, _p]),
    "loma_compress_step_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _i, _f, _i, _f, _u, _p,
                                     _sz, _p]),
    "loma_decode_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "loma_decode_attn_paged": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _p, _i, _i, _f, _u, _p, _sz, _p]),
    "loma_decode_attn_ragged": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _p, _i, _i, _f, _u, _p, _sz, _p]),
    "loma_decode_attn_ragged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _p, _i, _p, _f, _i, _f, _u, _p, _sz, _p]),
    "loma_decode_attn_paged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _p, _i, _p, _f, _i, _f, _u, _p, _sz,
                                         _p]),
    "loma_compress_step_ragged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _p, _i, _i, _i, _i, _p, _i, _f, _i, _f, _u, _p]),
    "loma_compress_step_paged_rope": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _p, _i, _i, _i, _i, _p, _i, _f, _i,
                                           _f, _u, _p]),
    "loma_decode_attn_static": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _f, _p]),
    "loma_decode_static_scratch_bytes": (_sz, []),
    "loma_compress_step": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _f, _u, _p, _sz,
                                _p]),
    "loma_compress_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _u]),
    "loma_compress_step_paged": (_i, [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _p, _i, _i, _i, _i, _i, _f, _u, _p]),
    "loma_compress_step_ragged": (_i, [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _p, _i, _i, _i, _i, _i, _f, _u, _p]),
    "loma_device_status": (_i, [_p]),
    "loma_selftest_bounded_wait": (_i, [_p]),
    "loma_launch_count": (ctypes.c_uint64, []),
    "loma_fallback_count": (ctypes.c_uint64, []),
    "loma_status_string": (ctypes.c_char_p, [_i]),
    "loma_version": (_i, []),
}


class LomaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def library_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Load libloma.so once.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2401_09486_b200.build` "
                "(there is no fallback path)")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().loma_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise LomaError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LOMA_F32
    if t.dtype == torch.bfloat16:
        return LOMA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif isinstance(stream, torch.cuda.Stream):
        stream = stream.cuda_stream
    return ctypes.c_void_p(int(stream))


def loma_version() -> int:
    return lib().loma_version()


def loma_launch_count() -> int:
    return int(lib().loma_launch_count())


def loma_fallback_count() -> int:
    """bf16 calls that ran on the CUDA-core kernels because the tensor-core path declined them."""
    return int(lib().loma_fallback_count())


def loma_selftest_bounded_wait(stream=None) -> None:
    _check(lib().loma_selftest_bounded_wait(_stream(stream)), "loma_selftest_bounded_wait")


def loma_device_status(stream=None) -> int:
    return lib().loma_device_status(_stream(stream))


def loma_layout_index(n_chunks: int, c: int, t: int, tail_read: int = 0, device="cpu", stream=None, flags: int = 0):
    """Returns int32 tensors (chunk, zone, offset, src_token, pos_id) on `device`."""
    tc = c * t
    S = n_chunks * ((tc + t) if (flags & LOMA_FLAG_NO_REP_ZONE) else (2 * tc + t)) + tail_read
    on_device = torch.device(device).type == "cuda"
    outs = [torch.empty(max(S, 0), dtype=torch.int32, device=device) for _ in range(5)]
    st = _stream(stream) if on_device else None
    rc = lib().loma_layout_index(n_chunks, c, t, tail_read, int(flags), *[_ptr(x) for x in outs], int(on_device), st)
    _check(rc, "loma_layout_index")
    return tuple(outs)


def loma_generation_index(n_tokens: int, c: int, t: int, device="cpu", stream=None):
    """Returns int32 tensors (slot, pos_id, compress_after) on `device`."""
    on_device = torch.device(device).type == "cuda"
    outs = [torch.empty(max(n_tokens, 0), dtype=torch.int32, device=device) for _ in range(3)]
    st = _stream(stream) if on_device else None
    rc = lib().loma_generation_index(n_tokens, c, t, *[_ptr(x) for x in outs], int(on_device), st)
    _check(rc, "loma_generation_index")
    return tuple(outs)


def loma_masked_attn_fwd(q, k, v, o, lse, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0,
                         softmax_scale: float = 0.0, stream=None) -> None:
    """q, k, v, o: [B, H, S, D] device tensors with identical strides, D contiguous;
    lse: fp32 [B, H, S] contiguous or None."""
    B, H, S, D = q.shape
    for x in (k, v, o):
        if x.shape != q.shape or x.stride() != q.stride() or x.dtype != q.dtype:
            raise ValueError("q, k, v, o must share shape, strides and dtype")
    if q.stride(3) != 1:
        raise ValueError("head dimension must be contiguous")
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous()):
        raise ValueError("lse must be contiguous fp32")
    rc = lib().loma_masked_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, D, n_chunks, c, t, c * t,
                                    tail_read, q.stride(0), q.stride(1), q.stride(2), _dtype_code(q),
                                    float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_masked_attn_fwd")


def loma_masked_attn_bwd_workspace_bytes(B: int, H: int, D: int, n_chunks: int, c: int, t: int, tail_read: int = 0,
                                         flags: int = 0) -> int:
    return int(lib().loma_masked_attn_bwd_workspace_bytes(B, H, D, n_chunks, c, t, tail_read, int(flags)))


def loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n_chunks: int, c: int, t: int, tail_read: int = 0,
                         flags: int = 0, workspace=None, softmax_scale: float = 0.0, stream=None) -> None:
    """Gradients of loma_masked_attn_fwd.  q, k, v, o, d_o, dq, dk, dv: [B, H, S, D] device tensors with
    identical strides; lse: the forward's fp32 [B, H, S]; workspace: a device byte buffer of at least
    loma_masked_attn_bwd_workspace_bytes(...) bytes."""
    B, H, S, D = q.shape
    for x in (k, v, o, d_o, dq, dk, dv):
        if x.shape != q.shape or x.stride() != q.stride() or x.dtype != q.dtype:
            raise ValueError("all tensors must share shape, strides and dtype")
    if q.stride(3) != 1:
        raise ValueError("head dimension must be contiguous")
    if lse.dtype != torch.float32 or not lse.is_contiguous():
        raise ValueError("lse must be contiguous fp32")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_masked_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                                    _ptr(dv), B, H, D, n_chunks, c, t, c * t, tail_read, q.stride(0), q.stride(1),
                                    q.stride(2), _dtype_code(q), float(softmax_scale), int(flags), _ptr(workspace),
                                    ws_bytes, _stream(stream))
    _check(rc, "loma_masked_attn_bwd")


def loma_masked_attn_plan_coverage(n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0) -> torch.Tensor:
    """Host replay of the tensor-core kernel's tile plan: uint8 [S, S] visit counts."""
    S = n_chunks * ((c * t + t) if (flags & LOMA_FLAG_NO_REP_ZONE) else (2 * c * t + t)) + tail_read
    counts = torch.empty((S, S), dtype=torch.uint8)
    rc = lib().loma_masked_attn_plan_coverage(n_chunks, c, t, tail_read, int(flags), _ptr(counts))
    _check(rc, "loma_masked_attn_plan_coverage")
    return counts


def loma_prefill_attn(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, flags: int = 0,
                      softmax_scale: float = 0.0, stream=None) -> None:
    """q, k_new, v_new, o: [B, H, l, D] contiguous; caches [B, H, cap, D] contiguous; appends then attends."""
    B, H, l, D = q.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("loma_prefill_attn takes contiguous tensors")
    rc = lib().loma_prefill_attn(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse),
                                 B, H, D, l, k_cache.shape[2], int(cache_len), _dtype_code(q), float(softmax_scale),
                                 int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn")


def loma_prefill_attn_ragged(q, k_new, v_new, k_cache, v_cache, o, lse, cache_lens, max_cache_len: int, flags: int = 0,
                             softmax_scale: float = 0.0, stream=None) -> None:
    """loma_prefill_attn with one cache length per sequence (cache_lens: int32 [B] on the device)."""
    B, H, l, D = q.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("loma_prefill_attn_ragged takes contiguous tensors")
    if cache_lens.dtype != torch.int32 or cache_lens.numel() != B or not cache_lens.is_contiguous():
        raise ValueError("cache_lens must be a contiguous int32 tensor of B entries")
    rc = lib().loma_prefill_attn_ragged(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse),
                                        B, H, D, l, k_cache.shape[2], _ptr(cache_lens), int(max_cache_len), _dtype_code(q),
                                        float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn_ragged")


def loma_prefill_attn_paged(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, cache_lens, max_cache_len: int,
                            flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """loma_prefill_attn over a paged cache: pools [n_pages, H, page_size, D], block_table int32 [B, max_pages]."""
    B, H, l, D = q.shape
    for x in (q, k_new, v_new, k_pool, v_pool, o, block_table):
        if x is not None and not x.is_contiguous():
            raise ValueError("loma_prefill_attn_paged takes contiguous tensors")
    if cache_lens.dtype != torch.int32 or cache_lens.numel() != B or block_table.dtype != torch.int32:
        raise ValueError("cache_lens and block_table must be int32")
    n_pages, _, page_size, _ = k_pool.shape
    rc = lib().loma_prefill_attn_paged(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                       _ptr(o), _ptr(lse), B, H, D, l, page_size, block_table.shape[1], n_pages,
                                       _ptr(cache_lens), int(max_cache_len), _dtype_code(q), float(softmax_scale),
                                       int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn_paged")


def loma_prefill_attn_rope(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, pos0: int, flags: int = 0,
                           softmax_scale: float = 0.0, theta_base: float = 0.0, stream=None) -> None:
    """loma_prefill_attn with q and k_new rotated at the ids pos0 .. pos0 + l - 1 on the way in."""
    B, H, l, D = q.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("loma_prefill_attn_rope takes contiguous tensors")
    rc = lib().loma_prefill_attn_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse),
                                      B, H, D, l, k_cache.shape[2], int(cache_len), int(pos0), float(theta_base),
                                      _dtype_code(q), float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn_rope")


def loma_prefill_attn_ragged_rope(q, k_new, v_new, k_cache, v_cache, o, lse, cache_lens, max_cache_len: int, positions,
                                  flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0, stream=None) -> None:
    """loma_prefill_attn_ragged with the rotation fused in; positions: int32 [B], id of every sequence's first new token."""
    B, H, l, D = q.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("loma_prefill_attn_ragged_rope takes contiguous tensors")
    _check_positions(positions, B, "positions")
    rc = lib().loma_prefill_attn_ragged_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                             _ptr(lse), B, H, D, l, k_cache.shape[2], _ptr(cache_lens), int(max_cache_len),
                                             _ptr(positions), float(theta_base), _dtype_code(q), float(softmax_scale),
                                             int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn_ragged_rope")


def loma_prefill_attn_paged_rope(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, cache_lens, max_cache_len: int,
                                 positions, flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0,
                                 stream=None) -> None:
    """loma_prefill_attn_paged with the rotation fused in."""
    B, H, l, D = q.shape
    _check_positions(positions, B, "positions")
    n_pages, _, page_size, _ = k_pool.shape
    rc = lib().loma_prefill_attn_paged_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                            _ptr(o), _ptr(lse), B, H, D, l, page_size, block_table.shape[1], n_pages,
                                            _ptr(cache_lens), int(max_cache_len), _ptr(positions), float(theta_base),
                                            _dtype_code(q), float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_prefill_attn_paged_rope")


def loma_prefill_attn_plan_coverage(l: int, cache_len: int) -> torch.Tensor:
    """Host replay of the tensor-core kernel's tile plan for loma_prefill_attn: uint8 [l, cache_len + l] visit counts."""
    counts = torch.empty((l, cache_len + l), dtype=torch.uint8)
    rc = lib().loma_prefill_attn_plan_coverage(int(l), int(cache_len), _ptr(counts))
    _check(rc, "loma_prefill_attn_plan_coverage")
    return counts


def loma_masked_attn_bwd_plan_coverage(n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0) -> torch.Tensor:
    """Host replay of the key-tile side of the plan (the backward's dK/dV pass): uint8 [S, S] visit counts."""
    S = n_chunks * ((c * t + t) if (flags & LOMA_FLAG_NO_REP_ZONE) else (2 * c * t + t)) + tail_read
    counts = torch.empty((S, S), dtype=torch.uint8)
    rc = lib().loma_masked_attn_bwd_plan_coverage(n_chunks, c, t, tail_read, int(flags), _ptr(counts))
    _check(rc, "loma_masked_attn_bwd_plan_coverage")
    return counts


LOMA_ROPE_INVERSE = 2


def loma_rope_apply(q, k, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0, theta_base: float = 0.0,
                    position_type: int = 0, stream=None) -> None:
    """Rotates q and k ([B, H, S, D] device tensors with identical strides; either may be None) in place at
    the layout's position ids.  position_type 0: Eq. 14; 1: the generator's contiguous memory ids."""
    ref = q if q is not None else k
    B, H, S, D = ref.shape
    if q is not None and k is not None and (k.shape != q.shape or k.stride() != q.stride() or k.dtype != q.dtype):
        raise ValueError("q and k must share shape, strides and dtype")
    if ref.stride(3) != 1:
        raise ValueError("head dimension must be contiguous")
    rc = lib().loma_rope_apply(_ptr(q), _ptr(k), B, H, D, n_chunks, c, t, c * t, tail_read, ref.stride(0), ref.stride(1),
                               ref.stride(2), _dtype_code(ref), float(theta_base), int(position_type), int(flags),
                               _stream(stream))
    _check(rc, "loma_rope_apply")


def loma_prefill_cache(k, v, k_cache, v_cache, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0,
                       stream=None) -> int:
    """Gathers the memory-zone rows and the reading tail of laid-out k, v [B, H, S, D] into the caches
    [B, H, cap, D]; returns the new cache length."""
    B, H, S, D = k.shape
    if v.shape != k.shape or v.stride() != k.stride() or k.stride(3) != 1:
        raise ValueError("k and v must share shape and strides, head dimension contiguous")
    if not (k_cache.is_contiguous() and v_cache.is_contiguous()):
        raise ValueError("caches must be contiguous")
    n = ctypes.c_int(0)
    rc = lib().loma_prefill_cache(_ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache), B, H, D, k_cache.shape[2], n_chunks, c,
                                  t, c * t, tail_read, k.stride(0), k.stride(1), k.stride(2), _dtype_code(k), int(flags),
                                  ctypes.byref(n), _stream(stream))
    _check(rc, "loma_prefill_cache")
    return n.value


def loma_decode_workspace_bytes(B: int, H: int, D: int, cache_len: int) -> int:
    return int(lib().loma_decode_workspace_bytes(B, H, D, cache_len))


def loma_decode_attn(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, workspace=None, flags: int = 0,
                     softmax_scale: float = 0.0, stream=None) -> None:
    """q, k_new, v_new, o: [B, H, 1, D]; caches [B, H, cap, D]; all contiguous."""
    B, H, cap, D = k_cache.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                _ptr(lse), B, H, D, cap, cache_len, _dtype_code(q), float(softmax_scale),
                                int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn")


def _ptr_array(tensors):
    """[host] array of device pointers, one per layer (None stays NULL)."""
    if tensors is None:
        return None
    arr = (ctypes.c_void_p * len(tensors))()
    for i, x in enumerate(tensors):
        arr[i] = None if x is None else x.data_ptr()
    return arr


def loma_decode_attn_layers(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, workspace=None, flags: int = 0,
                            softmax_scale: float = 0.0, stream=None) -> None:
    """Lists of per-layer tensors (shapes of loma_decode_attn); k_new, v_new, lse may be None."""
    n = len(q)
    B, H, cap, D = k_cache[0].shape
    for group in (q, k_new, v_new, k_cache, v_cache, o):
        for x in (group or []):
            if x is not None and not x.is_contiguous():
                raise ValueError("decode tensors must be contiguous")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    arrays = [_ptr_array(x) for x in (q, k_new, v_new, k_cache, v_cache, o, lse)]
    rc = lib().loma_decode_attn_layers(n, *arrays, B, H, D, cap, cache_len, _dtype_code(q[0]), float(softmax_scale), int(flags),
                                       _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_layers")


def loma_compress_step_layers(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, mem_len: int, c: int, t: int, workspace=None,
                              flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """Lists of per-layer tensors (shapes of loma_compress_step); lse may be None."""
    n = len(q_mem)
    B, H, cap, D = k_cache[0].shape
    for group in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem):
        for x in group:
            if not x.is_contiguous():
                raise ValueError("compress tensors must be contiguous")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    arrays = [_ptr_array(x) for x in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse)]
    rc = lib().loma_compress_step_layers(n, *arrays, B, H, D, cap, mem_len, c, t, c * t, _dtype_code(q_mem[0]),
                                         float(softmax_scale), int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_compress_step_layers")


def loma_decode_attn_rope(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, pos: int, workspace=None,
                          flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0, stream=None) -> None:
    """loma_decode_attn with q and k_new rotated inside the step by the position id `pos`."""
    B, H, cap, D = k_cache.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                     _ptr(lse), B, H, D, cap, cache_len, int(pos), float(theta_base), _dtype_code(q),
                                     float(softmax_scale), int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_rope")


def loma_compress_step_rope(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, mem_len: int, c: int, t: int, pos0: int,
                            pos_stride: int, workspace=None, flags: int = 0, softmax_scale: float = 0.0,
                            theta_base: float = 0.0, stream=None) -> None:
    """loma_compress_step with memory row j's query and key rotated inside the step by the id pos0 + j * pos_stride."""
    B, H, cap, D = k_cache.shape
    for x in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if q_mem.shape[2] != t:
        raise ValueError("q_mem must have t rows")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_compress_step_rope(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_cache), _ptr(v_cache), _ptr(o_mem),
                                       _ptr(lse), B, H, D, cap, mem_len, c, t, c * t, int(pos0), int(pos_stride),
                                       float(theta_base), _dtype_code(q_mem), float(softmax_scale), int(flags),
                                       _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_compress_step_rope")


def loma_decode_attn_ragged(q, k_new, v_new, k_cache, v_cache, o, lse, cache_lens, max_cache_len: int, workspace=None,
                            flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """loma_decode_attn with one cache length per sequence: cache_lens is a device int32 [B] tensor,
    max_cache_len a host-side upper bound of its entries."""
    B, H, cap, D = k_cache.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o, cache_lens):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    if cache_lens.dtype != torch.int32 or cache_lens.numel() != B:
        raise ValueError("cache_lens must be int32 [B]")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn_ragged(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                       _ptr(lse), B, H, D, cap, _ptr(cache_lens), int(max_cache_len), _dtype_code(q),
                                       float(softmax_scale), int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_ragged")


def loma_decode_attn_paged(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, cache_lens, max_cache_len: int,
                           workspace=None, flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """Ragged decode over a paged cache.  k_pool, v_pool: [n_pages, H, page_size, D]; block_table: device int32
    [B, max_pages]; cache_lens: device int32 [B]; q, k_new, v_new, o: [B, H, 1, D]."""
    n_pages, H, page_size, D = k_pool.shape
    B, max_pages = block_table.shape
    for x in (q, k_new, v_new, k_pool, v_pool, o, block_table, cache_lens):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    if block_table.dtype != torch.int32 or cache_lens.dtype != torch.int32 or cache_lens.numel() != B:
        raise ValueError("block_table must be int32 [B, max_pages] and cache_lens int32 [B]")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn_paged(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                      _ptr(o), _ptr(lse), B, H, D, page_size, max_pages, n_pages, _ptr(cache_lens),
                                      int(max_cache_len), _dtype_code(q), float(softmax_scale), int(flags),
                                      _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_paged")


def _check_positions(positions, B, what):
    if positions.dtype != torch.int32 or positions.numel() != B or not positions.is_contiguous():
        raise ValueError(f"{what} must be a contiguous int32 [B] tensor")


def loma_decode_attn_ragged_rope(q, k_new, v_new, k_cache, v_cache, o, lse, cache_lens, max_cache_len: int, positions,
                                 workspace=None, flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0,
                                 stream=None) -> None:
    """loma_decode_attn_ragged with q and k_new of sequence b rotated inside the step by positions[b] (device int32 [B])."""
    B, H, cap, D = k_cache.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o, cache_lens):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    if cache_lens.dtype != torch.int32 or cache_lens.numel() != B:
        raise ValueError("cache_lens must be int32 [B]")
    _check_positions(positions, B, "positions")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn_ragged_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse),
                                            B, H, D, cap, _ptr(cache_lens), int(max_cache_len), _ptr(positions),
                                            float(theta_base), _dtype_code(q), float(softmax_scale), int(flags),
                                            _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_ragged_rope")


def loma_decode_attn_paged_rope(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, cache_lens, max_cache_len: int, positions,
                                workspace=None, flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0,
                                stream=None) -> None:
    """loma_decode_attn_paged with the rotation fused in (positions: device int32 [B])."""
    n_pages, H, page_size, D = k_pool.shape
    B, max_pages = block_table.shape
    for x in (q, k_new, v_new, k_pool, v_pool, o, block_table, cache_lens):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    if block_table.dtype != torch.int32 or cache_lens.dtype != torch.int32 or cache_lens.numel() != B:
        raise ValueError("block_table must be int32 [B, max_pages] and cache_lens int32 [B]")
    _check_positions(positions, B, "positions")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_decode_attn_paged_rope(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                           _ptr(o), _ptr(lse), B, H, D, page_size, max_pages, n_pages, _ptr(cache_lens),
                                           int(max_cache_len), _ptr(positions), float(theta_base), _dtype_code(q),
                                           float(softmax_scale), int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_decode_attn_paged_rope")


def loma_compress_step_ragged_rope(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, mem_lens, max_mem_len: int, c: int, t: int,
                                   pos0s, pos_stride: int, flags: int = 0, softmax_scale: float = 0.0, theta_base: float = 0.0,
                                   stream=None) -> None:
    """loma_compress_step_ragged with memory row j of sequence b rotated by pos0s[b] + j * pos_stride inside the step."""
    B, H, cap, D = k_cache.shape
    for x in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, mem_lens):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if mem_lens.dtype != torch.int32 or mem_lens.numel() != B:
        raise ValueError("mem_lens must be int32 [B]")
    _check_positions(pos0s, B, "pos0s")
    rc = lib().loma_compress_step_ragged_rope(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_cache), _ptr(v_cache), _ptr(o_mem),
                                              _ptr(lse), B, H, D, cap, _ptr(mem_lens), int(max_mem_len), c, t, c * t,
                                              _ptr(pos0s), int(pos_stride), float(theta_base), _dtype_code(q_mem),
                                              float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_compress_step_ragged_rope")


def loma_compress_step_paged_rope(q_mem, k_mem, v_mem, k_pool, v_pool, block_table, o_mem, lse, mem_lens, max_mem_len: int,
                                  c: int, t: int, pos0s, pos_stride: int, flags: int = 0, softmax_scale: float = 0.0,
                                  theta_base: float = 0.0, stream=None) -> None:
    """loma_compress_step_paged with the rotation fused in (pos0s: device int32 [B])."""
    n_pages, H, page_size, D = k_pool.shape
    B, max_pages = block_table.shape
    for x in (q_mem, k_mem, v_mem, k_pool, v_pool, o_mem, mem_lens, block_table):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if block_table.dtype != torch.int32 or mem_lens.dtype != torch.int32 or mem_lens.numel() != B:
        raise ValueError("block_table must be int32 [B, max_pages] and mem_lens int32 [B]")
    _check_positions(pos0s, B, "pos0s")
    rc = lib().loma_compress_step_paged_rope(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_pool), _ptr(v_pool),
                                             _ptr(block_table), _ptr(o_mem), _ptr(lse), B, H, D, page_size, max_pages, n_pages,
                                             _ptr(mem_lens), int(max_mem_len), c, t, c * t, _ptr(pos0s), int(pos_stride),
                                             float(theta_base), _dtype_code(q_mem), float(softmax_scale), int(flags),
                                             _stream(stream))
    _check(rc, "loma_compress_step_paged_rope")


def loma_decode_static_scratch_bytes() -> int:
    return int(lib().loma_decode_static_scratch_bytes())


def loma_decode_attn_static(q, k_new, v_new, k_cache, v_cache, o, lse, cache_len: int, softmax_scale: float = 0.0,
                            stream=None) -> None:
    """loma_decode_attn without a workspace argument: the split partials go to
    the library's built-in 8 MiB array, so the call needs no device memory beyond
    the tensors passed in.  Same tensor conventions as loma_decode_attn (bf16)."""
    B, H, cap, D = k_cache.shape
    for x in (q, k_new, v_new, k_cache, v_cache, o):
        if x is not None and not x.is_contiguous():
            raise ValueError("decode tensors must be contiguous")
    rc = lib().loma_decode_attn_static(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                       _ptr(lse), B, H, D, cap, cache_len, _dtype_code(q), float(softmax_scale),
                                       _stream(stream))
    _check(rc, "loma_decode_attn_static")


def loma_compress_step_ragged(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, mem_lens, max_mem_len: int, c: int, t: int,
                              flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """loma_compress_step with one count of memory entries per sequence (device int32 [B]; negative = the
    sequence does not compress in this call)."""
    B, H, cap, D = k_cache.shape
    for x in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, mem_lens):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if mem_lens.dtype != torch.int32 or mem_lens.numel() != B:
        raise ValueError("mem_lens must be int32 [B]")
    rc = lib().loma_compress_step_ragged(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_cache), _ptr(v_cache), _ptr(o_mem),
                                         _ptr(lse), B, H, D, cap, _ptr(mem_lens), int(max_mem_len), c, t, c * t,
                                         _dtype_code(q_mem), float(softmax_scale), int(flags), _stream(stream))
    _check(rc, "loma_compress_step_ragged")


def loma_compress_step_paged(q_mem, k_mem, v_mem, k_pool, v_pool, block_table, o_mem, lse, mem_lens, max_mem_len: int,
                             c: int, t: int, flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """Ragged compress over a paged cache (pools [n_pages, H, page_size, D], block_table int32 [B, max_pages])."""
    n_pages, H, page_size, D = k_pool.shape
    B, max_pages = block_table.shape
    for x in (q_mem, k_mem, v_mem, k_pool, v_pool, o_mem, mem_lens, block_table):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if block_table.dtype != torch.int32 or mem_lens.dtype != torch.int32 or mem_lens.numel() != B:
        raise ValueError("block_table must be int32 [B, max_pages] and mem_lens int32 [B]")
    rc = lib().loma_compress_step_paged(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                        _ptr(o_mem), _ptr(lse), B, H, D, page_size, max_pages, n_pages, _ptr(mem_lens),
                                        int(max_mem_len), c, t, c * t, _dtype_code(q_mem), float(softmax_scale), int(flags),
                                        _stream(stream))
    _check(rc, "loma_compress_step_paged")


def loma_compress_workspace_bytes(B: int, H: int, D: int, t: int, mem_len: int, flags: int = 0) -> int:
    return int(lib().loma_compress_workspace_bytes(B, H, D, t, mem_len, int(flags)))


def loma_compress_step(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, mem_len: int, c: int, t: int,
                       workspace=None, flags: int = 0, softmax_scale: float = 0.0, stream=None) -> None:
    """q_mem, k_mem, v_mem, o_mem: [B, H, t, D]; caches [B, H, cap, D]; all contiguous."""
    B, H, cap, D = k_cache.shape
    for x in (q_mem, k_mem, v_mem, k_cache, v_cache, o_mem):
        if not x.is_contiguous():
            raise ValueError("compress tensors must be contiguous")
    if q_mem.shape[2] != t:
        raise ValueError("q_mem must have t rows")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().loma_compress_step(_ptr(q_mem), _ptr(k_mem), _ptr(v_mem), _ptr(k_cache), _ptr(v_cache),
                                  _ptr(o_mem), _ptr(lse), B, H, D, cap, mem_len, c, t, c * t, _dtype_code(q_mem),
                                  float(softmax_scale), int(flags), _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "loma_compress_step")
