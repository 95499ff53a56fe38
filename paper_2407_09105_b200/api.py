"""Python binding of the C-ABI library (``include/pk.h``): same names, argument
marshalling only.  Tensors are torch CUDA tensors used as device memory; every step of
the path runs inside ``libpk.so``.  There is no CPU fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

PK_OK = 0
PK_ERR_INVALID_ARG = 1
PK_ERR_UNSUPPORTED = 2
PK_ERR_WORKSPACE = 3
PK_ERR_CUDA = 4
PK_ERR_BAD_POSIDS = 5
PK_ERR_TIMEOUT = 6
PK_ERR_NO_PLAN = 7

PK_ERR_TOO_LARGE = 8
PK_NOALLOC_MAX_TOKENS = 32768

PK_BF16 = 0
PK_F32 = 1
PK_REUSE_PLAN, PK_REUSE_ROTATED = 1, 2

PK_WS_HEADER, PK_WS_FWD_ITEMS, PK_WS_BWD_ITEMS, PK_WS_FWD_ORDER, PK_WS_BWD_ORDER = range(5)
PK_WS_DELTA, PK_WS_DQ_ACC, PK_WS_ROPE_TABLE = 5, 6, 7
PK_HDR_STATUS, PK_HDR_DETAIL, PK_HDR_N_EXAMPLES, PK_HDR_MAX_SEQLEN, PK_HDR_N_ITEMS, PK_HDR_PLAN_T = range(6)

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpk.so")
_lib = None

_i32, _sz, _vp, _f32 = ctypes.c_int32, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_float

_SIGNATURES = {
    "pk_tile_shape": (ctypes.c_int, [ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pk_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "pk_workspace_section": (ctypes.c_int, [_i32, _i32, _i32, _i32, _i32,
                                            ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "pk_seqlens_from_posids": (ctypes.c_int, [_vp, _i32, _vp, _vp, _vp, _vp, _sz, _vp]),
    "pk_rope_apply": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _f32, _i32, _vp]),
    "pk_attn_fwd": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _f32, _f32, _i32,
                                   _vp, _i32, _vp, _i32, _vp, _sz, _vp]),
    "pk_attn_bwd": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp,
                                   _i32, _i32, _i32, _i32, _f32, _f32, _i32,
                                   _vp, _vp, _vp, _i32, _i32, _vp, _sz, _vp]),
    "pk_status_read": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pk_set_timing_events": (ctypes.c_int, [_i32, _vp, _vp]),
    "pk_set_rope_mode": (ctypes.c_int, [_i32]),
    "pk_collate_padding_free": (ctypes.c_int, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _i32, _vp]),
    "pk_collate_fixed_length": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp]),
    "pk_pack_first_fit_decreasing": (ctypes.c_int, [_vp, _i32, _i32, _vp, ctypes.POINTER(_i32)]),
    "pk_pack_next_fit": (ctypes.c_int, [_vp, _i32, _i32, _i32, _vp, ctypes.POINTER(_i32)]),
    "pk_pack_rows": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, ctypes.c_int64, _vp, _vp]),
    "pk_unpack_rows": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i32, ctypes.c_int64, _vp, _vp]),
    "pk_packed_loss_fwd": (ctypes.c_int, [_vp, _i32, _vp, _i32, _i32, ctypes.c_int64, _i32, _vp, _vp,
                                          _vp, _vp, _vp]),
    "pk_packed_loss_bwd": (ctypes.c_int, [_vp, _i32, _vp, _vp, _vp, ctypes.c_float, _i32, _i32,
                                          ctypes.c_int64, _i32, _vp, _vp]),
    "pk_selftest_bounded_wait": (ctypes.c_int, [_vp, ctypes.c_int64, _vp]),
    "pk_seqlens_from_posids_noalloc": (ctypes.c_int, [_vp, _i32, _vp, _vp, _vp, _vp]),
}

EXPORTED_SYMBOLS = tuple(_SIGNATURES)


class PkError(RuntimeError):
    def __init__(self, fn: str, code: int):
        super().__init__(f"{fn} failed with code {code}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Loads ``libpk.so`` (built by ``paper_2407_09105_b200.build``); fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} not found: build it with `python -m paper_2407_09105_b200.build`")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def _check(fn: str, code: int) -> None:
    if code != PK_OK:
        raise PkError(fn, code)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return PK_BF16
    if t.dtype == torch.float32:
        return PK_F32
    raise ValueError(f"unsupported dtype {t.dtype}")


def pk_tile_shape() -> Tuple[int, int]:
    bm, bn = _i32(), _i32()
    _check("pk_tile_shape", lib().pk_tile_shape(ctypes.byref(bm), ctypes.byref(bn)))
    return bm.value, bn.value


def pk_workspace_bytes(T: int, Hq: int, Hkv: int, D: int) -> int:
    return int(lib().pk_workspace_bytes(T, Hq, Hkv, D))


def pk_workspace_section(which: int, T: int, Hq: int, Hkv: int, D: int) -> Tuple[int, int]:
    off, nb = _sz(), _sz()
    _check("pk_workspace_section",
           lib().pk_workspace_section(which, T, Hq, Hkv, D, ctypes.byref(off), ctypes.byref(nb)))
    return off.value, nb.value


def alloc_workspace(T: int, Hq: int, Hkv: int, D: int, device="cuda") -> torch.Tensor:
    """A uint8 torch tensor of ``pk_workspace_bytes`` bytes (torch's allocator returns
    512-byte aligned blocks)."""
    n = pk_workspace_bytes(T, Hq, Hkv, D)
    if n == 0:
        raise PkError("pk_workspace_bytes", PK_ERR_UNSUPPORTED)
    return torch.empty(n, dtype=torch.uint8, device=device)


def pk_seqlens_from_posids(position_ids: torch.Tensor, cu_seqlens: torch.Tensor,
                           n_examples: torch.Tensor, max_seqlen: torch.Tensor,
                           workspace: torch.Tensor, stream=None) -> None:
    T = position_ids.numel()
    _check("pk_seqlens_from_posids",
           lib().pk_seqlens_from_posids(_ptr(position_ids), T, _ptr(cu_seqlens), _ptr(n_examples),
                                        _ptr(max_seqlen), _ptr(workspace), workspace.numel(),
                                        _stream(stream)))


def pk_seqlens_from_posids_noalloc(position_ids: torch.Tensor, cu_seqlens: torch.Tensor,
                                   n_examples: torch.Tensor, max_seqlen: torch.Tensor,
                                   stream=None) -> None:
    """Boundary recovery with the library's built-in scratch: no workspace argument and no
    allocation of any kind.  For callers that must not (or cannot) allocate device memory --
    e.g. a collation thread running while the framework's caching allocator owns the GPU's
    memory.  At most ``PK_NOALLOC_MAX_TOKENS`` tokens; calls on one device share the scratch,
    so keep them ordered on the GPU."""
    T = position_ids.numel()
    _check("pk_seqlens_from_posids_noalloc",
           lib().pk_seqlens_from_posids_noalloc(_ptr(position_ids), T, _ptr(cu_seqlens),
                                                _ptr(n_examples), _ptr(max_seqlen),
                                                _stream(stream)))


def pk_rope_apply(x: torch.Tensor, position_ids: torch.Tensor, theta: float,
                  inverse: bool = False, stream=None) -> None:
    T, H, D = x.shape
    _check("pk_rope_apply",
           lib().pk_rope_apply(_ptr(x), _ptr(position_ids), T, H, D, theta, int(inverse),
                               _stream(stream)))


def pk_attn_fwd(q, k, v, position_ids, softmax_scale: float, rope_theta: float,
                out: torch.Tensor, lse: torch.Tensor, workspace: torch.Tensor,
                reuse_plan: bool = False, window: int = 0, stream=None) -> None:
    """``window`` > 0: sliding-window attention (each row sees its ``window`` most recent keys)."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    _check("pk_attn_fwd",
           lib().pk_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(position_ids), T, Hq, Hkv, D,
                             softmax_scale, rope_theta, int(window), _ptr(out), _dtype_code(out),
                             _ptr(lse), int(reuse_plan), _ptr(workspace), workspace.numel(),
                             _stream(stream)))


def pk_attn_bwd(dout, q, k, v, out, lse, position_ids, softmax_scale: float, rope_theta: float,
                dq: torch.Tensor, dk: torch.Tensor, dv: torch.Tensor, workspace: torch.Tensor,
                reuse_plan: bool = True, reuse_rotated: bool = False, window: int = 0,
                stream=None) -> None:
    """``reuse_rotated``: the rotated q / k copies the forward left in ``workspace`` are still
    valid (same q, k, position_ids, rope_theta; workspace untouched since).  ``window``: the
    forward's sliding window (0 = none)."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    if not (dq.dtype == dk.dtype == dv.dtype):
        raise ValueError("dq, dk, dv must share a dtype")
    _check("pk_attn_bwd",
           lib().pk_attn_bwd(_ptr(dout), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _dtype_code(out),
                             _ptr(lse), _ptr(position_ids), T, Hq, Hkv, D, softmax_scale,
                             rope_theta, int(window), _ptr(dq), _ptr(dk), _ptr(dv), _dtype_code(dq),
                             (PK_REUSE_PLAN if reuse_plan else 0) |
                             (PK_REUSE_ROTATED if reuse_rotated else 0),
                             _ptr(workspace), workspace.numel(), _stream(stream)))


def pk_status_read(workspace: torch.Tensor, stream=None) -> Tuple[int, int]:
    code, detail = _i32(), _i32()
    _check("pk_status_read",
           lib().pk_status_read(_ptr(workspace), _stream(stream), ctypes.byref(code),
                                ctypes.byref(detail)))
    return code.value, detail.value


(PK_KERNEL_PLAN, PK_KERNEL_FWD, PK_KERNEL_DELTA, PK_KERNEL_BWD, PK_KERNEL_DQ_FINISH, PK_KERNEL_BWD_DQ,
 PK_KERNEL_LOSS_FWD, PK_KERNEL_LOSS_BWD) = range(8)


def pk_set_timing_events(which: int, start: Optional[torch.cuda.Event],
                         stop: Optional[torch.cuda.Event]) -> None:
    """``start``/``stop`` must have been created with ``enable_timing=True`` and recorded
    once (torch creates the underlying event lazily); ``None`` clears the hook."""
    s = None if start is None else start.cuda_event
    e = None if stop is None else stop.cuda_event
    _check("pk_set_timing_events", lib().pk_set_timing_events(which, s, e))


PK_ROPE_ROTATED_COPIES, PK_ROPE_IN_TILE = 0, 1


def pk_set_rope_mode(mode: int) -> None:
    _check("pk_set_rope_mode", lib().pk_set_rope_mode(mode))


def pk_collate_padding_free(input_ids: torch.Tensor, lengths: torch.Tensor,
                            position_ids: torch.Tensor, labels: Optional[torch.Tensor],
                            cu_seqlens: torch.Tensor, ignore_index: int = -100, stream=None) -> None:
    _check("pk_collate_padding_free",
           lib().pk_collate_padding_free(_ptr(input_ids), _ptr(lengths), lengths.numel(),
                                         position_ids.numel(), _ptr(position_ids), _ptr(labels),
                                         _ptr(cu_seqlens), ignore_index, _stream(stream)))


def pk_collate_fixed_length(input_ids: torch.Tensor, lengths: torch.Tensor, msl: int,
                            position_ids: torch.Tensor, labels: Optional[torch.Tensor],
                            cu_seqlens: torch.Tensor, ignore_index: int = -100, stream=None) -> None:
    _check("pk_collate_fixed_length",
           lib().pk_collate_fixed_length(_ptr(input_ids), _ptr(lengths), lengths.numel(),
                                         position_ids.numel(), msl, _ptr(position_ids),
                                         _ptr(labels), _ptr(cu_seqlens), ignore_index,
                                         _stream(stream)))


def _row_bytes(t: torch.Tensor, lead: int) -> int:
    n = 1
    for d in t.shape[lead:]:
        n *= d
    return n * t.element_size()


def pk_pack_rows(padded: torch.Tensor, cu_seqlens: torch.Tensor, packed: torch.Tensor,
                 stream=None) -> None:
    """padded [B, l_max, ...] -> packed [T, ...] (same trailing shape and dtype)."""
    B, l_max = padded.shape[:2]
    _check("pk_pack_rows",
           lib().pk_pack_rows(_ptr(padded), _ptr(cu_seqlens), B, l_max, packed.shape[0],
                              _row_bytes(packed, 1), _ptr(packed), _stream(stream)))


def pk_unpack_rows(packed: torch.Tensor, cu_seqlens: torch.Tensor, padded: torch.Tensor,
                   stream=None) -> None:
    """packed [T, ...] -> padded [B, l_max, ...]; padding rows become zero."""
    B, l_max = padded.shape[:2]
    _check("pk_unpack_rows",
           lib().pk_unpack_rows(_ptr(packed), _ptr(cu_seqlens), B, l_max, packed.shape[0],
                                _row_bytes(packed, 1), _ptr(padded), _stream(stream)))


def _logits_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return PK_BF16
    if t.dtype == torch.float32:
        return PK_F32
    raise ValueError("logits must be bfloat16 or float32")


def pk_packed_loss_fwd(logits: torch.Tensor, labels: torch.Tensor, token_loss: torch.Tensor,
                       lse: torch.Tensor, result: torch.Tensor, n_valid: torch.Tensor,
                       ignore_index: int = -100, stream=None) -> None:
    """logits [T, V] (rows may be padded: stride(0) >= V, stride(1) == 1)."""
    T, V = logits.shape
    if logits.stride(1) != 1 and T > 0:
        raise ValueError("logits rows must be contiguous")
    stride = logits.stride(0) if T > 1 else V
    _check("pk_packed_loss_fwd",
           lib().pk_packed_loss_fwd(logits.data_ptr(), _logits_dtype(logits), _ptr(labels), T, V,
                                    stride, ignore_index, _ptr(token_loss), _ptr(lse),
                                    _ptr(result), _ptr(n_valid), _stream(stream)))


def pk_packed_loss_bwd(logits: torch.Tensor, labels: torch.Tensor, lse: torch.Tensor,
                       n_valid: torch.Tensor, grad_out: float, dlogits: torch.Tensor,
                       ignore_index: int = -100, stream=None) -> None:
    T, V = logits.shape
    if dlogits.shape != logits.shape or dlogits.dtype != logits.dtype or \
            dlogits.stride() != logits.stride():
        raise ValueError("dlogits must match logits in shape, dtype and strides")
    stride = logits.stride(0) if T > 1 else V
    _check("pk_packed_loss_bwd",
           lib().pk_packed_loss_bwd(logits.data_ptr(), _logits_dtype(logits), _ptr(labels),
                                    _ptr(lse), _ptr(n_valid), float(grad_out), T, V, stride,
                                    ignore_index, dlogits.data_ptr(), _stream(stream)))


def _pack(fn_name, lengths, capacity, *extra):
    import numpy as np
    arr = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    out = np.empty_like(arr)
    nb = _i32()
    fn = getattr(lib(), fn_name)
    _check(fn_name, fn(arr.ctypes.data, arr.size, capacity, *extra, out.ctypes.data,
                       ctypes.byref(nb)))
    return out.tolist(), nb.value


def pk_pack_first_fit_decreasing(lengths, capacity: int):
    """Host-side: (bin index per example, number of bins)."""
    return _pack("pk_pack_first_fit_decreasing", lengths, capacity)


def pk_pack_next_fit(lengths, capacity: int, sort_descending: bool):
    return _pack("pk_pack_next_fit", lengths, capacity, int(sort_descending))


def pk_selftest_bounded_wait(workspace: torch.Tensor, budget_cycles: int, stream=None) -> None:
    _check("pk_selftest_bounded_wait",
           lib().pk_selftest_bounded_wait(_ptr(workspace), budget_cycles, _stream(stream)))


def workspace_view(workspace: torch.Tensor, which: int, T: int, Hq: int, Hkv: int, D: int,
                   dtype=torch.int32) -> torch.Tensor:
    """A typed view of one workspace section (for inspection and tests)."""
    off, nb = pk_workspace_section(which, T, Hq, Hkv, D)
    return workspace[off:off + nb].view(dtype)
