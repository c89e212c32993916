"""Thin ctypes binding of the C-ABI library ``libl4l.so`` (same names as ``include/l4l.h``).

Argument marshalling only: tensors become pointers + strides, the current CUDA stream
becomes a ``void*``. Every step of the attention path runs inside the library's kernels;
PyTorch is used for device memory and streams. There is no fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libl4l.so")

L4L_OK, L4L_ERR_INVALID_ARG, L4L_ERR_UNSUPPORTED, L4L_ERR_WORKSPACE, L4L_ERR_CUDA, L4L_ERR_TIMEOUT = range(6)
L4L_OP_PREFILL, L4L_OP_DECODE = 0, 1

EXPORTS = (
    "l4l_version", "l4l_status_string", "l4l_workspace_bytes", "l4l_workspace_init",
    "l4l_last_device_error", "l4l_kv_append", "l4l_attn_prefill", "l4l_attn_decode",
    "l4l_attn_decode_static", "l4l_attn_decode_append", "l4l_attn_prefill_chunk", "l4l_rope_kv_append",
    "l4l_kv_append_paged", "l4l_attn_decode_paged", "l4l_kv_append_fp8", "l4l_attn_decode_fp8", "l4l_rglru_scan", "l4l_rglru_workspace_bytes",
    "l4l_attn_decode_paged_fp8", "l4l_attn_merge", "l4l_attn_decode_rope_append", "l4l_attn_decode_paged_append",
    "l4l_attn_decode_paged_rope_append", "l4l_attn_decode_append_fp8", "l4l_attn_decode_paged_append_fp8",
    "l4l_attn_prefill_chunk_append", "l4l_attn_prefill_chunk_paged_append", "l4l_rglru_strip_channels",
    "l4l_decode_kernel_choice", "l4l_set_decode_override", "l4l_check_status", "l4l_selftest_wait_expiry",
    "l4l_attn_decode_rope_append_fp8", "l4l_attn_decode_paged_rope_append_fp8",
)
STATIC_SCRATCH_BYTES = 8 << 20


class Tensor4(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_b", ctypes.c_int64), ("stride_t", ctypes.c_int64),
                ("stride_h", ctypes.c_int64)]


class PagedKV(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("stride_page", ctypes.c_int64),
                ("stride_h", ctypes.c_int64), ("stride_t", ctypes.c_int64), ("page_size", ctypes.c_int32),
                ("num_pages", ctypes.c_int32)]


class KVCache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("stride_b", ctypes.c_int64),
                ("stride_h", ctypes.c_int64), ("stride_t", ctypes.c_int64), ("max_len", ctypes.c_int32)]


class L4LError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def load() -> ctypes.CDLL:
    """Opens libl4l.so; raises if it has not been built (``python -m paper_2608_21836_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2608_21836_b200.build`; there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    c_int, c_size, vp, i32p = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p
    lib.l4l_version.restype = ctypes.c_char_p
    lib.l4l_status_string.restype = ctypes.c_char_p
    lib.l4l_status_string.argtypes = [c_int]
    lib.l4l_workspace_bytes.restype = c_size
    lib.l4l_workspace_bytes.argtypes = [c_int] * 6
    lib.l4l_workspace_init.restype = c_int
    lib.l4l_workspace_init.argtypes = [vp, c_size, vp]
    lib.l4l_last_device_error.restype = c_int
    lib.l4l_last_device_error.argtypes = [vp, vp]
    lib.l4l_kv_append.restype = c_int
    lib.l4l_kv_append.argtypes = [KVCache, Tensor4, Tensor4, i32p, i32p, c_int, c_int, c_int, c_int, vp]
    lib.l4l_attn_prefill.restype = c_int
    lib.l4l_attn_prefill.argtypes = [Tensor4, Tensor4, Tensor4, Tensor4, KVCache, i32p, c_int, c_int, c_int, c_int,
                                     c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode.restype = c_int
    lib.l4l_attn_decode.argtypes = [vp, vp, KVCache, i32p, c_int, c_int, c_int, c_int, c_int, ctypes.c_float, vp,
                                    vp, c_size, vp]
    lib.l4l_attn_decode_static.restype = c_int
    lib.l4l_attn_decode_static.argtypes = [vp, vp, KVCache, i32p, c_int, c_int, c_int, c_int, c_int, ctypes.c_float, vp,
                                           vp]
    lib.l4l_kv_append_paged.restype = c_int
    lib.l4l_kv_append_paged.argtypes = [PagedKV, i32p, c_int, Tensor4, Tensor4, i32p, i32p, c_int, c_int, c_int, c_int, vp]
    lib.l4l_attn_decode_paged.restype = c_int
    lib.l4l_attn_decode_paged.argtypes = [vp, vp, PagedKV, i32p, c_int, i32p, c_int, c_int, c_int, c_int, c_int,
                                          ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_paged_append.restype = c_int
    lib.l4l_attn_decode_paged_append.argtypes = [vp, vp, PagedKV, i32p, c_int, Tensor4, Tensor4, i32p, c_int, c_int, c_int,
                                                 c_int, c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_paged_rope_append.restype = c_int
    lib.l4l_attn_decode_paged_rope_append.argtypes = [vp, vp, PagedKV, i32p, c_int, Tensor4, Tensor4, i32p, c_int, c_int,
                                                      c_int, c_int, c_int, ctypes.c_float, vp, vp, c_int, vp, vp,
                                                      ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_append_fp8.restype = c_int
    lib.l4l_attn_decode_append_fp8.argtypes = [vp, vp, KVCache, vp, vp, Tensor4, Tensor4, i32p, c_int, c_int, c_int, c_int,
                                               c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_paged_append_fp8.restype = c_int
    lib.l4l_attn_decode_paged_append_fp8.argtypes = [vp, vp, PagedKV, vp, vp, i32p, c_int, Tensor4, Tensor4, i32p, c_int,
                                                     c_int, c_int, c_int, c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_rope_append_fp8.restype = c_int
    lib.l4l_attn_decode_rope_append_fp8.argtypes = [vp, vp, KVCache, vp, vp, Tensor4, Tensor4, i32p, c_int, c_int, c_int,
                                                    c_int, c_int, ctypes.c_float, vp, vp, c_int, vp, vp, ctypes.c_float,
                                                    vp, vp, c_size, vp]
    lib.l4l_attn_decode_paged_rope_append_fp8.restype = c_int
    lib.l4l_attn_decode_paged_rope_append_fp8.argtypes = [vp, vp, PagedKV, vp, vp, i32p, c_int, Tensor4, Tensor4, i32p,
                                                          c_int, c_int, c_int, c_int, c_int, ctypes.c_float, vp, vp, c_int,
                                                          vp, vp, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_decode_kernel_choice.restype = c_int
    lib.l4l_decode_kernel_choice.argtypes = [c_int, c_int, c_int, c_int, c_int, c_int, ctypes.POINTER(c_int)]
    lib.l4l_set_decode_override.restype = None
    lib.l4l_set_decode_override.argtypes = [c_int, c_int, c_int]
    lib.l4l_check_status.restype = c_int
    lib.l4l_check_status.argtypes = [vp, vp]
    lib.l4l_selftest_wait_expiry.restype = c_int
    lib.l4l_selftest_wait_expiry.argtypes = [vp, c_size, ctypes.c_longlong, vp]
    lib.l4l_kv_append_fp8.restype = c_int
    lib.l4l_kv_append_fp8.argtypes = [KVCache, Tensor4, Tensor4, i32p, i32p, c_int, c_int, c_int, c_int, vp, vp, vp]
    lib.l4l_attn_decode_fp8.restype = c_int
    lib.l4l_attn_decode_fp8.argtypes = [vp, vp, KVCache, vp, vp, i32p, c_int, c_int, c_int, c_int, c_int,
                                        ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_paged_fp8.restype = c_int
    lib.l4l_attn_decode_paged_fp8.argtypes = [vp, vp, PagedKV, vp, vp, i32p, c_int, i32p, c_int, c_int, c_int, c_int, c_int,
                                              ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_rope_append.restype = c_int
    lib.l4l_attn_decode_rope_append.argtypes = [vp, vp, KVCache, Tensor4, Tensor4, i32p, c_int, c_int, c_int, c_int, c_int,
                                                ctypes.c_float, vp, vp, c_int, vp, vp, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_merge.restype = c_int
    lib.l4l_attn_merge.argtypes = [vp, vp, c_int, vp, vp, c_int, c_int, c_int, vp]
    lib.l4l_rglru_workspace_bytes.restype = c_size
    lib.l4l_rglru_workspace_bytes.argtypes = [c_int, c_int, c_int]
    lib.l4l_rglru_strip_channels.restype = c_int
    lib.l4l_rglru_strip_channels.argtypes = [c_int, c_int, c_int]
    lib.l4l_rglru_scan.restype = c_int
    lib.l4l_rglru_scan.argtypes = [vp, vp, vp, vp, i32p, i32p, vp, vp, c_int, c_int, c_int, vp, c_size, vp]
    lib.l4l_rope_kv_append.restype = c_int
    lib.l4l_rope_kv_append.argtypes = [Tensor4, Tensor4, Tensor4, KVCache, i32p, i32p, c_int, c_int, c_int, c_int, c_int,
                                       vp, vp, c_int, vp, vp, ctypes.c_float, vp]
    lib.l4l_attn_prefill_chunk.restype = c_int
    lib.l4l_attn_prefill_chunk.argtypes = [Tensor4, Tensor4, KVCache, i32p, i32p, c_int, c_int, c_int, c_int, c_int,
                                           ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_prefill_chunk_append.restype = c_int
    lib.l4l_attn_prefill_chunk_append.argtypes = [Tensor4, Tensor4, Tensor4, Tensor4, KVCache, i32p, i32p, c_int, c_int,
                                                  c_int, c_int, c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_prefill_chunk_paged_append.restype = c_int
    lib.l4l_attn_prefill_chunk_paged_append.argtypes = [Tensor4, Tensor4, Tensor4, Tensor4, PagedKV, i32p, c_int, i32p, i32p,
                                                        c_int, c_int, c_int, c_int, c_int, ctypes.c_float, vp, vp, c_size, vp]
    lib.l4l_attn_decode_append.restype = c_int
    lib.l4l_attn_decode_append.argtypes = [vp, vp, KVCache, Tensor4, Tensor4, i32p, c_int, c_int, c_int, c_int, c_int,
                                           ctypes.c_float, vp, vp, c_size, vp]
    _lib = lib
    return lib


def version() -> str:
    return load().l4l_version().decode()


def status_string(status: int) -> str:
    return load().l4l_status_string(int(status)).decode()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check_bf16_cuda(t: torch.Tensor, name: str) -> None:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.stride(-1) == 1):
        raise TypeError(f"{name} must be a CUDA bfloat16 tensor with a contiguous last dimension")


def tensor4(t: torch.Tensor, name: str = "tensor") -> Tensor4:
    """[B, T, H, D] view -> l4l_tensor4."""
    _check_bf16_cuda(t, name)
    if t.dim() != 4:
        raise ValueError(f"{name} must have 4 dimensions [B, T, H, D]")
    return Tensor4(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def kv_cache(cache_k: Optional[torch.Tensor], cache_v: Optional[torch.Tensor]) -> KVCache:
    """Caches indexed [B, Hkv, slot, D] (any strides with D contiguous) -> l4l_kv_cache; (None, None) -> no cache."""
    if cache_k is None and cache_v is None:
        return KVCache(None, None, 0, 0, 0, 0)
    _check_bf16_cuda(cache_k, "cache_k")
    _check_bf16_cuda(cache_v, "cache_v")
    if cache_k.dim() != 4 or cache_k.shape != cache_v.shape or cache_k.stride() != cache_v.stride():
        raise ValueError("cache_k and cache_v must be [B, Hkv, max_len, D] views with equal shapes and strides")
    return KVCache(cache_k.data_ptr(), cache_v.data_ptr(), cache_k.stride(0), cache_k.stride(1), cache_k.stride(2),
                   cache_k.shape[2])


def _i32_dev(t: Optional[torch.Tensor], name: str) -> Optional[int]:
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA int32 tensor")
    return t.data_ptr()


def l4l_workspace_bytes(op: int, B: int, Hq: int, Hkv: int, head_dim: int, max_len: int) -> int:
    return int(load().l4l_workspace_bytes(op, B, Hq, Hkv, head_dim, max_len))


def l4l_workspace_init(workspace: torch.Tensor) -> None:
    st = load().l4l_workspace_init(workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_workspace_init")


def new_workspace(op: int, B: int, Hq: int, Hkv: int, head_dim: int, max_len: int, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and initialises a workspace of the size the library asks for."""
    n = l4l_workspace_bytes(op, B, Hq, Hkv, head_dim, max_len)
    if n == 0:
        raise L4LError(L4L_ERR_UNSUPPORTED, "l4l_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    l4l_workspace_init(ws)
    return ws


def l4l_last_device_error(workspace: torch.Tensor) -> int:
    return int(load().l4l_last_device_error(workspace.data_ptr(), _stream()))


def l4l_kv_append(cache_k, cache_v, k_new, v_new, write_pos, n_new=None) -> None:
    """cache [B,Hkv,max_len,D]; k_new/v_new [B,T,Hkv,D]; write_pos, n_new: CUDA int32 [B]."""
    B, T, Hkv, D = k_new.shape
    st = load().l4l_kv_append(kv_cache(cache_k, cache_v), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                              _i32_dev(write_pos, "write_pos"), _i32_dev(n_new, "n_new"), T, B, Hkv, D, _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_kv_append")


def l4l_attn_prefill(q, k, v, o, seq_lens, scale: float, workspace, cache_k=None, cache_v=None, lse=None) -> None:
    """q,o [B,S,Hq,D]; k,v [B,S,Hkv,D]; seq_lens CUDA int32 [B]; lse optional CUDA float32 [B,Hq,S]."""
    B, S, Hq, D = q.shape
    Hkv = k.shape[2]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq, S)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq, S]")
    st = load().l4l_attn_prefill(tensor4(q, "q"), tensor4(k, "k"), tensor4(v, "v"), tensor4(o, "o"),
                                 kv_cache(cache_k, cache_v), _i32_dev(seq_lens, "seq_lens"), S, B, Hq, Hkv, D,
                                 float(scale), None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_prefill")


def l4l_attn_decode(q, o, cache_k, cache_v, kv_lens, max_kv_len: int, scale: float, workspace, lse=None) -> None:
    """q,o dense [B,Hq,D]; cache [B,Hkv,max_len,D]; kv_lens CUDA int32 [B] (current token included)."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k.shape[1]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    st = load().l4l_attn_decode(q.data_ptr(), o.data_ptr(), kv_cache(cache_k, cache_v),
                                _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode")


def l4l_attn_decode_static(q, o, cache_k, cache_v, kv_lens, max_kv_len: int, scale: float, lse=None) -> None:
    """Decode for callers that may not allocate: same arguments as l4l_attn_decode but no workspace.

    The scratch is a fixed array of STATIC_SCRATCH_BYTES inside the library, shared by every call on the
    device, so calls that could overlap on the GPU must be ordered by the caller. Problems whose partials
    do not fit raise L4LError(L4L_ERR_WORKSPACE). Make the first call on a device during start-up."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k.shape[1]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    st = load().l4l_attn_decode_static(q.data_ptr(), o.data_ptr(), kv_cache(cache_k, cache_v),
                                       _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                       None if lse is None else lse.data_ptr(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_static")


def l4l_attn_decode_append(q, o, cache_k, cache_v, k_new, v_new, kv_lens, max_kv_len: int, scale: float, workspace,
                           lse=None) -> None:
    """One launch per decode step: writes k_new / v_new ([B,1,Hkv,D]) into cache slot kv_lens[b]-1 and attends
    over slots 0..kv_lens[b]-1. Same result as l4l_kv_append followed by l4l_attn_decode."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k.shape[1]
    if tuple(k_new.shape) != (B, 1, Hkv, D) or tuple(v_new.shape) != (B, 1, Hkv, D):
        raise ValueError("k_new and v_new must be [B, 1, Hkv, D]")
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    st = load().l4l_attn_decode_append(q.data_ptr(), o.data_ptr(), kv_cache(cache_k, cache_v),
                                       tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                                       _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                       None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                       workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_append")


def l4l_attn_prefill_chunk(q, o, cache_k, cache_v, past_lens, q_lens, scale: float, workspace, lse=None) -> None:
    """Chunk of new tokens over a populated cache. q,o [B,S,Hq,D]; the chunk's K/V are already in the cache at
    slots past..past+q_len-1; past_lens, q_lens CUDA int32 [B]; lse optional CUDA float32 [B,Hq,S]."""
    B, S, Hq, D = q.shape
    Hkv = cache_k.shape[1]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq, S)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq, S]")
    st = load().l4l_attn_prefill_chunk(tensor4(q, "q"), tensor4(o, "o"), kv_cache(cache_k, cache_v),
                                       _i32_dev(past_lens, "past_lens"), _i32_dev(q_lens, "q_lens"), S, B, Hq, Hkv, D,
                                       float(scale), None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                       workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_prefill_chunk")


def l4l_attn_prefill_chunk_append(q, k_new, v_new, o, cache_k, cache_v, past_lens, q_lens, scale: float, workspace,
                                  lse=None, block_table=None) -> None:
    """Chunk of new tokens over a populated cache with the cache update fused in (one launch). q,o [B,S,Hq,D];
    k_new, v_new [B,S,Hkv,D] go to slots past..past+q_len-1. With block_table (CUDA int32 [B, n]) cache_k / cache_v
    are a page pool [pages,Hkv,page_size,D]; without it a contiguous cache [B,Hkv,max_len,D]."""
    B, S, Hq, D = q.shape
    Hkv = k_new.shape[2]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq, S)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq, S]")
    common = (_i32_dev(past_lens, "past_lens"), _i32_dev(q_lens, "q_lens"), S, B, Hq, Hkv, D, float(scale),
              None if lse is None else lse.data_ptr(), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
              _stream())
    if block_table is None:
        st = load().l4l_attn_prefill_chunk_append(tensor4(q, "q"), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                                                  tensor4(o, "o"), kv_cache(cache_k, cache_v), *common)
    else:
        tbl, stride = _block_table(block_table, B)
        st = load().l4l_attn_prefill_chunk_paged_append(tensor4(q, "q"), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                                                        tensor4(o, "o"), paged_kv(cache_k, cache_v), tbl, stride, *common)
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_prefill_chunk_append")


def _f32_dev(t, name: str, shape=None):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA float32 tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}")
    return t.data_ptr()


def l4l_rope_kv_append(q, k_new, v_new, cache_k, cache_v, pos, n_new, cos, sin, q_weight=None, k_weight=None,
                       eps: float = 0.0) -> None:
    """Rotary embedding (+ optional per-head RMS norm) of q (in place) and k, with K and V written to the cache.
    q [B,T,Hq,D]; k_new, v_new [B,T,Hkv,D]; pos CUDA int32 [B]; n_new CUDA int32 [B] or None;
    cos, sin CUDA float32 [n_pos, D/2]; q_weight, k_weight CUDA float32 [D] or None."""
    B, T, Hq, D = q.shape
    Hkv = k_new.shape[2]
    n_pos = cos.shape[0]
    st = load().l4l_rope_kv_append(tensor4(q, "q"), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                                   kv_cache(cache_k, cache_v), _i32_dev(pos, "pos"),
                                   None if n_new is None else _i32_dev(n_new, "n_new"), T, B, Hq, Hkv, D,
                                   _f32_dev(cos, "cos", (n_pos, D // 2)), _f32_dev(sin, "sin", (n_pos, D // 2)), n_pos,
                                   _f32_dev(q_weight, "q_weight", (D,)), _f32_dev(k_weight, "k_weight", (D,)),
                                   float(eps), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_rope_kv_append")


def paged_kv(pool_k, pool_v) -> PagedKV:
    """Page pools indexed [page, Hkv, slot, D] (any strides with D contiguous) -> l4l_paged_kv."""
    _check_bf16_cuda(pool_k, "pool_k")
    _check_bf16_cuda(pool_v, "pool_v")
    if pool_k.dim() != 4 or pool_k.shape != pool_v.shape or pool_k.stride() != pool_v.stride():
        raise ValueError("pool_k and pool_v must be [pages, Hkv, page_size, D] views with equal shapes and strides")
    return PagedKV(pool_k.data_ptr(), pool_v.data_ptr(), pool_k.stride(0), pool_k.stride(1), pool_k.stride(2),
                   pool_k.shape[2], pool_k.shape[0])


def _block_table(t, B: int):
    if not (t.is_cuda and t.dtype == torch.int32 and t.dim() == 2 and t.shape[0] == B and t.is_contiguous()):
        raise TypeError("block_table must be a contiguous CUDA int32 tensor [B, pages per sequence]")
    return t.data_ptr(), t.shape[1]


def l4l_kv_append_paged(pool_k, pool_v, block_table, k_new, v_new, write_pos, n_new=None) -> None:
    """k_new, v_new [B,T,Hkv,D] into the pages of a paged cache; write_pos CUDA int32 [B]."""
    B, T, Hkv, D = k_new.shape
    tbl, stride = _block_table(block_table, B)
    st = load().l4l_kv_append_paged(paged_kv(pool_k, pool_v), tbl, stride, tensor4(k_new, "k_new"),
                                    tensor4(v_new, "v_new"), _i32_dev(write_pos, "write_pos"),
                                    None if n_new is None else _i32_dev(n_new, "n_new"), T, B, Hkv, D, _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_kv_append_paged")


def l4l_attn_decode_paged(q, o, pool_k, pool_v, block_table, kv_lens, max_kv_len: int, scale: float, workspace,
                          lse=None) -> None:
    """Decode over a paged cache. q,o dense [B,Hq,D]; pools [pages,Hkv,page_size,D]; block_table CUDA int32 [B, n]."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = pool_k.shape[1]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    tbl, stride = _block_table(block_table, B)
    st = load().l4l_attn_decode_paged(q.data_ptr(), o.data_ptr(), paged_kv(pool_k, pool_v), tbl, stride,
                                      _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                      None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                      workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_paged")


def l4l_attn_decode_paged_append(q, o, pool_k, pool_v, block_table, k_new, v_new, kv_lens, max_kv_len: int, scale: float,
                                 workspace, lse=None) -> None:
    """One launch per decode step over a paged cache: k_new / v_new ([B,1,Hkv,D]) go to slot kv_lens[b]-1 of sequence b
    (the page the block table names) and are attended with the rest. Same result as l4l_kv_append_paged followed by
    l4l_attn_decode_paged."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = pool_k.shape[1]
    if tuple(k_new.shape) != (B, 1, Hkv, D) or tuple(v_new.shape) != (B, 1, Hkv, D):
        raise ValueError("k_new and v_new must be [B, 1, Hkv, D]")
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    tbl, stride = _block_table(block_table, B)
    st = load().l4l_attn_decode_paged_append(q.data_ptr(), o.data_ptr(), paged_kv(pool_k, pool_v), tbl, stride,
                                             tensor4(k_new), tensor4(v_new), _i32_dev(kv_lens, "kv_lens"),
                                             int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                             None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                             workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_paged_append")


def l4l_attn_decode_paged_rope_append(q, o, pool_k, pool_v, block_table, k_new, v_new, kv_lens, max_kv_len: int,
                                      scale: float, cos, sin, workspace, q_weight=None, k_weight=None, eps: float = 0.0,
                                      lse=None) -> None:
    """l4l_attn_decode_rope_append over a paged cache: rotation (+ optional RMS norm) of q and k_new at position
    kv_lens - 1, write of the rotated k and of v_new into the page slot, attention: one launch."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = pool_k.shape[1]
    if tuple(k_new.shape) != (B, 1, Hkv, D) or tuple(v_new.shape) != (B, 1, Hkv, D):
        raise ValueError("k_new and v_new must be [B, 1, Hkv, D]")
    n_pos = cos.shape[0]
    tbl, stride = _block_table(block_table, B)
    st = load().l4l_attn_decode_paged_rope_append(
        q.data_ptr(), o.data_ptr(), paged_kv(pool_k, pool_v), tbl, stride, tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
        _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
        _f32_dev(cos, "cos", (n_pos, D // 2)), _f32_dev(sin, "sin", (n_pos, D // 2)), n_pos,
        _f32_dev(q_weight, "q_weight", (D,)), _f32_dev(k_weight, "k_weight", (D,)), float(eps),
        None if lse is None else lse.data_ptr(), workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_paged_rope_append")


def l4l_attn_decode_rope_append_fp8(q, o, cache_k8, cache_v8, k_scale, v_scale, k_new, v_new, kv_lens, max_kv_len: int,
                                    scale: float, cos, sin, workspace, q_weight=None, k_weight=None, eps: float = 0.0,
                                    lse=None, block_table=None) -> None:
    """One launch per decode step over an fp8 cache with the rotation fused in: q and k_new are rotated (+ optional RMS
    norm) at position kv_lens - 1, the rotated k (rounded to bf16) and v_new are quantised as l4l_kv_append_fp8 does and
    written to slot kv_lens - 1, the rotated q attends. With block_table, the caches are a page pool."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k8.shape[1]
    if tuple(k_new.shape) != (B, 1, Hkv, D) or tuple(v_new.shape) != (B, 1, Hkv, D):
        raise ValueError("k_new and v_new must be [B, 1, Hkv, D]")
    n_pos = cos.shape[0]
    c = kv_cache8(cache_k8, cache_v8)
    common = (tensor4(k_new, "k_new"), tensor4(v_new, "v_new"), _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv,
              D, float(scale), _f32_dev(cos, "cos", (n_pos, D // 2)), _f32_dev(sin, "sin", (n_pos, D // 2)), n_pos,
              _f32_dev(q_weight, "q_weight", (D,)), _f32_dev(k_weight, "k_weight", (D,)), float(eps),
              None if lse is None else lse.data_ptr(), workspace.data_ptr(),
              workspace.numel() * workspace.element_size(), _stream())
    ks, vs = _f32_dev(k_scale, "k_scale", (Hkv,)), _f32_dev(v_scale, "v_scale", (Hkv,))
    if block_table is None:
        st = load().l4l_attn_decode_rope_append_fp8(q.data_ptr(), o.data_ptr(), c, ks, vs, *common)
    else:
        pool = PagedKV(c.k, c.v, c.stride_b, c.stride_h, c.stride_t, cache_k8.shape[2], cache_k8.shape[0])
        tbl, stride = _block_table(block_table, B)
        st = load().l4l_attn_decode_paged_rope_append_fp8(q.data_ptr(), o.data_ptr(), pool, ks, vs, tbl, stride, *common)
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_rope_append_fp8")


def kv_cache8(cache_k8, cache_v8) -> KVCache:
    """fp8 caches indexed [B, Hkv, slot, D], dtype uint8 or float8_e4m3fn -> l4l_kv_cache with byte strides."""
    for t, name in ((cache_k8, "cache_k8"), (cache_v8, "cache_v8")):
        if not (t.is_cuda and t.dtype in (torch.uint8, torch.float8_e4m3fn) and t.dim() == 4 and t.stride(-1) == 1):
            raise TypeError(f"{name} must be a CUDA uint8 / float8_e4m3fn tensor [B, Hkv, max_len, D] with D contiguous")
    if cache_k8.shape != cache_v8.shape or cache_k8.stride() != cache_v8.stride():
        raise ValueError("cache_k8 and cache_v8 must have equal shapes and strides")
    return KVCache(cache_k8.data_ptr(), cache_v8.data_ptr(), cache_k8.stride(0), cache_k8.stride(1), cache_k8.stride(2),
                   cache_k8.shape[2])


def l4l_kv_append_fp8(cache_k8, cache_v8, k_new, v_new, write_pos, k_scale, v_scale, n_new=None) -> None:
    """k_new, v_new [B,T,Hkv,D] bf16, divided by the per-KV-head scales and rounded to e4m3, into the fp8 cache."""
    B, T, Hkv, D = k_new.shape
    st = load().l4l_kv_append_fp8(kv_cache8(cache_k8, cache_v8), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
                                  _i32_dev(write_pos, "write_pos"), None if n_new is None else _i32_dev(n_new, "n_new"),
                                  T, B, Hkv, D, _f32_dev(k_scale, "k_scale", (Hkv,)), _f32_dev(v_scale, "v_scale", (Hkv,)),
                                  _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_kv_append_fp8")


def l4l_attn_decode_fp8(q, o, cache_k8, cache_v8, k_scale, v_scale, kv_lens, max_kv_len: int, scale: float, workspace,
                        lse=None) -> None:
    """Decode over an fp8 (e4m3) cache with per-KV-head scales. q,o dense bf16 [B,Hq,D] (at head_dim 64 the cache's
    token rows must be dense and even in number)."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k8.shape[1]
    if lse is not None and not (lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                                and tuple(lse.shape) == (B, Hq)):
        raise TypeError("lse must be a contiguous CUDA float32 tensor [B, Hq]")
    st = load().l4l_attn_decode_fp8(q.data_ptr(), o.data_ptr(), kv_cache8(cache_k8, cache_v8),
                                    _f32_dev(k_scale, "k_scale", (Hkv,)), _f32_dev(v_scale, "v_scale", (Hkv,)),
                                    _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                    None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_fp8")


def l4l_rglru_scan(x, gate_x, gate_a, a_param, state, y, workspace, position=None, seq_lens=None) -> None:
    """Gated linear recurrence (RG-LRU) over the sequence. x, gate_x, gate_a, y dense CUDA bf16 [B,T,W];
    a_param CUDA float32 [W]; state CUDA float32 [B,W] (in/out); position CUDA int32 [B,T] or None;
    seq_lens CUDA int32 [B] or None."""
    for t, name in ((x, "x"), (gate_x, "gate_x"), (gate_a, "gate_a"), (y, "y")):
        _check_bf16_cuda(t, name)
        if not (t.dim() == 3 and t.is_contiguous() and t.shape == x.shape):
            raise ValueError(f"{name} must be a dense [B, T, W] tensor of the same shape as x")
    B, T, W = x.shape
    if position is not None and not (position.is_cuda and position.dtype == torch.int32 and position.is_contiguous()
                                     and tuple(position.shape) == (B, T)):
        raise TypeError("position must be a contiguous CUDA int32 tensor [B, T]")
    st = load().l4l_rglru_scan(x.data_ptr(), gate_x.data_ptr(), gate_a.data_ptr(), _f32_dev(a_param, "a_param", (W,)),
                               None if position is None else position.data_ptr(),
                               None if seq_lens is None else _i32_dev(seq_lens, "seq_lens"),
                               _f32_dev(state, "state", (B, W)), y.data_ptr(), B, T, W, workspace.data_ptr(),
                               workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_rglru_scan")


def new_rglru_workspace(B: int, T: int, W: int, device=None) -> torch.Tensor:
    """Zeroed workspace for l4l_rglru_scan, large enough for the segment-parallel mode at these sizes."""
    n = int(load().l4l_rglru_workspace_bytes(B, T, W))
    if n == 0:
        raise ValueError("unsupported sizes")
    ws = torch.zeros((n + 7) // 8, dtype=torch.int64, device=device or "cuda")
    return ws


def l4l_attn_decode_paged_fp8(q, o, pool_k8, pool_v8, k_scale, v_scale, block_table, kv_lens, max_kv_len: int, scale: float,
                              workspace, lse=None) -> None:
    """Decode over an fp8 page pool [pages, Hkv, page_size, 128] (uint8 / float8_e4m3fn) read through a block table."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    c = kv_cache8(pool_k8, pool_v8)                     # same checks; fields reinterpreted as a page pool
    pool = PagedKV(c.k, c.v, c.stride_b, c.stride_h, c.stride_t, pool_k8.shape[2], pool_k8.shape[0])
    Hkv = pool_k8.shape[1]
    tbl, stride = _block_table(block_table, B)
    st = load().l4l_attn_decode_paged_fp8(q.data_ptr(), o.data_ptr(), pool, _f32_dev(k_scale, "k_scale", (Hkv,)),
                                          _f32_dev(v_scale, "v_scale", (Hkv,)), tbl, stride, _i32_dev(kv_lens, "kv_lens"),
                                          int(max_kv_len), B, Hq, Hkv, D, float(scale),
                                          None if lse is None else lse.data_ptr(), workspace.data_ptr(),
                                          workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_paged_fp8")


def l4l_attn_decode_append_fp8(q, o, cache_k8, cache_v8, k_scale, v_scale, k_new, v_new, kv_lens, max_kv_len: int,
                               scale: float, workspace, lse=None, block_table=None) -> None:
    """One launch per decode step over an fp8 cache: bf16 k_new / v_new ([B,1,Hkv,128]) are quantised as
    l4l_kv_append_fp8 does, written to slot kv_lens[b]-1 and attended with the rest. With block_table, cache_k8 /
    cache_v8 are a page pool [pages, Hkv, page_size, 128]."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k8.shape[1]
    if tuple(k_new.shape) != (B, 1, Hkv, D) or tuple(v_new.shape) != (B, 1, Hkv, D):
        raise ValueError("k_new and v_new must be [B, 1, Hkv, D]")
    c = kv_cache8(cache_k8, cache_v8)
    common = (tensor4(k_new, "k_new"), tensor4(v_new, "v_new"), _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv,
              D, float(scale), None if lse is None else lse.data_ptr(), workspace.data_ptr(),
              workspace.numel() * workspace.element_size(), _stream())
    ks, vs = _f32_dev(k_scale, "k_scale", (Hkv,)), _f32_dev(v_scale, "v_scale", (Hkv,))
    if block_table is None:
        st = load().l4l_attn_decode_append_fp8(q.data_ptr(), o.data_ptr(), c, ks, vs, *common)
    else:
        pool = PagedKV(c.k, c.v, c.stride_b, c.stride_h, c.stride_t, cache_k8.shape[2], cache_k8.shape[0])
        tbl, stride = _block_table(block_table, B)
        st = load().l4l_attn_decode_paged_append_fp8(q.data_ptr(), o.data_ptr(), pool, ks, vs, tbl, stride, *common)
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_append_fp8")


def l4l_decode_kernel_choice(B: int, Hq: int, Hkv: int, D: int, max_kv_len: int, fp8: bool = False):
    """(name, detail) of the kernel the decode calls would run for these sizes on the current device: ("split", consumer
    warps), ("cluster", CTAs per cluster) or ("warp", 0); None for sizes the calls reject."""
    detail = ctypes.c_int(0)
    k = load().l4l_decode_kernel_choice(B, Hq, Hkv, D, int(max_kv_len), int(bool(fp8)), ctypes.byref(detail))
    return None if k < 0 else (("split", "cluster", "warp")[k], detail.value)


_override = {"cluster": -1, "warp": -1, "split_warps": 0}


def l4l_set_decode_override(cluster: int = -1, warp: int = -1, split_warps: int = 0) -> None:
    """Process-wide tuning override of the decode kernel choice (see the header); the defaults restore the library's own
    choice."""
    load().l4l_set_decode_override(int(cluster), int(warp), int(split_warps))
    _override.update(cluster=int(cluster), warp=int(warp), split_warps=int(split_warps))


class decode_override:
    """``with decode_override(cluster=0): ...`` holds the decode calls of the block on one kernel and puts the previous
    settings back afterwards. Only the settings that are named change."""

    def __init__(self, cluster: Optional[int] = None, warp: Optional[int] = None, split_warps: Optional[int] = None):
        self.want = {k: v for k, v in (("cluster", cluster), ("warp", warp), ("split_warps", split_warps)) if v is not None}

    def __enter__(self):
        self.old = dict(_override)
        l4l_set_decode_override(**{**self.old, **self.want})
        return self

    def __exit__(self, *exc):
        l4l_set_decode_override(**self.old)
        return False


def l4l_check_status(workspace: Optional[torch.Tensor] = None) -> int:
    """L4L_OK, or L4L_ERR_TIMEOUT if a bounded device-side wait has run out since the status block was cleared
    (synchronises the stream). workspace=None: the status block of the library's own scratch array."""
    return int(load().l4l_check_status(None if workspace is None else workspace.data_ptr(), _stream()))


def l4l_selftest_wait_expiry(workspace: torch.Tensor, budget_cycles: int = 100000) -> None:
    """Launches the one-warp kernel whose bounded wait runs out by construction (see the header)."""
    st = load().l4l_selftest_wait_expiry(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                         int(budget_cycles), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_selftest_wait_expiry")


def l4l_rglru_strip_channels(B: int, T: int, W: int) -> int:
    """Channels per strip (64, 32 or 16) the scan would use for these sizes on the current device."""
    return int(load().l4l_rglru_strip_channels(int(B), int(T), int(W)))


def l4l_attn_merge(o_parts, lse_parts, o, lse=None) -> None:
    """Combines R partial decode results over disjoint key ranges. o_parts CUDA bf16 [R,B,Hq,D]; lse_parts CUDA
    float32 [R,B,Hq]; o CUDA bf16 [B,Hq,D]; lse optional CUDA float32 [B,Hq]."""
    _check_bf16_cuda(o_parts, "o_parts")
    _check_bf16_cuda(o, "o")
    R, B, Hq, D = o_parts.shape
    if not (o_parts.is_contiguous() and o.is_contiguous() and tuple(o.shape) == (B, Hq, D)):
        raise ValueError("o_parts must be dense [R, B, Hq, D] and o dense [B, Hq, D]")
    st = load().l4l_attn_merge(o_parts.data_ptr(), _f32_dev(lse_parts, "lse_parts", (R, B, Hq)), R, o.data_ptr(),
                               None if lse is None else _f32_dev(lse, "lse", (B, Hq)), B, Hq, D, _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_merge")


def l4l_attn_decode_rope_append(q, o, cache_k, cache_v, k_new, v_new, kv_lens, max_kv_len: int, scale: float, cos, sin,
                                workspace, q_weight=None, k_weight=None, eps: float = 0.0, lse=None) -> None:
    """One launch per decode step: rotary embedding (+ optional RMS norm) of q and k_new at position kv_lens - 1, cache
    update and attention. q,o dense [B,Hq,D] (q is not modified); k_new, v_new [B,1,Hkv,D]; cos, sin CUDA float32
    [n_pos, D/2]."""
    _check_bf16_cuda(q, "q")
    _check_bf16_cuda(o, "o")
    if not (q.is_contiguous() and o.is_contiguous() and q.dim() == 3 and q.shape == o.shape):
        raise ValueError("q and o must be dense [B, Hq, D]")
    B, Hq, D = q.shape
    Hkv = cache_k.shape[1]
    n_pos = cos.shape[0]
    st = load().l4l_attn_decode_rope_append(
        q.data_ptr(), o.data_ptr(), kv_cache(cache_k, cache_v), tensor4(k_new, "k_new"), tensor4(v_new, "v_new"),
        _i32_dev(kv_lens, "kv_lens"), int(max_kv_len), B, Hq, Hkv, D, float(scale),
        _f32_dev(cos, "cos", (n_pos, D // 2)), _f32_dev(sin, "sin", (n_pos, D // 2)), n_pos,
        _f32_dev(q_weight, "q_weight", (D,)), _f32_dev(k_weight, "k_weight", (D,)), float(eps),
        None if lse is None else lse.data_ptr(), workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream())
    if st != L4L_OK:
        raise L4LError(st, "l4l_attn_decode_rope_append")
