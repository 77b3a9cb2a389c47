"""Thin ctypes binding of the C ABI in ``include/attn.h`` and ``include/gemm_rowsum.h`` -- argument marshalling only.

Every step of the attention forward pass (and of the GEMM + row sum) runs inside the CUDA kernels of
``libb200attn.so``.  torch is used for device memory and streams.  There is no CPU or
library fallback: if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

from .build import LIB_PATH

ATTN_OK = 0
ATTN_BF16, ATTN_FP32 = 0, 1
ATTN_NORM_SOFTMAX, ATTN_NORM_SIGMOID, ATTN_NORM_RELU = 0, 1, 2
ATTN_MASK_CAUSAL, ATTN_MASK_WINDOW, ATTN_MASK_DOCUMENT, ATTN_MASK_PREFIX, ATTN_MASK_TEST_QUERY = 1, 2, 4, 8, 16
ATTN_MASK_GLOBAL = 32


class AttnVariantDesc(ctypes.Structure):
    """Mirror of ``attn_variant_desc``."""

    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("dtype", ctypes.c_uint32),
        ("o_dtype", ctypes.c_uint32),
        ("normalizer", ctypes.c_uint32),
        ("mask_flags", ctypes.c_uint32),
        ("window_left", ctypes.c_int32),
        ("window_right", ctypes.c_int32),
        ("scale", ctypes.c_float),
        ("softcap", ctypes.c_float),
        ("bias_slopes", ctypes.c_void_p),
        ("sigmoid_bias", ctypes.c_float),
        ("out_scale", ctypes.c_float),
        ("cu_seqlens", ctypes.c_void_p),
        ("num_docs", ctypes.c_int32),
        ("prefix_len", ctypes.c_int32),
        ("test_query_start", ctypes.c_int32),
        ("global_len", ctypes.c_int32),
        ("q_strides", ctypes.c_int64 * 3),
        ("k_strides", ctypes.c_int64 * 3),
        ("v_strides", ctypes.c_int64 * 3),
        ("o_strides", ctypes.c_int64 * 3),
        ("status_word", ctypes.c_void_p),
    ]


class AttnError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"call failed: {status_string(status)} (status {status})")


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2605_05023_b200/build.py` "
        "(there is no fallback path)")

_lib = ctypes.CDLL(LIB_PATH)
_lib.attn_fwd.restype = ctypes.c_int
_lib.attn_fwd.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 6 + [
    ctypes.POINTER(AttnVariantDesc), ctypes.c_void_p]
_lib.attn_fwd_host.restype = ctypes.c_int
_lib.attn_fwd_host.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 6 + [
    ctypes.POINTER(AttnVariantDesc), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
_lib.attn_host_workspace_bytes.restype = ctypes.c_size_t
_lib.attn_host_workspace_bytes.argtypes = [ctypes.c_int] * 6 + [ctypes.POINTER(AttnVariantDesc)]
_lib.attn_status_string.restype = ctypes.c_char_p
_lib.attn_status_string.argtypes = [ctypes.c_int]
_lib.attn_version.restype = ctypes.c_int
_lib.attn_launch_count.restype = ctypes.c_int64
_lib.attn_clear_cache.restype = ctypes.c_int
_lib.attn_cache_hits.restype = ctypes.c_int64
_lib.attn_selftest_timeout.restype = ctypes.c_int
_lib.attn_selftest_timeout.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p]


def status_string(status: int) -> str:
    return _lib.attn_status_string(int(status)).decode()


def version() -> int:
    return int(_lib.attn_version())


def launch_count() -> int:
    return int(_lib.attn_launch_count())


def clear_cache() -> int:
    """``attn_clear_cache``: empties the cache of encoded tensor maps."""
    return int(_lib.attn_clear_cache())


def cache_hits() -> int:
    return int(_lib.attn_cache_hits())


def selftest_timeout(status_word: torch.Tensor, limit_ns: int, second_waiter: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> int:
    """``attn_selftest_timeout``: one bounded wait that runs out, on purpose; returns the attn_status of the launch."""
    st = stream if stream is not None else torch.cuda.current_stream(status_word.device)
    return int(_lib.attn_selftest_timeout(status_word.data_ptr(), int(limit_ns),
                                          second_waiter.data_ptr() if second_waiter is not None else None, st.cuda_stream))


def raw_attn_fwd(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D,
                 desc: Optional[AttnVariantDesc], stream_ptr) -> int:
    """The C call itself, pointers as integers; returns the attn_status."""
    return int(_lib.attn_fwd(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D,
                             ctypes.byref(desc) if desc is not None else None, stream_ptr))


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return ATTN_BF16
    if dt == torch.float32:
        return ATTN_FP32
    raise TypeError(f"unsupported element type {dt}")


def _strides3(t: torch.Tensor):
    if t.stride(3) != 1:
        raise ValueError("the innermost dimension must be dense")
    return (ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def make_desc(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, o: torch.Tensor, *,
              causal: bool = False, window_left: Optional[int] = None,
              window_right: Optional[int] = None, scale: Optional[float] = None,
              softcap: float = 0.0, slopes: Optional[torch.Tensor] = None,
              normalizer: str = "softmax", sigmoid_bias: float = 0.0, out_scale: float = 1.0,
              cu_seqlens: Optional[torch.Tensor] = None, prefix_len: Optional[int] = None,
              test_query_start: Optional[int] = None, global_len: Optional[int] = None,
              status_word: Optional[torch.Tensor] = None) -> AttnVariantDesc:
    d = AttnVariantDesc()
    d.struct_size = ctypes.sizeof(AttnVariantDesc)
    d.dtype = _dtype_code(q.dtype)
    d.o_dtype = _dtype_code(o.dtype)
    d.normalizer = {"softmax": ATTN_NORM_SOFTMAX, "sigmoid": ATTN_NORM_SIGMOID, "relu": ATTN_NORM_RELU}[normalizer]
    flags = 0
    if causal:
        flags |= ATTN_MASK_CAUSAL
    if window_left is not None or window_right is not None:
        flags |= ATTN_MASK_WINDOW
    d.window_left = -1 if window_left is None else int(window_left)
    d.window_right = -1 if window_right is None else int(window_right)
    d.scale = 0.0 if scale is None else float(scale)
    d.softcap = float(softcap)
    if slopes is not None:
        if slopes.dtype != torch.float32 or not slopes.is_cuda or not slopes.is_contiguous():
            raise TypeError("slopes must be a contiguous fp32 device tensor [Hq]")
        d.bias_slopes = slopes.data_ptr()
    d.sigmoid_bias = float(sigmoid_bias)
    d.out_scale = float(out_scale)
    if cu_seqlens is not None:
        if cu_seqlens.dtype != torch.int32 or not cu_seqlens.is_cuda or not cu_seqlens.is_contiguous():
            raise TypeError("cu_seqlens must be a contiguous int32 device tensor")
        flags |= ATTN_MASK_DOCUMENT
        d.cu_seqlens = cu_seqlens.data_ptr()
        d.num_docs = cu_seqlens.numel() - 1
    if prefix_len is not None:
        flags |= ATTN_MASK_PREFIX
        d.prefix_len = int(prefix_len)
    if test_query_start is not None:
        flags |= ATTN_MASK_TEST_QUERY
        d.test_query_start = int(test_query_start)
    if global_len is not None:
        flags |= ATTN_MASK_GLOBAL
        d.global_len = int(global_len)
    d.mask_flags = flags
    d.q_strides = _strides3(q)
    d.k_strides = _strides3(k)
    d.v_strides = _strides3(v)
    d.o_strides = _strides3(o)
    if status_word is not None:
        d.status_word = status_word.data_ptr()
    return d


def attn_fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, *,
             o: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
             o_dtype: Optional[torch.dtype] = None, want_lse: bool = True,
             stream: Optional[torch.cuda.Stream] = None, **variant) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """Fused attention forward on the current CUDA device (see ``include/attn.h``).

    q [B,Hq,Sq,D], k, v [B,Hkv,Sk,D] device tensors (bf16 or fp32).  ``variant`` takes the
    keyword arguments of :func:`make_desc`.  Returns (O, LSE); LSE is None for the sigmoid and
    ReLU normalisers or when ``want_lse`` is False.  The call is asynchronous on ``stream``.
    """
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise ValueError("q, k, v must be CUDA tensors: this library has no CPU path")
    B, Hq, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    if v.shape != k.shape or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v shapes")
    if o is None:
        o = torch.empty((B, Hq, Sq, D), device=q.device, dtype=o_dtype or q.dtype)
    sigmoid = variant.get("normalizer", "softmax") != "softmax"      # no row normalisation: no LSE
    if lse is None and want_lse and not sigmoid:
        lse = torch.empty((B, Hq, Sq), device=q.device, dtype=torch.float32)
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous()):
        raise TypeError("lse must be a contiguous fp32 tensor [B,Hq,Sq]")
    desc = make_desc(q, k, v, o, **variant)
    st = stream if stream is not None else torch.cuda.current_stream(q.device)
    rc = raw_attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                      lse.data_ptr() if lse is not None else None,
                      B, Hq, Hkv, Sq, Sk, D, desc, st.cuda_stream)
    if rc != ATTN_OK:
        raise AttnError(rc)
    return o, (None if sigmoid else lse)


def host_workspace_bytes(B, Hq, Hkv, Sq, Sk, D, desc: AttnVariantDesc) -> int:
    return int(_lib.attn_host_workspace_bytes(B, Hq, Hkv, Sq, Sk, D, ctypes.byref(desc)))


def attn_fwd_host(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, o: torch.Tensor,
                  lse: Optional[torch.Tensor], workspace: torch.Tensor, *,
                  stream: Optional[torch.cuda.Stream] = None, **variant) -> None:
    """``attn_fwd_host`` of the C ABI: q, k, v, o, lse are contiguous HOST tensors (pin them for
    asynchronous copies); ``workspace`` is a uint8 device tensor of at least
    :func:`host_workspace_bytes` bytes.  Enqueues copies and the kernel on ``stream``."""
    for t in (q, k, v, o) + ((lse,) if lse is not None else ()):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("attn_fwd_host takes contiguous host tensors")
    B, Hq, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    desc = AttnVariantDesc()
    tmp = make_desc(q, k, v, o, **variant)
    ctypes.memmove(ctypes.byref(desc), ctypes.byref(tmp), ctypes.sizeof(desc))
    for name in ("q_strides", "k_strides", "v_strides", "o_strides"):
        setattr(desc, name, (ctypes.c_int64 * 3)(0, 0, 0))
    st = stream if stream is not None else torch.cuda.current_stream(workspace.device)
    rc = int(_lib.attn_fwd_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                lse.data_ptr() if lse is not None else None,
                                B, Hq, Hkv, Sq, Sk, D, ctypes.byref(desc), workspace.data_ptr(),
                                workspace.numel() * workspace.element_size(), st.cuda_stream))
    if rc != ATTN_OK:
        raise AttnError(rc)


def variant_kwargs(w, device) -> dict:
    """Keyword arguments of :func:`make_desc` for a ``synth_inputs.Workload`` description."""
    kw = dict(causal=w.causal, window_left=w.window_left, window_right=w.window_right,
              scale=w.scale, softcap=w.softcap, normalizer=w.normalizer,
              sigmoid_bias=w.sigmoid_bias, out_scale=w.out_scale, prefix_len=w.prefix_len,
              test_query_start=w.test_query_start, global_len=w.global_len)
    if w.slopes is not None:
        kw["slopes"] = torch.tensor(w.slopes, dtype=torch.float32, device=device)
    if w.cu_seqlens is not None:
        kw["cu_seqlens"] = torch.tensor(w.cu_seqlens, dtype=torch.int32, device=device)
    return kw


# ------------------------------------------------------------------------------------------------
# GEMM + row sum (include/gemm_rowsum.h): argument marshalling only
# ------------------------------------------------------------------------------------------------
class GemmRowsumDesc(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("reserved", ctypes.c_uint32),
        ("lda", ctypes.c_int64),
        ("ldb", ctypes.c_int64),
        ("ldc", ctypes.c_int64),
        ("status_word", ctypes.c_void_p),
    ]


_lib.gemm_rowsum.restype = ctypes.c_int
_lib.gemm_rowsum.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 3 + [ctypes.POINTER(GemmRowsumDesc), ctypes.c_void_p]
_lib.gemm_rowsum_host.restype = ctypes.c_int
_lib.gemm_rowsum_host.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 3 + [
    ctypes.POINTER(GemmRowsumDesc), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
_lib.gemm_rowsum_host_workspace_bytes.restype = ctypes.c_size_t
_lib.gemm_rowsum_host_workspace_bytes.argtypes = [ctypes.c_int] * 3
_lib.gemm_rowsum_launch_count.restype = ctypes.c_int64


def raw_gemm_rowsum(a_ptr, b_ptr, c_ptr, rowsum_ptr, M, N, K, desc: Optional[GemmRowsumDesc], stream_ptr) -> int:
    """Direct call of the C entry point with raw addresses; returns the status."""
    return int(_lib.gemm_rowsum(a_ptr, b_ptr, c_ptr, rowsum_ptr, M, N, K,
                                ctypes.byref(desc) if desc is not None else None, stream_ptr))


def gemm_rowsum_launch_count() -> int:
    return int(_lib.gemm_rowsum_launch_count())


def gemm_rowsum_host_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.gemm_rowsum_host_workspace_bytes(M, N, K))


def _gemm_desc(a=None, b=None, c=None, status_word: Optional[torch.Tensor] = None) -> GemmRowsumDesc:
    d = GemmRowsumDesc()
    d.struct_size = ctypes.sizeof(GemmRowsumDesc)
    d.lda = a.stride(0) if a is not None else 0
    d.ldb = b.stride(0) if b is not None else 0
    d.ldc = c.stride(0) if c is not None else 0
    d.status_word = status_word.data_ptr() if status_word is not None else None
    return d


def gemm_rowsum(a: torch.Tensor, b: torch.Tensor, *, c: Optional[torch.Tensor] = None, want_c: bool = True,
                rowsum: Optional[torch.Tensor] = None, status_word: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None) -> Tuple[Optional[torch.Tensor], torch.Tensor]:
    """``C = A B`` and the row sums of C in one kernel (see ``include/gemm_rowsum.h``).

    a [M, K], b [K, N]: bf16 device tensors whose rows are dense (a row stride is allowed).  Returns
    (C, rowsum): C bf16 [M, N] (None with ``want_c=False``), rowsum fp32 [M].  Asynchronous on ``stream``.
    """
    if not (a.is_cuda and b.is_cuda):
        raise ValueError("a and b must be CUDA tensors: this library has no CPU path")
    if a.dtype != torch.bfloat16 or b.dtype != torch.bfloat16:
        raise TypeError("a and b must be bf16")
    if a.dim() != 2 or b.dim() != 2 or a.shape[1] != b.shape[0] or a.stride(1) != 1 or b.stride(1) != 1:
        raise ValueError("a must be [M, K] and b [K, N] with dense rows")
    M, K = a.shape
    N = b.shape[1]
    if c is None and want_c:
        c = torch.empty((M, N), device=a.device, dtype=torch.bfloat16)
    if c is not None and (c.dtype != torch.bfloat16 or c.shape != (M, N) or c.stride(1) != 1):
        raise TypeError("c must be a bf16 tensor [M, N] with dense rows")
    if rowsum is None:
        rowsum = torch.empty((M,), device=a.device, dtype=torch.float32)
    if rowsum.dtype != torch.float32 or not rowsum.is_contiguous() or rowsum.numel() != M:
        raise TypeError("rowsum must be a contiguous fp32 tensor [M]")
    desc = _gemm_desc(a, b, c, status_word)
    st = stream if stream is not None else torch.cuda.current_stream(a.device)
    rc = raw_gemm_rowsum(a.data_ptr(), b.data_ptr(), c.data_ptr() if c is not None else None, rowsum.data_ptr(),
                         M, N, K, desc, st.cuda_stream)
    if rc != ATTN_OK:
        raise AttnError(rc)
    return c, rowsum


def gemm_rowsum_host(a: torch.Tensor, b: torch.Tensor, c: Optional[torch.Tensor], rowsum: torch.Tensor,
                     workspace: torch.Tensor, *, status_word: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """``gemm_rowsum_host`` of the C ABI: a, b, c, rowsum are contiguous HOST tensors (pin them for asynchronous
    copies); ``workspace`` is a uint8 device tensor of at least :func:`gemm_rowsum_host_workspace_bytes` bytes."""
    for t in (a, b, rowsum) + ((c,) if c is not None else ()):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("gemm_rowsum_host takes contiguous host tensors")
    M, K = a.shape
    N = b.shape[1]
    desc = _gemm_desc(status_word=status_word)
    st = stream if stream is not None else torch.cuda.current_stream(workspace.device)
    rc = int(_lib.gemm_rowsum_host(a.data_ptr(), b.data_ptr(), c.data_ptr() if c is not None else None,
                                   rowsum.data_ptr(), M, N, K, ctypes.byref(desc), workspace.data_ptr(),
                                   workspace.numel() * workspace.element_size(), st.cuda_stream))
    if rc != ATTN_OK:
        raise AttnError(rc)
