"""Unmasked work of an attention problem: visible (query, key) pairs and the FLOPs they cost.

Bookkeeping for the benchmark and the tests (it counts pairs from the mask parameters of a workload; it holds
none of the attention arithmetic and loads no compiled library, so both the CUDA arm and the CPU-oracle arm of
the benchmark can use it).

Every mask this library builds (causal, window, same document, PrefixLM, the test-query
clause of the causal blockwise mask) leaves each query row one contiguous key interval
[lo(i), hi(i)], so the count is a sum of interval lengths.  4*D FLOPs per visible pair
(2*D for q.k, 2*D for p*v); masked pairs count nothing.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np


def row_intervals(Sq: int, Sk: int, causal: bool = False, window_left: Optional[int] = None,
                  window_right: Optional[int] = None, cu_seqlens: Optional[Sequence[int]] = None,
                  prefix_len: Optional[int] = None, test_query_start: Optional[int] = None,
                  global_len: Optional[int] = None):
    """Inclusive visible key interval (lo, hi) of every query row; lo > hi means no visible key.
    With global tokens a row may see the keys below ``global_len`` as a second piece: use
    :func:`row_visibility`, which returns that piece's length too."""
    pre, lo, hi = row_visibility(Sq, Sk, causal, window_left, window_right, cu_seqlens, prefix_len,
                                 test_query_start, global_len)
    if np.any(pre > 0):
        raise ValueError("two visible pieces per row: use row_visibility")
    return lo, hi


def row_visibility(Sq: int, Sk: int, causal: bool = False, window_left: Optional[int] = None,
                   window_right: Optional[int] = None, cu_seqlens: Optional[Sequence[int]] = None,
                   prefix_len: Optional[int] = None, test_query_start: Optional[int] = None,
                   global_len: Optional[int] = None):
    """(pre, lo, hi) per query row: keys j < pre and keys lo <= j <= hi are visible (pre <= lo - 1 when pre > 0)."""
    i = np.arange(Sq, dtype=np.int64)
    ip = i + (Sk - Sq)
    lo = np.zeros(Sq, dtype=np.int64)
    hi = np.full(Sq, Sk - 1, dtype=np.int64)
    if causal:      # PrefixLM: the first prefix_len keys stay visible to every row
        hi = np.minimum(hi, ip if prefix_len is None else np.maximum(ip, prefix_len - 1))
    if window_left is not None and window_left >= 0:
        lo = np.maximum(lo, ip - window_left)
    if window_right is not None and window_right >= 0:
        hi = np.minimum(hi, ip + window_right)
    if cu_seqlens is not None:
        cu = np.asarray(cu_seqlens, dtype=np.int64)
        d = np.searchsorted(cu, i, side="right") - 1
        isolated = np.ones(Sq, dtype=bool) if test_query_start is None else (i < test_query_start)
        lo = np.where(isolated, np.maximum(lo, cu[d]), lo)
        hi = np.where(isolated, np.minimum(hi, cu[d + 1] - 1), hi)
    pre = np.zeros(Sq, dtype=np.int64)
    if global_len is not None:
        g = min(int(global_len), Sk)
        hi_causal = np.full(Sq, Sk - 1, dtype=np.int64)
        if causal:
            hi_causal = np.minimum(hi_causal, ip if prefix_len is None else np.maximum(ip, prefix_len - 1))
        is_global_row = ip < g
        empty = lo > hi
        touch = (~empty) & (lo <= g)
        lo = np.where(is_global_row | empty | touch, 0, lo)
        hi = np.where(is_global_row, hi_causal, np.where(empty, g - 1, np.where(touch, np.maximum(hi, g - 1), hi)))
        pre = np.where(is_global_row | empty | touch, 0, g)
    return pre, lo, hi


def visible_pairs(Sq: int, Sk: int, **mask) -> int:
    """Number of visible (i, j) pairs of one (batch, head)."""
    pre, lo, hi = row_visibility(Sq, Sk, **mask)
    return int((np.maximum(hi - lo + 1, 0) + pre).sum())


def unmasked_flops(w) -> int:
    """4*D per visible pair over all batches and query heads of a ``synth_inputs.Workload``."""
    pairs = visible_pairs(w.Sq, w.Sk, causal=w.causal, window_left=w.window_left,
                          window_right=w.window_right, cu_seqlens=w.cu_seqlens, prefix_len=w.prefix_len,
                          test_query_start=w.test_query_start, global_len=w.global_len)
    return 4 * w.D * w.B * w.Hq * pairs


def algorithmic_bytes(w) -> int:
    """Bytes that must cross HBM once: Q, K, V in, O and LSE out."""
    e_in = 2 if w.dtype == "bf16" else 4
    e_out = 2 if w.o_dtype == "bf16" else 4
    q = w.B * w.Hq * w.Sq * w.D
    kv = 2 * w.B * w.Hkv * w.Sk * w.D
    lse = 4 * w.B * w.Hq * w.Sq if w.normalizer == "softmax" else 0
    return (q + kv) * e_in + q * e_out + lse
