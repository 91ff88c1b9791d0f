"""TEST INFRASTRUCTURE -- ctypes wrapper around the fp64 CPU oracle (hook_attn_oracle.c).

The oracle evaluates, row by row and in fp64, the hooked attention forward written out
from its definition (scores, two-pass softmax, value sum, steering add, span sums).  It
shares no code with the CUDA library.  Inputs are handed over as raw bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

from .build import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build())
        lib.hook_attn_oracle.restype = ctypes.c_int
        lib.hook_attn_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().hook_attn_oracle_threads())


def _bits(t: torch.Tensor) -> np.ndarray:
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def run(case, rows: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Evaluate ``case`` (any object with the input-generator's attribute names).

    Returns ``(out, mass)``: ``out`` fp64 ``[R, Hq, D]`` and ``mass`` fp64 ``[R, P, S]``
    (``None`` if nothing is probed) for the ``R`` requested global query rows (all rows when
    ``rows`` is ``None``).  ``mass`` is given for every evaluated row.
    """
    lib = _load()
    q = _bits(case.q)
    k = _bits(case.k_cache)
    v = _bits(case.v_cache)
    assert case.k_cache.is_contiguous() and case.v_cache.is_contiguous()
    nb, page, hkv, d = case.k_cache.shape
    bstride, tstride, hstride = page * hkv * d, hkv * d, d
    bt = np.ascontiguousarray(case.block_table.numpy(), dtype=np.int32)
    sl = np.ascontiguousarray(case.seq_lens.numpy(), dtype=np.int32)
    cu = np.ascontiguousarray(case.cu_q_lens.numpy(), dtype=np.int32)
    total_q = int(case.q.shape[0])
    hq = int(case.num_q_heads)
    spans = None if case.spans is None else np.ascontiguousarray(case.spans.numpy(), dtype=np.int32)
    hm = None if case.head_mask is None else np.ascontiguousarray(case.head_mask.numpy(), dtype=np.uint8)
    al = None if case.alpha is None else np.ascontiguousarray(case.alpha.numpy(), dtype=np.float32)
    sv = None if case.steer_vec is None else np.ascontiguousarray(case.steer_vec.numpy(), dtype=np.float32)
    num_spans = 0 if spans is None else int(spans.shape[1])
    rows_a = None if rows is None else np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
    nrows = total_q if rows_a is None else int(rows_a.shape[0])
    nprobed = 0 if hm is None else int((hm != 0).sum())
    out = np.zeros((nrows, hq, d), dtype=np.float64)
    mass = np.zeros((nrows, nprobed, num_spans), dtype=np.float64) if nprobed and num_spans else None
    rc = lib.hook_attn_oracle(
        ctypes.c_int(case.num_seqs), ctypes.c_int(total_q), ctypes.c_int(hq), ctypes.c_int(hkv),
        ctypes.c_int(d), ctypes.c_int(page), ctypes.c_int(bt.shape[1]), ctypes.c_int(num_spans),
        ctypes.c_double(case.scale), _ptr(q), _ptr(k), _ptr(v),
        ctypes.c_int64(bstride), ctypes.c_int64(tstride), ctypes.c_int64(hstride),
        _ptr(bt), _ptr(sl), _ptr(cu), _ptr(spans), _ptr(sv), _ptr(hm), _ptr(al),
        _ptr(rows_a), ctypes.c_int(nrows), _ptr(out), _ptr(mass))
    if rc != 0:
        raise ValueError(f"hook_attn_oracle rejected its arguments (code {rc})")
    return out, mass


def last_rows(case) -> list:
    """Global index of the last query row of every sequence that has rows."""
    cu = case.cu_q_lens.tolist()
    return [cu[s + 1] - 1 for s in range(case.num_seqs) if cu[s + 1] > cu[s]]
