"""TEST INFRASTRUCTURE -- plain numpy oracles of the operations that sit next to the hooked attention:
the analyzer's score reduction, residual-stream steering and the raw q/k capture.  fp64 where
floating point is involved, plain indexing where bytes are moved.  Shares nothing with the CUDA code.

`scores`: parity unpinned against the paper -- its analyzer body is elided, so the formula below is a
reading of the paper's words; the arithmetic of that reading is pinned by closed forms and brute force.
Readings where the paper is silent: `mean` averages the span masses
over the probed heads; `sum_normalize` first divides every head's span masses by that head's total
over the configured spans (instruction mass / (instruction + data mass) for two spans) and then
averages over the heads; a head whose total is zero contributes zero.
"""
from __future__ import annotations

import numpy as np
import torch

SCORE_MEAN = 0
SCORE_SUM_NORMALIZE = 1


def scores(span_mass: np.ndarray, mode: int) -> np.ndarray:
    """span_mass [R, P, S] -> scores [R, S] (Section 2.2, attn2score; Section 3 focus / relevance scores)."""
    m = np.asarray(span_mass, dtype=np.float64)
    if mode == SCORE_MEAN:
        return m.mean(axis=1)
    out = np.zeros((m.shape[0], m.shape[2]))
    for r in range(m.shape[0]):
        for p in range(m.shape[1]):
            tot = m[r, p].sum()
            if tot > 0:
                out[r] += m[r, p] / tot
    return out / m.shape[1]


def steer_residual(hidden_bf16_as_f32: np.ndarray, vec: np.ndarray, alpha: float) -> np.ndarray:
    """hidden [T, H] (bf16 values widened exactly) + alpha * vec [H], in fp64 (Section 1, activation steering:
    a steering vector added to a layer's activations)."""
    return np.asarray(hidden_bf16_as_f32, dtype=np.float64) + float(alpha) * np.asarray(vec, dtype=np.float64)[None, :]


def capture_qk(case):
    """The worker hook's payload (Section 2.1): q of the probed heads for the probed rows and the
    all-token k of those heads, gathered through the block table.  Returns int16 bit patterns:
    q_out [rows, P, D], k_out [sum L, P, D], cu_k [num_seqs + 1]."""
    hq, hkv, d = case.num_q_heads, case.num_kv_heads, case.head_dim
    g = hq // hkv
    heads = [h for h in range(hq) if case.head_mask is not None and int(case.head_mask[h])]
    qb = case.q.contiguous().view(torch.int16).numpy()
    kb = case.k_cache.contiguous().view(torch.int16).numpy()
    cu_q = case.cu_q_lens.tolist()
    lens = case.seq_lens.tolist()
    last_only = case.is_decode or case.probe_rows == 1
    rows = []
    for s in range(case.num_seqs):
        n = cu_q[s + 1] - cu_q[s]
        rows.append([cu_q[s + 1] - 1] if (last_only and n > 0) else ([] if last_only else list(range(cu_q[s], cu_q[s + 1]))))
    if last_only:
        q_out = np.zeros((case.num_seqs, len(heads), d), dtype=np.int16)
        for s, r in enumerate(rows):
            if r:
                q_out[s] = qb[r[0]][heads]
    else:
        flat = [r for rr in rows for r in rr]
        q_out = qb[flat][:, heads] if flat else np.zeros((0, len(heads), d), dtype=np.int16)
    cu_k = np.zeros(case.num_seqs + 1, dtype=np.int32)
    cu_k[1:] = np.cumsum(lens)
    k_out = np.zeros((int(cu_k[-1]), len(heads), d), dtype=np.int16)
    bt = case.block_table.numpy()
    page = case.page_size
    for s, L in enumerate(lens):
        for t in range(L):
            blk = bt[s, t // page]
            for pi, h in enumerate(heads):
                k_out[cu_k[s] + t, pi] = kb[blk, t % page, h // g]
    return q_out, k_out, cu_k
