"""Brute-force evaluation used to pin the oracle on tiny inputs.

Independent of the oracle's C code: K and V are first gathered into contiguous per-sequence
arrays with numpy fancy indexing, the whole [rows x keys] probability matrix is
materialised in extended precision, and everything else is read off that matrix.
"""
from __future__ import annotations

import numpy as np


def gather_contiguous(case, s: int):
    """K, V of sequence ``s`` as contiguous long-double arrays [L, Hkv, D]."""
    L = int(case.seq_lens[s])
    page = case.page_size
    t = np.arange(L)
    phys = case.block_table[s].numpy()[t // page]
    k = case.k_cache.float().numpy()[phys, t % page]
    v = case.v_cache.float().numpy()[phys, t % page]
    return k.astype(np.longdouble), v.astype(np.longdouble)


def brute(case):
    """Returns (out [T,Hq,D], probs list per sequence of [n,Hq,L]) in long double."""
    Hq, Hkv, D = case.num_q_heads, case.num_kv_heads, case.head_dim
    G = Hq // Hkv
    q = case.q.float().numpy().astype(np.longdouble)
    cu = case.cu_q_lens.tolist()
    out = np.zeros((case.total_q, Hq, D), dtype=np.longdouble)
    probs = []
    for s in range(case.num_seqs):
        n = cu[s + 1] - cu[s]
        L = int(case.seq_lens[s])
        k, v = gather_contiguous(case, s)
        P = np.zeros((n, Hq, L), dtype=np.longdouble)
        for i in range(n):
            pos = L - n + i
            for h in range(Hq):
                x = np.longdouble(case.scale) * (k[: pos + 1, h // G, :] @ q[cu[s] + i, h, :])
                e = np.exp(x - x.max())
                P[i, h, : pos + 1] = e / e.sum()
                out[cu[s] + i, h] = P[i, h, : pos + 1] @ v[: pos + 1, h // G, :]
                if case.alpha is not None and float(case.alpha[h]) != 0.0:
                    out[cu[s] + i, h] += np.longdouble(float(case.alpha[h])) * \
                        case.steer_vec[h].numpy().astype(np.longdouble)
        probs.append(P)
    return out, probs


def span_mass_from_probs(case, probs):
    """[T, P, S] span sums read off the materialised matrices."""
    heads = [h for h in range(case.num_q_heads) if case.head_mask is not None and case.head_mask[h]]
    S = case.num_spans
    cu = case.cu_q_lens.tolist()
    mass = np.zeros((case.total_q, len(heads), S), dtype=np.longdouble)
    for s in range(case.num_seqs):
        P = probs[s]
        L = P.shape[2]
        for j in range(S):
            a, b = (int(x) for x in case.spans[s, j])
            a, b = max(a, 0), min(b, L)
            if b > a:
                for pi, h in enumerate(heads):
                    mass[cu[s]:cu[s + 1], pi, j] = P[:, h, a:b].sum(-1)
    return mass
