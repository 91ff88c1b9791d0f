"""Seeded synthetic inputs for the hooked paged-attention path.

This module only *draws* tensors and lays them out in a paged KV cache.  It holds
none of the attention / softmax / span / steer arithmetic, so that the CUDA path and
the CPU oracle can both consume exactly the same bits without sharing any of the
method's code.

Conventions (shared by every consumer):

* ``q``           bf16 ``[total_q, Hq, D]`` -- query rows of all sequences, concatenated.
* ``k_cache``     bf16 ``[num_blocks, page, Hkv, D]`` -- physical pages; ``v_cache`` alike.
* ``block_table`` int32 ``[num_seqs, max_blocks]`` -- logical page -> physical page; entries
  past ``ceil(seq_len / page)`` are ``-1`` and must never be dereferenced.
* ``seq_lens``    int32 ``[num_seqs]`` -- keys visible to the last query row of the
  sequence, *including* the rows of this call (their K/V already sit in the cache).
* ``cu_q_lens``   int32 ``[num_seqs + 1]`` -- prefix sums of the query rows per sequence.
* ``spans``       int32 ``[num_seqs, S, 2]`` -- half-open absolute key ranges ``[a, b)``.
* ``head_mask``   uint8 ``[Hq]`` -- nonzero = probed query head (the config's
  ``important_heads`` of one layer).
* ``alpha``       fp32 ``[Hq]``, ``steer_vec`` fp32 ``[Hq, D]`` -- per-head steering.

All values are drawn in fp32 from a ``torch.Generator`` on the CPU and rounded to bf16
once; those bf16 bits are what every consumer reads.  With ``device="cuda"`` the large
tensors (queries, K/V pages, page permutation) are drawn by a seeded generator of that
device instead -- the same recipe and distributions, other values -- which turns seconds
of host-side drawing into milliseconds for the benchmark's largest workloads;
:func:`to_host` gives the CPU copy of such a case for the oracle.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence

import torch

BASE_SEED = 26030658
PAGE = 16

PROBE_ROWS_ALL = 0
PROBE_ROWS_LAST = 1


@dataclass
class HookAttnCase:
    name: str
    is_decode: bool
    num_seqs: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_blocks: int
    max_blocks_per_seq: int
    num_spans: int
    probe_rows: int
    scale: float
    q: torch.Tensor
    k_cache: torch.Tensor
    v_cache: torch.Tensor
    block_table: torch.Tensor
    seq_lens: torch.Tensor
    cu_q_lens: torch.Tensor
    spans: Optional[torch.Tensor] = None
    head_mask: Optional[torch.Tensor] = None
    alpha: Optional[torch.Tensor] = None
    steer_vec: Optional[torch.Tensor] = None
    meta: dict = field(default_factory=dict)

    @property
    def total_q(self) -> int:
        return int(self.q.shape[0])

    @property
    def num_probed(self) -> int:
        return 0 if self.head_mask is None else int((self.head_mask != 0).sum())

    def q_lens(self) -> List[int]:
        c = self.cu_q_lens.tolist()
        return [c[i + 1] - c[i] for i in range(self.num_seqs)]

    def without_hooks(self) -> "HookAttnCase":
        """Same tensors, hooks disabled (no probe, no steer)."""
        return replace(self, name=self.name + "/nohook", spans=None, head_mask=None,
                       alpha=None, steer_vec=None, num_spans=0)

    def kv_tokens(self) -> int:
        return int(self.seq_lens.sum())

    def visible_pairs(self) -> int:
        """Visible (row, key) pairs per query head, summed over the sequences."""
        tot = 0
        for L, n in zip(self.seq_lens.tolist(), self.q_lens()):
            # rows at positions L-n .. L-1 see pos+1 keys each
            tot += n * (L - n) + n * (n + 1) // 2
        return tot


# ----------------------------------------------------------------------------------------
# building blocks
# ----------------------------------------------------------------------------------------

def _gen(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn_bf16(shape: Sequence[int], g: torch.Generator, std: float = 1.0,
                chunk: int = 1 << 26) -> torch.Tensor:
    """N(0, std^2) drawn in fp32 and rounded to bf16 once (chunked to bound memory)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=torch.bfloat16, device=g.device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        x = torch.randn(hi - lo, generator=g, dtype=torch.float32, device=g.device)
        if std != 1.0:
            x.mul_(std)
        out[lo:hi] = x.to(torch.bfloat16)
    return out.view(*shape)


def paged_cache(seq_lens: Sequence[int], num_kv_heads: int, head_dim: int, g: torch.Generator,
                k_std: float = 1.0, v_std: float = 1.0, pool: float = 1.25,
                poison: bool = False, shuffle: bool = True, max_blocks: Optional[int] = None):
    """Draw K/V for every sequence and scatter them into shuffled physical pages.

    Returns ``(k_cache, v_cache, block_table, num_blocks, max_blocks)``.  Unused pages
    and the tails of last pages are NaN when ``poison`` is set (they must never
    influence a result), zero otherwise.
    """
    pages = [(L + PAGE - 1) // PAGE for L in seq_lens]
    need = sum(pages)
    num_blocks = max(1, int(math.ceil(need * pool)))
    mb = max(pages) if pages else 1
    mb = max(mb, 1)
    if max_blocks is not None:
        assert max_blocks >= mb
        mb = max_blocks
    dev = g.device
    perm = torch.randperm(num_blocks, generator=g, device=dev) if shuffle else torch.arange(num_blocks, device=dev)
    block_table = torch.full((len(seq_lens), mb), -1, dtype=torch.int32, device=dev)
    fill = float("nan") if poison else 0.0
    k_cache = torch.full((num_blocks, PAGE, num_kv_heads, head_dim), fill, dtype=torch.bfloat16, device=dev)
    v_cache = torch.full((num_blocks, PAGE, num_kv_heads, head_dim), fill, dtype=torch.bfloat16, device=dev)
    cursor = 0
    for s, L in enumerate(seq_lens):
        np_s = pages[s]
        phys = perm[cursor:cursor + np_s]
        cursor += np_s
        block_table[s, :np_s] = phys.to(torch.int32)
        if L == 0:
            continue
        k = _randn_bf16((L, num_kv_heads, head_dim), g, k_std)
        v = _randn_bf16((L, num_kv_heads, head_dim), g, v_std)
        pad = np_s * PAGE - L
        if pad:
            tail = torch.full((pad, num_kv_heads, head_dim), fill, dtype=torch.bfloat16, device=dev)
            k = torch.cat([k, tail], 0)
            v = torch.cat([v, tail], 0)
        k_cache[phys] = k.view(np_s, PAGE, num_kv_heads, head_dim)
        v_cache[phys] = v.view(np_s, PAGE, num_kv_heads, head_dim)
    return k_cache, v_cache, block_table, num_blocks, mb


def partition_spans(seq_lens: Sequence[int], num_spans: int, g: torch.Generator) -> torch.Tensor:
    """``num_spans`` half-open spans per sequence that partition ``[0, L)``: sorted distinct
    seeded cut points in ``(0, L)``."""
    out = torch.zeros((len(seq_lens), num_spans, 2), dtype=torch.int32)
    for s, L in enumerate(seq_lens):
        if L <= 0:
            continue
        ncut = min(num_spans - 1, max(L - 1, 0))
        cuts = (torch.randperm(L - 1, generator=g)[:ncut] + 1).sort().values.tolist() if ncut else []
        edges = [0] + cuts + [L] * (num_spans - len(cuts))
        for j in range(num_spans):
            out[s, j, 0] = edges[j]
            out[s, j, 1] = edges[j + 1]
    return out


def choose_heads(num_heads: int, count: int, g: torch.Generator) -> torch.Tensor:
    mask = torch.zeros(num_heads, dtype=torch.uint8)
    if count > 0:
        mask[torch.randperm(num_heads, generator=g)[:count]] = 1
    return mask


def _cu(q_lens: Sequence[int]) -> torch.Tensor:
    c = [0]
    for n in q_lens:
        c.append(c[-1] + int(n))
    return torch.tensor(c, dtype=torch.int32)


def make_case(name: str, *, is_decode: bool, seq_lens: Sequence[int], q_lens: Sequence[int],
              num_q_heads: int, num_kv_heads: int, head_dim: int, seed: int,
              num_spans: int = 0, spans: Optional[torch.Tensor] = None,
              head_mask: Optional[torch.Tensor] = None, alpha: Optional[torch.Tensor] = None,
              steer: bool = False, probe_rows: int = PROBE_ROWS_ALL,
              q_std: float = 1.0, k_std: float = 1.0, v_std: float = 1.0,
              poison: bool = False, shuffle: bool = True, pool: float = 1.25,
              max_blocks: Optional[int] = None, scale: Optional[float] = None,
              device: str = "cpu") -> HookAttnCase:
    """Generic seeded case builder used by the named configurations and by the tests.  ``device``
    other than ``"cpu"`` draws q, K/V and the page permutation with that device's generator (the small
    host-side arrays stay on the CPU and come from a CPU generator of the same seed)."""
    g = _gen(seed, device)
    g_host = g if str(device) == "cpu" else _gen(seed)
    seq_lens = [int(x) for x in seq_lens]
    q_lens = [int(x) for x in q_lens]
    assert len(seq_lens) == len(q_lens)
    k_cache, v_cache, bt, nb, mb = paged_cache(seq_lens, num_kv_heads, head_dim, g, k_std, v_std,
                                              pool=pool, poison=poison, shuffle=shuffle,
                                              max_blocks=max_blocks)
    tq = sum(q_lens)
    q = _randn_bf16((tq, num_q_heads, head_dim), g, q_std)
    if spans is None and num_spans > 0:
        spans = partition_spans(seq_lens, num_spans, g_host)
    steer_vec = None
    if steer:
        steer_vec = torch.randn((num_q_heads, head_dim), generator=g_host, dtype=torch.float32)
    if spans is not None:
        num_spans = int(spans.shape[1])
    return HookAttnCase(
        name=name, is_decode=is_decode, num_seqs=len(seq_lens), num_q_heads=num_q_heads,
        num_kv_heads=num_kv_heads, head_dim=head_dim, page_size=PAGE, num_blocks=nb,
        max_blocks_per_seq=mb, num_spans=num_spans, probe_rows=probe_rows,
        scale=float(scale) if scale is not None else 1.0 / math.sqrt(head_dim),
        q=q, k_cache=k_cache, v_cache=v_cache, block_table=bt,
        seq_lens=torch.tensor(seq_lens, dtype=torch.int32), cu_q_lens=_cu(q_lens),
        spans=spans, head_mask=head_mask, alpha=alpha, steer_vec=steer_vec,
        meta={"seed": int(seed)})


# ----------------------------------------------------------------------------------------
# the five named workloads (shapes of the paper's demonstrations: two spans + last-token
# probe for instruction/data monitoring, several passage spans + a head subset for
# attention-based reranking, per-head steering vectors for activation steering)
# ----------------------------------------------------------------------------------------

def config1_tiny_prefill(poison: bool = False) -> HookAttnCase:
    seed = BASE_SEED + 1
    Hq = 8
    spans = torch.tensor([[[0, 64], [64, 256]]], dtype=torch.int32)
    alpha = torch.zeros(Hq, dtype=torch.float32)
    alpha[0:2] = 0.5
    return make_case("cfg1_tiny_prefill", is_decode=False, seq_lens=[256], q_lens=[256],
                     num_q_heads=Hq, num_kv_heads=8, head_dim=64, seed=seed, spans=spans,
                     head_mask=torch.ones(Hq, dtype=torch.uint8), alpha=alpha, steer=True,
                     probe_rows=PROBE_ROWS_ALL, poison=poison)


def config2_decode(num_seqs: int = 64, lo: int = 512, hi: int = 4096, poison: bool = False,
                   seed_offset: int = 0, device: str = "cpu") -> HookAttnCase:
    seed = BASE_SEED + 2 + seed_offset
    g = _gen(seed ^ 0x5EED)
    Hq, Hkv, D = 32, 8, 128
    L = torch.randint(lo, hi + 1, (num_seqs,), generator=g).tolist()
    spans = torch.zeros((num_seqs, 2, 2), dtype=torch.int32)
    for s, Ls in enumerate(L):
        c = int(torch.randint(1, max(Ls // 2, 1) + 1, (1,), generator=g))
        spans[s, 0, 0], spans[s, 0, 1] = 0, c
        spans[s, 1, 0], spans[s, 1, 1] = c, Ls
    head_mask = choose_heads(Hq, 16, g)
    alpha = torch.zeros(Hq, dtype=torch.float32)
    alpha[torch.randperm(Hq, generator=g)[:4]] = 1.0
    return make_case("cfg2_decode", is_decode=True, seq_lens=L, q_lens=[1] * num_seqs,
                     num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, seed=seed, spans=spans,
                     head_mask=head_mask, alpha=alpha, steer=True,
                     probe_rows=PROBE_ROWS_LAST, poison=poison, device=device)


def config3_layer_masks(num_layers: int = 32, num_heads: int = 32, frac: float = 0.10) -> torch.Tensor:
    """Seeded 10 % of the (layer, head) pairs -> uint8 ``[layers, heads]``."""
    g = _gen(BASE_SEED + 3)
    n = num_layers * num_heads
    k = int(round(frac * n))
    m = torch.zeros(n, dtype=torch.uint8)
    m[torch.randperm(n, generator=g)[:k]] = 1
    return m.view(num_layers, num_heads)


def config3_prefill(layer: int = 0, num_seqs: int = 8, tokens: int = 4096,
                    poison: bool = False, force_probe: bool = False, device: str = "cpu") -> HookAttnCase:
    seed = BASE_SEED + 3 + 1000 * layer
    Hq, Hkv, D = 32, 8, 128
    mask = config3_layer_masks()[layer % 32].clone()
    if force_probe and int(mask.sum()) == 0:
        mask[(layer * 7) % Hq] = 1
    return make_case(f"cfg3_prefill_l{layer}", is_decode=False, seq_lens=[tokens] * num_seqs,
                     q_lens=[tokens] * num_seqs, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                     seed=seed, num_spans=3, head_mask=mask, alpha=None, steer=False,
                     probe_rows=PROBE_ROWS_ALL, k_std=128.0 ** -0.5, poison=poison, device=device)


def _config4_common(g: torch.Generator):
    Hq = 28
    head_mask = choose_heads(Hq, 14, g)
    alpha = torch.zeros(Hq, dtype=torch.float32)
    idx = torch.randperm(Hq, generator=g)[:8]
    alpha[idx] = (torch.rand(8, generator=g) * 4.0 - 2.0)
    return head_mask, alpha


def config4_decode(num_seqs: int = 256, lo: int = 1024, hi: int = 8192,
                   poison: bool = False, device: str = "cpu") -> HookAttnCase:
    seed = BASE_SEED + 4
    g = _gen(seed ^ 0x5EED)
    head_mask, alpha = _config4_common(g)
    L = torch.randint(lo, hi + 1, (num_seqs,), generator=g).tolist()
    return make_case("cfg4_mixed_decode", is_decode=True, seq_lens=L, q_lens=[1] * num_seqs,
                     num_q_heads=28, num_kv_heads=4, head_dim=128, seed=seed, num_spans=4,
                     head_mask=head_mask, alpha=alpha, steer=True,
                     probe_rows=PROBE_ROWS_LAST, poison=poison, device=device)


def config4_prefill(chunks: int = 2, n: int = 2048, ctx: int = 4096,
                    poison: bool = False, device: str = "cpu") -> HookAttnCase:
    seed = BASE_SEED + 4 + 500
    g = _gen((BASE_SEED + 4) ^ 0x5EED)
    head_mask, alpha = _config4_common(g)
    return make_case("cfg4_mixed_prefill", is_decode=False, seq_lens=[ctx + n] * chunks,
                     q_lens=[n] * chunks, num_q_heads=28, num_kv_heads=4, head_dim=128,
                     seed=seed, num_spans=4, head_mask=head_mask, alpha=alpha, steer=True,
                     probe_rows=PROBE_ROWS_ALL, poison=poison, device=device)


def _config5_common(probed: int):
    g = _gen((BASE_SEED + 5) ^ 0x5EED)
    Hq = 64
    head_mask = torch.ones(Hq, dtype=torch.uint8) if probed >= Hq else choose_heads(Hq, probed, g)
    alpha = torch.zeros(Hq, dtype=torch.float32)
    alpha[torch.randperm(Hq, generator=g)[:8]] = 0.8
    return head_mask, alpha


def config5_prefill(num_seqs: int = 4, tokens: int = 32768, probed: int = 64,
                    poison: bool = False, device: str = "cpu") -> HookAttnCase:
    head_mask, alpha = _config5_common(probed)
    return make_case("cfg5_long_prefill", is_decode=False, seq_lens=[tokens] * num_seqs,
                     q_lens=[tokens] * num_seqs, num_q_heads=64, num_kv_heads=8, head_dim=128,
                     seed=BASE_SEED + 5, num_spans=8, head_mask=head_mask, alpha=alpha,
                     steer=True, probe_rows=PROBE_ROWS_ALL, poison=poison, device=device)


def config5_decode(num_seqs: int = 4, tokens: int = 32768, steps: int = 128, step: int = 0,
                   probed: int = 64, poison: bool = False, device: str = "cpu") -> HookAttnCase:
    """Decode step ``step`` of the long-context workload.  The cache is pre-filled to
    ``tokens + steps`` keys so that no append is part of a step; step ``t`` sees
    ``tokens + t + 1`` keys (its own row included)."""
    head_mask, alpha = _config5_common(probed)
    cap = tokens + steps
    case = make_case("cfg5_long_decode", is_decode=True, seq_lens=[cap] * num_seqs,
                     q_lens=[1] * num_seqs, num_q_heads=64, num_kv_heads=8, head_dim=128,
                     seed=BASE_SEED + 5 + 500, num_spans=8, head_mask=head_mask, alpha=alpha,
                     steer=True, probe_rows=PROBE_ROWS_LAST, poison=poison, device=device)
    return with_seq_lens(case, [tokens + step + 1] * num_seqs)


def config5_session(num_seqs: int = 4, tokens: int = 32768, steps: int = 128, probed: int = 64,
                    device: str = "cpu"):
    """The long-context workload as one session on one cache: a full causal prefill of ``tokens`` keys per
    sequence followed by ``steps`` decode steps.  The cache is pre-filled to ``tokens + steps`` keys so that
    no append is part of a step.  Returns ``(prefill_case, [decode case of step 0 .. steps-1])``; all cases
    share the K/V pages, the block table, the head mask and the steering."""
    dec0 = config5_decode(num_seqs=num_seqs, tokens=tokens, steps=steps, step=0, probed=probed, device=device)
    g_dev = _gen(BASE_SEED + 5, device)
    g_host = _gen(BASE_SEED + 5 + 7)
    q_pf = _randn_bf16((num_seqs * tokens, dec0.num_q_heads, dec0.head_dim), g_dev)
    prefill = replace(dec0, name="cfg5_long_prefill", is_decode=False, q=q_pf,
                      seq_lens=torch.tensor([tokens] * num_seqs, dtype=torch.int32),
                      cu_q_lens=_cu([tokens] * num_seqs),
                      spans=partition_spans([tokens] * num_seqs, dec0.num_spans, g_host),
                      probe_rows=PROBE_ROWS_ALL)
    decodes = [with_seq_lens(dec0, [tokens + t + 1] * num_seqs) for t in range(steps)]
    return prefill, decodes


def to_host(case: HookAttnCase) -> HookAttnCase:
    """The same case with every tensor on the CPU (for consumers that read host memory)."""
    moved = {f: getattr(case, f).cpu() for f in ("q", "k_cache", "v_cache", "block_table")}
    return replace(case, **moved)


def with_seq_lens(case: HookAttnCase, seq_lens: Sequence[int]) -> HookAttnCase:
    """Same cache and tables, shorter visible lengths (spans are clipped by consumers)."""
    return replace(case, seq_lens=torch.tensor([int(x) for x in seq_lens], dtype=torch.int32))


def sample_rows(case: HookAttnCase, extra_random: int = 32, seed: int = 7) -> List[int]:
    """Deterministic sample of global query-row indices for spot checks at sizes where the
    full CPU evaluation is too slow: per sequence rows 0, 1, 15, 16, 17, 127, 128, 129, the
    rows at every span boundary +-1, the last row, plus seeded random rows."""
    g = _gen(seed)
    rows: List[int] = []
    cu = case.cu_q_lens.tolist()
    Ls = case.seq_lens.tolist()
    for s in range(case.num_seqs):
        n = cu[s + 1] - cu[s]
        if n == 0:
            continue
        first_pos = Ls[s] - n
        local = {0, 1, 15, 16, 17, 127, 128, 129, n - 1, n - 2, n // 2}
        if case.spans is not None:
            for a, b in case.spans[s].tolist():
                for e in (a, b):
                    for d in (-1, 0, 1):
                        local.add(e + d - first_pos)
        if extra_random > 0:
            local.update(torch.randint(0, n, (extra_random,), generator=g).tolist())
        rows.extend(cu[s] + i for i in sorted(local) if 0 <= i < n)
    return rows
