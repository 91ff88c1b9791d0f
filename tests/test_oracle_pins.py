"""Pins for the CPU oracle: what the mathematics fixes, independent of the oracle's code.

The paper prints no worked numeric example for this path, so the oracle is pinned by
(1) a brute-force evaluation with a materialised probability matrix on tiny contiguous
inputs, (2) closed forms, (3) invariants of softmax attention and of span sums, and
(4) the library special case (hooks off == causal scaled-dot-product attention, fp64).
Each pin is chosen so that a plausible mistake (dropped scale, wrong GQA map, off-by-one
in the causal limit or a span edge, transposed operand, wrong page arithmetic, steering
applied before the normalisation) fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2603_06588_b200 import inputs
from tests import _brute


def tiny(seed=11, seq_lens=(37, 48, 5), q_lens=(37, 9, 1), Hq=4, Hkv=2, D=8, S=3, **kw):
    g = inputs._gen(seed + 99)
    head_mask = inputs.choose_heads(Hq, max(1, Hq // 2), g)
    alpha = torch.zeros(Hq)
    alpha[0] = 0.75
    alpha[Hq - 1] = -1.5
    return inputs.make_case("tiny", is_decode=False, seq_lens=seq_lens, q_lens=q_lens,
                            num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, seed=seed, num_spans=S,
                            head_mask=head_mask, alpha=alpha, steer=True, poison=True, **kw)


# ---------------------------------------------------------------------------- brute force
@pytest.mark.parametrize("shape", [
    dict(seq_lens=(37, 48, 5), q_lens=(37, 9, 1), Hq=4, Hkv=2, D=8),
    dict(seq_lens=(16, 33), q_lens=(16, 33), Hq=6, Hkv=2, D=64),
    dict(seq_lens=(1, 17, 32), q_lens=(1, 1, 1), Hq=8, Hkv=1, D=8),
    dict(seq_lens=(40,), q_lens=(0,), Hq=2, Hkv=2, D=8),
])
def test_brute_force_materialised_matrix(shape):
    case = tiny(**shape)
    out, mass = oracle.run(case)
    b_out, probs = _brute.brute(case)
    b_mass = _brute.span_mass_from_probs(case, probs)
    assert out.shape == b_out.shape
    if out.size:
        assert np.abs(out - b_out.astype(np.float64)).max() < 1e-12
        assert np.abs(mass - b_mass.astype(np.float64)).max() < 1e-12


def test_brute_force_overlapping_and_degenerate_spans():
    spans = torch.tensor([[[0, 100], [5, 5], [9, 3], [-4, 7], [30, 31]]], dtype=torch.int32)
    case = inputs.make_case("t", is_decode=False, seq_lens=[31], q_lens=[31], num_q_heads=2,
                            num_kv_heads=1, head_dim=8, seed=3, spans=spans,
                            head_mask=torch.tensor([1, 1], dtype=torch.uint8))
    out, mass = oracle.run(case)
    _, probs = _brute.brute(case)
    b_mass = _brute.span_mass_from_probs(case, probs).astype(np.float64)
    assert np.abs(mass - b_mass).max() < 1e-12
    assert np.allclose(mass[:, :, 0], 1.0, atol=1e-12)       # covers everything
    assert np.all(mass[:, :, 1] == 0) and np.all(mass[:, :, 2] == 0)   # empty / reversed
    assert np.all(mass[:30, :, 4] == 0) and np.all(mass[30, :, 4] > 0)  # key 30 only visible to row 30


# ---------------------------------------------------------------------------- closed forms
def test_identical_keys_give_uniform_attention():
    case = tiny(seq_lens=(29,), q_lens=(29,), Hq=4, Hkv=2, D=8, S=3)
    case.k_cache[:] = case.k_cache[case.block_table[0, 0].item(), 0, 0, :]   # every key identical
    case.alpha = None
    out, mass = oracle.run(case)
    k, v = _brute.gather_contiguous(case, 0)
    heads = [h for h in range(4) if case.head_mask[h]]
    for i in range(29):
        for h in range(4):
            assert np.allclose(out[i, h], np.asarray(v[: i + 1, h // 2].mean(0), dtype=np.float64),
                               atol=1e-13)
        for pi, h in enumerate(heads):
            for j in range(3):
                a, b = (int(x) for x in case.spans[0, j])
                cnt = max(0, min(b, i + 1) - max(a, 0))
                assert abs(mass[i, pi, j] - cnt / (i + 1)) < 1e-13


def test_zero_query_gives_uniform_attention():
    case = tiny(seq_lens=(20,), q_lens=(20,), Hq=2, Hkv=2, D=8, S=2)
    case.q.zero_()
    case.alpha = None
    out, _ = oracle.run(case)
    _, v = _brute.gather_contiguous(case, 0)
    assert np.allclose(out[19, 1], np.asarray(v[:20, 1].mean(0), dtype=np.float64), atol=1e-13)


def test_first_row_returns_first_value_plus_steer():
    case = tiny(seq_lens=(24,), q_lens=(24,), Hq=4, Hkv=2, D=8, S=3)
    out, mass = oracle.run(case)
    _, v = _brute.gather_contiguous(case, 0)
    for h in range(4):
        want = np.asarray(v[0, h // 2], dtype=np.float64) + \
            float(case.alpha[h]) * case.steer_vec[h].double().numpy()
        assert np.allclose(out[0, h], want, atol=1e-14)
    # mass is exactly 1 for the span containing key 0 and 0 elsewhere
    for j in range(3):
        a, b = (int(x) for x in case.spans[0, j])
        assert np.all(mass[0, :, j] == (1.0 if a <= 0 < b else 0.0))


def test_two_keys_sigmoid():
    case = tiny(seq_lens=(2,), q_lens=(1,), Hq=2, Hkv=1, D=8, S=2, scale=0.37)
    case.spans = torch.tensor([[[0, 1], [1, 2]]], dtype=torch.int32)
    case.head_mask = torch.tensor([1, 1], dtype=torch.uint8)
    _, mass = oracle.run(case)
    k, _ = _brute.gather_contiguous(case, 0)
    q = case.q.double().numpy()
    for h in range(2):
        x0 = 0.37 * float(np.dot(q[0, h], np.asarray(k[0, 0], dtype=np.float64)))
        x1 = 0.37 * float(np.dot(q[0, h], np.asarray(k[1, 0], dtype=np.float64)))
        sig = 1.0 / (1.0 + math.exp(-(x0 - x1)))
        assert abs(mass[0, h, 0] - sig) < 1e-14
        assert abs(mass[0, h, 1] - (1 - sig)) < 1e-14


def test_dominating_key_selects_its_value_row():
    case = tiny(seq_lens=(40,), q_lens=(1,), Hq=2, Hkv=2, D=8, S=2)
    case.alpha = None
    case.spans = torch.tensor([[[0, 23], [23, 40]]], dtype=torch.int32)
    case.head_mask = torch.tensor([1, 1], dtype=torch.uint8)
    case.k_cache.zero_()
    case.q[:] = 16.0
    t = 23
    case.k_cache[case.block_table[0, t // 16].item(), t % 16] = 16.0   # logit gap = 16*16*8*scale
    out, mass = oracle.run(case)
    _, v = _brute.gather_contiguous(case, 0)
    assert np.allclose(out[0, 1], np.asarray(v[t, 1], dtype=np.float64), atol=1e-13)
    assert np.allclose(mass[0, :, 1], 1.0) and np.all(mass[0, :, 0] < 1e-100)


# ------------------------------------------------------------------------------ invariants
def test_partition_sums_to_one_and_additivity():
    case = tiny(seq_lens=(45, 19), q_lens=(45, 7), Hq=4, Hkv=2, D=8, S=4)
    _, mass = oracle.run(case)
    assert np.abs(mass.sum(-1) - 1.0).max() < 1e-13
    # additivity: [a,c) = [a,b) + [b,c)
    sp = case.spans.clone()
    merged = torch.stack([torch.stack([sp[:, 0, 0], sp[:, 1, 1]], -1), sp[:, 2], sp[:, 3]], 1)
    case2 = inputs.replace(case, spans=merged, num_spans=3)
    _, mass2 = oracle.run(case2)
    assert np.abs(mass2[:, :, 0] - (mass[:, :, 0] + mass[:, :, 1])).max() < 1e-13


def test_alpha_zero_is_identity_and_steer_is_additive():
    case = tiny()
    out, mass = oracle.run(case)
    off = inputs.replace(case, alpha=torch.zeros(case.num_q_heads), name="off")
    out0, mass0 = oracle.run(off)
    none = inputs.replace(case, alpha=None, steer_vec=None)
    out_n, _ = oracle.run(none)
    assert np.array_equal(out0, out_n)
    assert np.array_equal(mass, mass0)            # probing is unaffected by steering
    want = case.alpha.double().numpy()[None, :, None] * case.steer_vec.double().numpy()[None]
    assert np.abs((out - out0) - want).max() < 1e-14


def test_probe_does_not_change_output():
    case = tiny()
    out, _ = oracle.run(case)
    out2, m2 = oracle.run(inputs.replace(case, head_mask=None, spans=None, num_spans=0))
    assert m2 is None and np.array_equal(out, out2)


def test_gqa_equals_head_replicated_mha():
    case = tiny(seq_lens=(33, 20), q_lens=(33, 4), Hq=6, Hkv=2, D=8)
    out, mass = oracle.run(case)
    rep = inputs.replace(case, num_kv_heads=6,
                         k_cache=case.k_cache.repeat_interleave(3, dim=2).contiguous(),
                         v_cache=case.v_cache.repeat_interleave(3, dim=2).contiguous())
    out_r, mass_r = oracle.run(rep)
    assert np.array_equal(out, out_r) and np.array_equal(mass, mass_r)


def test_decode_equals_last_prefill_row_and_chunk_equals_rows():
    full = tiny(seq_lens=(41, 30), q_lens=(41, 30), Hq=4, Hkv=2, D=8)
    out_f, mass_f = oracle.run(full)
    cu = full.cu_q_lens.tolist()
    # chunked prefill: only the last 5 / 11 rows of each sequence are in the call
    tail = (5, 11)
    rows = [r for s in range(2) for r in range(cu[s + 1] - tail[s], cu[s + 1])]
    chunk = inputs.replace(full, q=full.q[rows].contiguous(),
                           cu_q_lens=torch.tensor([0, 5, 16], dtype=torch.int32))
    out_c, mass_c = oracle.run(chunk)
    assert np.array_equal(out_c, out_f[rows]) and np.array_equal(mass_c, mass_f[rows])
    # decode: one row per sequence == last row of the full prefill
    last = [cu[1] - 1, cu[2] - 1]
    dec = inputs.replace(full, q=full.q[last].contiguous(), is_decode=True,
                         cu_q_lens=torch.tensor([0, 1, 2], dtype=torch.int32))
    out_d, mass_d = oracle.run(dec)
    assert np.array_equal(out_d, out_f[last]) and np.array_equal(mass_d, mass_f[last])
    # row subset argument == slicing the full result
    out_s, mass_s = oracle.run(full, rows=rows)
    assert np.array_equal(out_s, out_f[rows]) and np.array_equal(mass_s, mass_f[rows])


def test_page_permutation_does_not_change_results():
    case = tiny(seq_lens=(50, 23), q_lens=(50, 23))
    out, mass = oracle.run(case)
    g = inputs._gen(5)
    perm = torch.randperm(case.num_blocks, generator=g)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(case.num_blocks)
    bt = case.block_table.clone()
    valid = bt >= 0
    bt[valid] = inv[bt[valid].long()].to(torch.int32)
    moved = inputs.replace(case, k_cache=case.k_cache[perm].contiguous(),
                           v_cache=case.v_cache[perm].contiguous(), block_table=bt)
    out_p, mass_p = oracle.run(moved)
    assert np.array_equal(out, out_p) and np.array_equal(mass, mass_p)


def test_poisoned_pages_never_reach_the_result():
    case = tiny()          # unused pages, page tails are NaN; unused table entries are -1
    out, mass = oracle.run(case)
    assert np.isfinite(out).all() and np.isfinite(mass).all()


def test_scale_is_applied_to_the_logits():
    a = tiny(scale=0.2)
    b = inputs.replace(a, scale=0.4, q=(a.q.float() * 0.5).to(torch.bfloat16))  # exact halving
    out_a, m_a = oracle.run(a)
    out_b, m_b = oracle.run(b)
    assert np.abs(out_a - out_b).max() < 1e-13 and np.abs(m_a - m_b).max() < 1e-13
    c = inputs.replace(a, scale=0.4)
    out_c, _ = oracle.run(c)
    assert np.abs(out_a - out_c).max() > 1e-3


# ------------------------------------------------------------------- library special case
@pytest.mark.parametrize("Hq,Hkv,D", [(4, 4, 16), (8, 2, 64)])
def test_hooks_off_matches_scaled_dot_product_attention(Hq, Hkv, D):
    L = 70
    case = inputs.make_case("sdpa", is_decode=False, seq_lens=[L], q_lens=[L], num_q_heads=Hq,
                            num_kv_heads=Hkv, head_dim=D, seed=21, shuffle=False, pool=1.0)
    out, mass = oracle.run(case)
    assert mass is None
    q = case.q.double().permute(1, 0, 2)[None]                                    # [1,Hq,L,D]
    k = case.k_cache.double().reshape(-1, Hkv, D)[:L].permute(1, 0, 2)[None]
    v = case.v_cache.double().reshape(-1, Hkv, D)[:L].permute(1, 0, 2)[None]
    k = k.repeat_interleave(Hq // Hkv, dim=1)
    v = v.repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(out - ref).max() < 1e-12


def test_named_configs_have_the_stated_shapes():
    c1 = inputs.config1_tiny_prefill()
    assert (c1.num_seqs, c1.total_q, c1.num_q_heads, c1.num_kv_heads, c1.head_dim) == (1, 256, 8, 8, 64)
    assert c1.spans.tolist() == [[[0, 64], [64, 256]]] and c1.num_probed == 8
    assert c1.alpha.tolist()[:3] == [0.5, 0.5, 0.0]
    c2 = inputs.config2_decode(num_seqs=8, lo=20, hi=60)
    assert c2.is_decode and c2.num_probed == 16 and int((c2.alpha != 0).sum()) == 4
    for s in range(8):
        L = int(c2.seq_lens[s])
        (a0, b0), (a1, b1) = c2.spans[s].tolist()
        assert a0 == 0 and b0 == a1 and b1 == L and 1 <= b0 <= max(L // 2, 1)
    m = inputs.config3_layer_masks()
    assert m.shape == (32, 32) and int(m.sum()) == 102
    c3 = inputs.config3_prefill(layer=1, num_seqs=1, tokens=64)
    assert c3.num_spans == 3 and c3.alpha is None
    sp = c3.spans[0].tolist()
    assert sp[0][0] == 0 and sp[-1][1] == 64 and all(sp[j][1] == sp[j + 1][0] for j in range(2))
    assert abs(c3.k_cache[c3.block_table[0, 0].item()].float().std().item() - 128 ** -0.5) < 0.01
