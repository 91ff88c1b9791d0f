"""The mixed step: a decode batch and prefill chunks issued together (hook_attn_mixed), against the oracle
and against the two stand-alone calls."""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2603_06588_b200 import binding, inputs

TOL_OUT = 2e-2
TOL_MASS = 1e-3


def _params(**over):
    p = binding.HookAttnParams()
    p.num_seqs, p.total_q, p.num_q_heads, p.num_kv_heads = 2, 2, 32, 8
    p.head_dim, p.page_size, p.num_blocks, p.max_blocks_per_seq = 128, 16, 64, 8
    fake = 0x10000
    p.q = p.k_cache = p.v_cache = p.block_table = p.seq_lens = p.cu_q_lens = p.out = fake
    p.kv_block_stride, p.kv_token_stride, p.kv_head_stride = 16 * 8 * 128, 8 * 128, 128
    for k, v in over.items():
        setattr(p, k, v)
    return p


def test_mixed_checks_both_halves_before_any_launch():
    lib = binding.load_library()
    ok_pf, ok_dec = _params(total_q=300), _params()
    call = lambda a, b: lib.hook_attn_mixed(None, ctypes.byref(a) if a is not None else None,
                                            ctypes.byref(b) if b is not None else None, None)
    assert call(None, ok_dec) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert call(ok_pf, None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert call(_params(total_q=300, head_dim=96), ok_dec) == binding.HOOK_ATTN_ERR_UNSUPPORTED
    assert call(ok_pf, _params(total_q=3)) == binding.HOOK_ATTN_ERR_INVALID_ARG          # decode: one row per sequence
    assert call(ok_pf, ok_dec) == binding.HOOK_ATTN_ERR_WORKSPACE                        # no workspace for the decode half
    need = lib.hook_attn_workspace_bytes(ctypes.byref(ok_dec), 2)
    assert need >= lib.hook_attn_workspace_bytes(ctypes.byref(ok_dec), 1) > 0
    # many units: the stand-alone call cuts fixed chunks, the one-launch path page shares; mode 2 covers both
    big = _params(num_seqs=256, total_q=256, num_q_heads=28, num_kv_heads=4, max_blocks_per_seq=512)
    assert lib.hook_attn_workspace_bytes(ctypes.byref(big), 2) >= lib.hook_attn_workspace_bytes(ctypes.byref(big), 1)
    ok_dec.workspace, ok_dec.workspace_bytes = 0x20000, need - 1
    assert call(ok_pf, ok_dec) == binding.HOOK_ATTN_ERR_WORKSPACE
    ok_dec.workspace_bytes = need
    assert call(ok_pf, ok_dec) == binding.HOOK_ATTN_ERR_INVALID_ARG                      # everything but the handle


# ---------------------------------------------------------------------------------------------- GPU
def _check_half(case, out, mass, rows=None):
    ref_out, ref_mass = oracle.run(case, rows)
    idx = list(range(case.total_q)) if rows is None else list(rows)
    got = out.float().cpu().numpy().astype(np.float64)[idx]
    assert np.isfinite(got).all() and np.abs(got - ref_out).max() <= TOL_OUT
    if ref_mass is not None:
        gm = mass.cpu().numpy().astype(np.float64)
        if case.is_decode or case.probe_rows == inputs.PROBE_ROWS_LAST:
            last = {r: s for s, r in zip([s for s in range(case.num_seqs) if case.q_lens()[s] > 0], oracle.last_rows(case))}
            sel = [i for i, r in enumerate(idx) if r in last]
            assert np.abs(gm[[last[idx[i]] for i in sel]] - ref_mass[sel]).max() <= TOL_MASS
        else:
            assert np.abs(gm[idx] - ref_mass).max() <= TOL_MASS


def _run_mixed(eng, pf, dec):
    st_pf = torch.zeros(1, dtype=torch.int32, device="cuda")
    st_dec = torch.zeros(1, dtype=torch.int32, device="cuda")
    (o_pf, m_pf), (o_dec, m_dec) = eng.hook_attn_mixed(dict(binding.case_to_device(pf), status=st_pf),
                                                       dict(binding.case_to_device(dec), status=st_dec))
    torch.cuda.synchronize()
    assert int(st_pf.item()) == 0 and int(st_dec.item()) == 0
    return o_pf, m_pf, o_dec, m_dec


@pytest.mark.gpu
@pytest.mark.parametrize("dec_ctas,spans_dec", [(0, 3), (1, 3), (37, 3), (0, 6), (0, 8)])
def test_mixed_small_ragged_step_matches_the_oracle(dec_ctas, spans_dec, monkeypatch):
    """Ragged decode batch (a unit shared by many warps, warps that cross units, empty shares) next to chunked
    prefill with partial tiles; every row of both halves is checked.  Run with the split chosen from the
    shapes, with a single decode CTA and with more decode CTAs than the batch has work for, and with span counts
    of the decode half on either side of the decode role's two probing forms (up to 4 spans, up to 8)."""
    if dec_ctas:
        monkeypatch.setenv("HOOK_ATTN_MIXED_DECODE_CTAS", str(dec_ctas))
    else:
        monkeypatch.delenv("HOOK_ATTN_MIXED_DECODE_CTAS", raising=False)
    eng = binding.HookAttn(0)
    g = inputs._gen(91)
    lens = torch.randint(1, 300, (40,), generator=g).tolist()
    lens[3], lens[17] = 5000, 1
    alpha = torch.zeros(8)
    alpha[2], alpha[5] = 0.8, -0.5
    mask = torch.tensor([1, 0, 0, 1, 1, 0, 1, 0], dtype=torch.uint8)
    dec = inputs.make_case("mix_dec", is_decode=True, seq_lens=lens, q_lens=[1] * len(lens), num_q_heads=8, num_kv_heads=2,
                           head_dim=128, seed=92, num_spans=spans_dec, head_mask=mask, alpha=alpha, steer=True,
                           probe_rows=inputs.PROBE_ROWS_LAST, poison=True)
    pf = inputs.make_case("mix_pf", is_decode=False, seq_lens=[700, 300, 90, 260], q_lens=[200, 300, 0, 129], num_q_heads=8,
                          num_kv_heads=2, head_dim=128, seed=93, num_spans=3, head_mask=mask, alpha=alpha, steer=True,
                          probe_rows=inputs.PROBE_ROWS_ALL, poison=True)
    o_pf, m_pf, o_dec, m_dec = _run_mixed(eng, pf, dec)
    _check_half(pf, o_pf, m_pf)
    _check_half(dec, o_dec, m_dec)
    # the prefill half runs the code of the stand-alone call: same bits
    ref_o, ref_m = eng.hook_attn_prefill(**binding.case_to_device(pf))
    torch.cuda.synchronize()
    assert torch.equal(ref_o.view(torch.int16), o_pf.view(torch.int16)) and torch.equal(ref_m, m_pf)
    # and the step is deterministic from run to run
    o_pf2, m_pf2, o_dec2, m_dec2 = _run_mixed(eng, pf, dec)
    assert torch.equal(o_dec.view(torch.int16), o_dec2.view(torch.int16)) and torch.equal(m_dec, m_dec2)


@pytest.mark.gpu
def test_mixed_full_size_step_matches_the_oracle():
    """The mixed chunked batch at full size: 256 decode sequences (all rows) plus two 2048-row chunks (the
    fixed row sample)."""
    eng = binding.HookAttn(0)
    dec, pf = inputs.config4_decode(), inputs.config4_prefill()
    o_pf, m_pf, o_dec, m_dec = _run_mixed(eng, pf, dec)
    _check_half(dec, o_dec, m_dec)
    _check_half(pf, o_pf, m_pf, rows=inputs.sample_rows(pf, extra_random=16))


@pytest.mark.gpu
def test_mixed_falls_back_to_the_two_calls_and_takes_empty_halves():
    eng = binding.HookAttn(0)
    # head_dim 64: not served by the one-launch kernel -> same bits as the two calls
    dec = inputs.make_case("fb_dec", is_decode=True, seq_lens=[70, 900, 33], q_lens=[1, 1, 1], num_q_heads=8, num_kv_heads=8,
                           head_dim=64, seed=5, num_spans=2, head_mask=torch.ones(8, dtype=torch.uint8),
                           probe_rows=inputs.PROBE_ROWS_LAST)
    pf = inputs.make_case("fb_pf", is_decode=False, seq_lens=[300, 140], q_lens=[300, 40], num_q_heads=8, num_kv_heads=8,
                          head_dim=64, seed=6, num_spans=2, head_mask=torch.ones(8, dtype=torch.uint8))
    o_pf, m_pf, o_dec, m_dec = _run_mixed(eng, pf, dec)
    r_pf = eng.hook_attn_prefill(**binding.case_to_device(pf))
    r_dec = eng.hook_attn_decode(**binding.case_to_device(dec))
    torch.cuda.synchronize()
    assert torch.equal(o_pf.view(torch.int16), r_pf[0].view(torch.int16)) and torch.equal(m_pf, r_pf[1])
    assert torch.equal(o_dec.view(torch.int16), r_dec[0].view(torch.int16)) and torch.equal(m_dec, r_dec[1])
    # more than 512 decode sequences at head_dim 128: the fallback as well
    many = inputs.make_case("fb_many", is_decode=True, seq_lens=[20] * 600, q_lens=[1] * 600, num_q_heads=2, num_kv_heads=1,
                            head_dim=128, seed=7)
    pf128 = inputs.make_case("fb_pf128", is_decode=False, seq_lens=[200], q_lens=[200], num_q_heads=2, num_kv_heads=1,
                             head_dim=128, seed=8)
    o_pf, _, o_dec, _ = _run_mixed(eng, pf128, many)
    _check_half(many, o_dec, None)
    _check_half(pf128, o_pf, None)
    # an empty prefill half: the decode call alone
    none = inputs.make_case("fb_none", is_decode=False, seq_lens=[50], q_lens=[0], num_q_heads=8, num_kv_heads=2,
                            head_dim=128, seed=9)
    d128 = inputs.config2_decode(num_seqs=5, lo=30, hi=400)
    o_pf, _, o_dec, m_dec = _run_mixed(eng, none, d128)
    assert o_pf.shape[0] == 0
    _check_half(d128, o_dec, m_dec)
