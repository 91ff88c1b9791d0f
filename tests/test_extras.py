"""Score reduction, residual-stream steering and raw q/k capture: oracle pins (CPU) and GPU parity."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import extras, oracle
from paper_2603_06588_b200 import binding, inputs


# ------------------------------------------------------------------ pins of the numpy oracles (CPU)
def test_score_oracle_closed_forms():
    # all mass on the instruction span -> 1 / 0; equal split -> 1/2 each; a dead head contributes zero
    m = np.array([[[0.7, 0.0], [0.2, 0.0]], [[0.3, 0.3], [0.1, 0.1]], [[0.4, 0.4], [0.0, 0.0]]])
    sn = extras.scores(m, extras.SCORE_SUM_NORMALIZE)
    assert np.allclose(sn[0], [1.0, 0.0]) and np.allclose(sn[1], [0.5, 0.5]) and np.allclose(sn[2], [0.25, 0.25])
    assert np.allclose(extras.scores(m, extras.SCORE_MEAN)[0], [0.45, 0.0])
    # brute force with python loops on random input
    g = np.random.default_rng(0)
    m = g.random((5, 3, 4))
    want = np.zeros((5, 4))
    for r in range(5):
        for j in range(4):
            want[r, j] = sum(m[r, p, j] / m[r, p].sum() for p in range(3)) / 3
    assert np.abs(extras.scores(m, 1) - want).max() < 1e-15
    assert np.abs(extras.scores(m, 1).sum(-1) - 1).max() < 1e-14          # normalised scores sum to one


def test_score_oracle_on_uniform_attention():
    """Identical keys give uniform attention, so the instruction score is |instr| / (|instr| + |data|)."""
    case = inputs.make_case("u", is_decode=True, seq_lens=[50], q_lens=[1], num_q_heads=4, num_kv_heads=2, head_dim=8,
                            seed=1, spans=torch.tensor([[[3, 13], [20, 50]]], dtype=torch.int32),
                            head_mask=torch.ones(4, dtype=torch.uint8))
    case.k_cache[:] = case.k_cache[case.block_table[0, 0].item(), 0, 0, :]
    _, mass = oracle.run(case)
    sc = extras.scores(mass, extras.SCORE_SUM_NORMALIZE)
    assert abs(sc[0, 0] - 10 / 40) < 1e-13 and abs(sc[0, 1] - 30 / 40) < 1e-13


def test_steer_oracle_and_capture_oracle_by_brute_force():
    h = torch.randn(3, 8, generator=inputs._gen(1)).to(torch.bfloat16)
    v = torch.randn(8, generator=inputs._gen(2))
    out = extras.steer_residual(h.float().numpy(), v.numpy(), -0.75)
    for t in range(3):
        for c in range(8):
            assert out[t, c] == float(h[t, c]) + (-0.75) * float(v[c])
    case = inputs.config2_decode(num_seqs=3, lo=5, hi=40)
    q_out, k_out, cu = extras.capture_qk(case)
    heads = [i for i in range(32) if case.head_mask[i]]
    assert cu.tolist() == [0] + np.cumsum(case.seq_lens.numpy()).tolist()
    s, t, pi = 1, int(case.seq_lens[1]) - 1, 5
    want = case.k_cache[case.block_table[s, t // 16].item(), t % 16, heads[pi] // 4].view(torch.int16).numpy()
    assert np.array_equal(k_out[cu[s] + t, pi], want)
    assert np.array_equal(q_out[2, 0], case.q[2, heads[0]].view(torch.int16).numpy())


def test_the_two_readings_of_sum_normalize_differ():
    """The paper names the reduction ("sum_normalize") and describes it in words only: attention on the
    instruction against attention on instruction plus data, over the important heads.  Two formulas fit
    those words.  (A, the library's) normalise every head's span masses by that head's total, then average
    the heads: each head votes with equal weight.  (B) sum the masses over the heads first, then normalise
    once: heads that put more mass on the configured spans weigh more.  They agree when all heads carry the
    same total and differ otherwise; this test keeps the difference visible."""
    m = np.array([[[0.10, 0.10], [0.60, 0.20]]])           # head 0: total 0.2, split 1:1; head 1: total 0.8, split 3:1
    a = extras.scores(m, extras.SCORE_SUM_NORMALIZE)[0]
    b = m[0].sum(axis=0) / m[0].sum()
    assert np.allclose(a, [(0.5 + 0.75) / 2, (0.5 + 0.25) / 2])      # 0.625 / 0.375
    assert np.allclose(b, [0.7, 0.3])
    assert abs(a[0] - b[0]) > 0.05
    same_totals = np.array([[[0.2, 0.2], [0.3, 0.1]]])                # both heads total 0.4: the readings coincide
    assert np.allclose(extras.scores(same_totals, extras.SCORE_SUM_NORMALIZE)[0], same_totals[0].sum(0) / same_totals[0].sum())


def _capture_by_loops(case):
    """The capture payload written out with explicit loops over (sequence, key, probed head) on K gathered
    contiguously by tests/_brute.py -- nothing shared with oracle/extras.py."""
    from tests import _brute
    hq, hkv, d = case.num_q_heads, case.num_kv_heads, case.head_dim
    heads = [h for h in range(hq) if int(case.head_mask[h])]
    cu_q = case.cu_q_lens.tolist()
    lens = case.seq_lens.tolist()
    last_only = case.is_decode or case.probe_rows == inputs.PROBE_ROWS_LAST
    q = case.q.float().numpy()
    k_rows, q_rows = [], []
    for s in range(case.num_seqs):
        k, _ = _brute.gather_contiguous(case, s)                       # [L, Hkv, D]
        for t in range(lens[s]):
            k_rows.append([[float(k[t, h // (hq // hkv), e]) for e in range(d)] for h in heads])
        n = cu_q[s + 1] - cu_q[s]
        if last_only:
            q_rows.append([[float(q[cu_q[s + 1] - 1, h, e]) if n > 0 else 0.0 for e in range(d)] for h in heads])
        else:
            for i in range(n):
                q_rows.append([[float(q[cu_q[s] + i, h, e]) for e in range(d)] for h in heads])
    cu_k = [0]
    for L in lens:
        cu_k.append(cu_k[-1] + L)
    return np.array(q_rows, dtype=np.float64).reshape(-1, len(heads), d), np.array(k_rows, dtype=np.float64).reshape(-1, len(heads), d), cu_k


@pytest.mark.parametrize("mode", ["decode", "all_tokens", "last_token"])
def test_capture_oracle_every_element_in_all_three_modes(mode):
    """Tiny case, every element: a sequence without rows in the call, probed heads that skip a KV head and
    share another (heads 0, 1 -> KV 0; 5 -> KV 2; 7 -> KV 3), sequence lengths that end inside a page."""
    mask = torch.tensor([1, 1, 0, 0, 0, 1, 0, 1], dtype=torch.uint8)
    if mode == "decode":
        case = inputs.make_case("cap_pin_d", is_decode=True, seq_lens=[5, 33, 16], q_lens=[1, 1, 1], num_q_heads=8,
                                num_kv_heads=4, head_dim=8, seed=41, head_mask=mask, poison=True)
    else:
        case = inputs.make_case("cap_pin_p", is_decode=False, seq_lens=[5, 33, 16, 20], q_lens=[5, 0, 3, 20], num_q_heads=8,
                                num_kv_heads=4, head_dim=8, seed=42, head_mask=mask, poison=True,
                                probe_rows=inputs.PROBE_ROWS_LAST if mode == "last_token" else inputs.PROBE_ROWS_ALL)
    q_out, k_out, cu = extras.capture_qk(case)
    want_q, want_k, want_cu = _capture_by_loops(case)
    as_f = lambda bits: torch.from_numpy(np.ascontiguousarray(bits)).view(torch.bfloat16).float().numpy().astype(np.float64)
    assert cu.tolist() == want_cu
    assert q_out.shape == want_q.shape and k_out.shape == want_k.shape
    assert np.array_equal(as_f(k_out), want_k)
    assert np.array_equal(as_f(q_out), want_q)
    if mode == "last_token":
        assert not q_out[1].any()                                      # the sequence without rows: zeros
        assert np.array_equal(as_f(q_out)[2, 3], case.q[7, 7].float().numpy())   # sequence 2's last row is global row 7


def test_extras_reject_bad_arguments_without_a_gpu():
    lib = binding.load_library()
    assert lib.hook_attn_score(None, 0x1000, 4, 0, 2, 1, 0x1000, None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert lib.hook_attn_score(None, 0x1000, 4, 2, 9, 1, 0x1000, None) == binding.HOOK_ATTN_ERR_UNSUPPORTED
    assert lib.hook_attn_score(None, 0x1000, 4, 2, 2, 5, 0x1000, None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert lib.hook_attn_score(None, 0x1000, 4, 2, 2, 1, 0x1000, None) == binding.HOOK_ATTN_ERR_INVALID_ARG   # no handle
    assert lib.hook_steer_residual(None, 0x1000, 0x1000, 1.0, 4, 12, 12, None) == binding.HOOK_ATTN_ERR_UNSUPPORTED
    assert lib.hook_steer_residual(None, 0x1000, 0x1000, 1.0, 4, 16, 8, None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert lib.hook_steer_residual(None, 0x1000, 0x1000, float("nan"), 4, 16, 16, None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    assert lib.hook_capture_qk(None, None, 1, None, None, None, None) == binding.HOOK_ATTN_ERR_INVALID_ARG


# ---------------------------------------------------------------------------------- GPU parity
@pytest.fixture(scope="module")
def eng():
    return binding.HookAttn(0)


@pytest.mark.gpu
@pytest.mark.parametrize("mode", [binding.HOOK_SCORE_MEAN, binding.HOOK_SCORE_SUM_NORMALIZE])
def test_score_matches_oracle(eng, mode):
    g = inputs._gen(5)
    for shape in [(1, 1, 1), (7, 16, 2), (300, 41, 8), (64, 3, 5)]:
        m = torch.rand(shape, generator=g, dtype=torch.float32)
        m[0, 0] = 0.0                                          # a head with no mass on any span
        got = eng.hook_attn_score(m.cuda(), mode).cpu().numpy()
        want = extras.scores(m.numpy(), mode)
        assert np.abs(got - want).max() <= 1e-5


@pytest.mark.gpu
def test_score_end_to_end_from_decode(eng):
    """decode -> span_mass -> instruction score, all on the device; only [num_seqs, 2] floats come back."""
    case = inputs.config2_decode(num_seqs=12, lo=60, hi=900)
    kw = binding.case_to_device(case)
    _, mass = eng.hook_attn_decode(**kw)
    sc = eng.hook_attn_score(mass, binding.HOOK_SCORE_SUM_NORMALIZE)
    torch.cuda.synchronize()
    _, ref_mass = oracle.run(case)
    want = extras.scores(ref_mass, extras.SCORE_SUM_NORMALIZE)
    assert np.abs(sc.cpu().numpy() - want).max() <= 1e-3
    assert np.abs(sc.cpu().numpy().sum(-1) - 1.0).max() <= 1e-5     # the two spans partition the context


@pytest.mark.gpu
@pytest.mark.parametrize("T,H,pad", [(1, 8, 0), (37, 4096, 0), (513, 1536, 64), (0, 64, 0)])
def test_residual_steering_matches_oracle(eng, T, H, pad):
    g = inputs._gen(T + H)
    h = (torch.randn(T, H + pad, generator=g) * 3).to(torch.bfloat16)
    v = torch.randn(H, generator=g)
    alpha = 1.75
    dev = h.cuda()
    view = dev[:, :H]                                          # strided rows when pad > 0
    eng.hook_steer_residual(view, v.cuda(), alpha)
    torch.cuda.synchronize()
    want = extras.steer_residual(h[:, :H].float().numpy(), v.numpy(), alpha)
    got = dev[:, :H].float().cpu().numpy().astype(np.float64)
    # fp32 add then one rounding to bf16: within half a bf16 ulp (2^-9 relative) of the exact sum
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)
    if pad:
        assert torch.equal(dev[:, H:].cpu().view(torch.int16), h[:, H:].view(torch.int16))   # padding untouched
    before = dev.clone()
    eng.hook_steer_residual(view, v.cuda(), 0.0)               # alpha = 0 leaves every bit in place
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.int16), dev.view(torch.int16))


@pytest.mark.gpu
@pytest.mark.parametrize("which", ["decode", "prefill_all", "prefill_last", "d64"])
def test_capture_is_byte_exact(eng, which):
    if which == "decode":
        case = inputs.config2_decode(num_seqs=9, lo=1, hi=700, poison=True)
    elif which == "d64":
        case = inputs.make_case("c64", is_decode=True, seq_lens=[5, 64, 129], q_lens=[1, 1, 1], num_q_heads=8,
                                num_kv_heads=8, head_dim=64, seed=4, head_mask=torch.tensor([0, 1, 1, 0, 0, 0, 0, 1], dtype=torch.uint8))
    else:
        case = inputs.make_case("cap", is_decode=False, seq_lens=[300, 40, 77], q_lens=[300, 0, 5], num_q_heads=14,
                                num_kv_heads=2, head_dim=128, seed=9, head_mask=inputs.choose_heads(14, 5, inputs._gen(3)),
                                probe_rows=inputs.PROBE_ROWS_LAST if which == "prefill_last" else inputs.PROBE_ROWS_ALL,
                                poison=True)
    kw = binding.case_to_device(case)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q_out, k_out, cu = eng.hook_capture_qk(case.is_decode, status=status, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rq, rk, rcu = extras.capture_qk(case)
    assert np.array_equal(cu.cpu().numpy(), rcu)
    assert np.array_equal(q_out.cpu().view(torch.int16).numpy(), rq)
    assert np.array_equal(k_out.cpu().view(torch.int16).numpy(), rk)
