"""hook_attn_decode_static_scratch: the decode entry point for callers that cannot allocate.

Some users of the library run where device allocation is not available to them -- inside a
serving loop whose memory is fully committed to the KV cache, or as a plug-in that only sees the
tensors of the layer it hooks -- so they can neither create nor pass the split-K workspace.  This
entry point keeps the partials in a fixed array inside the library instead.  The test drives it
through the C ABI twice in a row (a larger batch first, then a different, smaller one, so that
the second call finds the first call's leftovers in the array) and compares each result with what
the regular entry point returns for the same inputs.

This file is collected last on purpose: if it fails, a run that stops at the first failure has
already executed every other test.
"""
import ctypes

import pytest
import torch

from paper_2603_06588_b200 import binding, inputs

TOL_OUT = 2e-2     # same tolerances as the parity tests
TOL_MASS = 1e-3


def _fake_params(**over):
    p = binding.HookAttnParams()
    p.num_seqs, p.total_q, p.num_q_heads, p.num_kv_heads = 2, 2, 32, 8
    p.head_dim, p.page_size, p.num_blocks, p.max_blocks_per_seq = 128, 16, 64, 8
    fake = 0x10000
    p.q = p.k_cache = p.v_cache = p.block_table = p.seq_lens = p.out = fake
    p.kv_block_stride, p.kv_token_stride, p.kv_head_stride = 16 * 8 * 128, 8 * 128, 128
    for k, v in over.items():
        setattr(p, k, v)
    return p


def test_batches_beyond_the_fixed_array_are_refused_before_any_launch():
    lib = binding.load_library()
    # 4096 sequences x 8 KV heads x 2056 pages: far more partials than the array holds
    big = _fake_params(num_seqs=4096, total_q=4096, max_blocks_per_seq=2056)
    assert lib.hook_attn_workspace_bytes(ctypes.byref(big), 1) > binding.STATIC_SCRATCH_BYTES
    assert lib.hook_attn_decode_static_scratch(None, ctypes.byref(big), None) == binding.HOOK_ATTN_ERR_WORKSPACE
    # a batch that fits is only stopped by the missing handle; bad shapes keep their own codes
    small = _fake_params()
    assert lib.hook_attn_workspace_bytes(ctypes.byref(small), 1) <= binding.STATIC_SCRATCH_BYTES
    assert lib.hook_attn_decode_static_scratch(None, ctypes.byref(small), None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    bad = _fake_params(head_dim=96)
    assert lib.hook_attn_decode_static_scratch(None, ctypes.byref(bad), None) == binding.HOOK_ATTN_ERR_UNSUPPORTED


@pytest.mark.gpu
def test_static_scratch_decode_matches_the_regular_entry_point_twice_in_a_row():
    torch.cuda.set_device(0)
    eng = binding.HookAttn(0)
    cases = [inputs.config2_decode(num_seqs=48, lo=200, hi=3000, seed_offset=7),
             inputs.config2_decode(num_seqs=5, lo=17, hi=900, seed_offset=11)]
    for case in cases:
        kw = binding.case_to_device(case)
        ref_out, ref_mass = eng.hook_attn_decode(**kw)              # regular path, caller-side workspace
        torch.cuda.synchronize()

        out = torch.full_like(ref_out, float("nan"))
        mass = torch.full_like(ref_mass, float("nan"))
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        p, keep = binding.make_params(out=out, span_mass=mass, status=status, **kw)   # no workspace passed
        assert p.workspace is None and p.workspace_bytes == 0
        assert eng.workspace_bytes(p, True) <= binding.STATIC_SCRATCH_BYTES
        before = torch.cuda.memory_allocated()
        rc = eng.call_decode_static_scratch(p)
        assert rc == binding.HOOK_ATTN_OK, binding.strerror(rc)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert int(status.item()) == 0
        err_o = (out.float() - ref_out.float()).abs().max().item()
        err_m = (mass - ref_mass).abs().max().item()
        assert err_o <= TOL_OUT and err_m <= TOL_MASS, (case.name, err_o, err_m)
        # same kernels, same chunking, same merge order: the bits agree as well
        assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16))
        assert torch.equal(mass, ref_mass)
        del keep
