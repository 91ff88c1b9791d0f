"""CPU-side checks of the C-ABI boundary: the library loads without a GPU, exports every
symbol the header declares, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest
import torch

import __graft_entry__  # noqa: F401  (repo root on sys.path via conftest)
from paper_2603_06588_b200 import binding
from paper_2603_06588_b200.csrc import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hook_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hook_attn_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert {"hook_attn_create", "hook_attn_destroy", "hook_attn_prefill", "hook_attn_decode",
            "hook_attn_workspace_bytes", "hook_attn_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in the header but not exported"


def test_struct_mirror_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "hook_attn.h")).read()
    body = text[text.index("typedef struct {"):text.index("} hook_attn_params;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        names = decl.split(",")
        first = names[0].split()[-1].lstrip("*")
        fields.append(first)
        fields.extend(n.strip().lstrip("*") for n in names[1:])
    assert fields == [f[0] for f in binding.HookAttnParams._fields_]


def test_strerror(lib):
    assert binding.strerror(0) == "ok"
    for code in range(-6, 0):
        assert binding.strerror(code) not in ("ok", "unknown code")
    assert binding.strerror(-99) == "unknown code"


def _params(**over):
    """A structurally valid parameter block with fake (never dereferenced) device addresses."""
    p = binding.HookAttnParams()
    p.num_seqs, p.total_q, p.num_q_heads, p.num_kv_heads = 2, 2, 32, 8
    p.head_dim, p.page_size, p.num_blocks, p.max_blocks_per_seq = 128, 16, 64, 8
    p.num_spans, p.probe_rows, p.scale = 0, 0, 0.0
    fake = 0x10000
    p.q = p.k_cache = p.v_cache = p.block_table = p.seq_lens = p.cu_q_lens = p.out = fake
    p.kv_block_stride, p.kv_token_stride, p.kv_head_stride = 16 * 8 * 128, 8 * 128, 128
    for k, v in over.items():
        setattr(p, k, v)
    return p


@pytest.mark.parametrize("over,code", [
    (dict(num_q_heads=30), binding.HOOK_ATTN_ERR_INVALID_ARG),          # Hq % Hkv != 0
    (dict(head_dim=96), binding.HOOK_ATTN_ERR_UNSUPPORTED),
    (dict(page_size=32), binding.HOOK_ATTN_ERR_UNSUPPORTED),
    (dict(num_q_heads=128, num_kv_heads=16), binding.HOOK_ATTN_ERR_UNSUPPORTED),
    (dict(num_q_heads=32, num_kv_heads=2), binding.HOOK_ATTN_ERR_UNSUPPORTED),   # group 16
    (dict(num_spans=9), binding.HOOK_ATTN_ERR_UNSUPPORTED),
    (dict(num_seqs=-1), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(max_seq_len=-1), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(probe_rows=7), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(q=None), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(out=None), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(block_table=None), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(kv_head_stride=100), binding.HOOK_ATTN_ERR_UNSUPPORTED),      # not a multiple of 8
    (dict(kv_token_stride=0), binding.HOOK_ATTN_ERR_INVALID_ARG),
    (dict(q=0x10002), binding.HOOK_ATTN_ERR_UNSUPPORTED),               # misaligned
])
def test_bad_arguments_are_rejected_before_any_launch(lib, over, code):
    p = _params(**over)
    for fn in (lib.hook_attn_prefill, lib.hook_attn_decode):
        assert fn(None, ctypes.byref(p), None) == code


def test_hook_arguments_are_checked(lib):
    hm = (ctypes.c_uint8 * 32)(*([1] * 32))
    al = (ctypes.c_float * 32)(*([0.5] * 32))
    # probed heads but no span list / no output buffer
    p = _params(num_spans=2, head_mask=ctypes.addressof(hm))
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    # steered heads but no steering vectors
    p = _params(alpha=ctypes.addressof(al))
    assert lib.hook_attn_prefill(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    # non-finite alpha
    al[3] = float("nan")
    p = _params(alpha=ctypes.addressof(al), steer_vec=0x10000)
    assert lib.hook_attn_prefill(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_INVALID_ARG


def test_decode_shape_and_workspace_checks(lib):
    p = _params(total_q=3)                                   # decode needs one row per sequence
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    p = _params()
    need = lib.hook_attn_workspace_bytes(ctypes.byref(p), 1)
    assert need > 0 and lib.hook_attn_workspace_bytes(ctypes.byref(p), 0) == 0
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_WORKSPACE
    p.workspace, p.workspace_bytes = 0x20000, need - 1
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_WORKSPACE
    p.workspace_bytes = need
    p.workspace = 0x20010                                    # the header asks for 256-byte alignment
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_WORKSPACE
    p.workspace = 0x20000
    # everything valid except the handle: still refused, and nothing was launched
    assert lib.hook_attn_decode(None, ctypes.byref(p), None) == binding.HOOK_ATTN_ERR_INVALID_ARG
    # invalid shapes size to zero
    assert lib.hook_attn_workspace_bytes(ctypes.byref(_params(head_dim=96)), 1) == 0
    assert lib.hook_attn_workspace_bytes(None, 1) == 0


def test_workspace_scales_with_the_bounds(lib):
    # one partial per (sequence, KV head) plus one per worker of the fixed grid
    a = lib.hook_attn_workspace_bytes(ctypes.byref(_params(num_seqs=4, total_q=4)), 1)
    b = lib.hook_attn_workspace_bytes(ctypes.byref(_params(num_seqs=8, total_q=8)), 1)
    c = lib.hook_attn_workspace_bytes(ctypes.byref(_params(num_seqs=12, total_q=12)), 1)
    assert a > 0 and c - b == b - a > 0


def test_length_bound_sizes_the_workspace_instead_of_the_table_width(lib):
    """A block table padded to a model's maximum length must not inflate the plan: with the host's bound
    on the sequence lengths the workspace is the one of the tight table."""
    tight = lib.hook_attn_workspace_bytes(ctypes.byref(_params(num_seqs=64, total_q=64, max_blocks_per_seq=256)), 1)
    padded = lib.hook_attn_workspace_bytes(ctypes.byref(_params(num_seqs=64, total_q=64, max_blocks_per_seq=8192)), 1)
    hinted = lib.hook_attn_workspace_bytes(
        ctypes.byref(_params(num_seqs=64, total_q=64, max_blocks_per_seq=8192, max_seq_len=4096)), 1)
    assert padded > tight and hinted == tight
    # a bound beyond what the table can address changes nothing
    same = lib.hook_attn_workspace_bytes(
        ctypes.byref(_params(num_seqs=64, total_q=64, max_blocks_per_seq=256, max_seq_len=1 << 20)), 1)
    assert same == tight


@pytest.mark.gpu
def test_the_handles_device_must_be_current():
    """Every entry point that launches refuses a handle whose device is not the current one.  The box has
    one GPU, so the test edits the device ordinal the handle remembers (its first field) instead of
    switching devices, and puts it back."""
    from paper_2603_06588_b200 import inputs
    eng = binding.HookAttn(0)
    lib_ = binding.load_library()
    case = inputs.config2_decode(num_seqs=2, lo=20, hi=60)
    kw = binding.case_to_device(case)
    plan = eng.plan(True, **kw)
    plan.run()
    torch.cuda.synchronize()
    field = ctypes.cast(eng._h, ctypes.POINTER(ctypes.c_int))
    assert field[0] == 0
    field[0] = 1
    try:
        stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        ref = ctypes.byref(plan.params)
        assert lib_.hook_attn_decode(eng._h, ref, stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
        assert lib_.hook_attn_decode_static_scratch(eng._h, ref, stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
        pf = inputs.config3_prefill(layer=0, num_seqs=1, tokens=256, force_probe=True)
        pkw = binding.case_to_device(pf)
        pout = torch.empty_like(pkw["q"])
        pmass = torch.zeros(pf.total_q, pf.num_probed, pf.num_spans, device="cuda")
        pp, _keep = binding.make_params(out=pout, span_mass=pmass, **pkw)
        assert lib_.hook_attn_prefill(eng._h, ctypes.byref(pp), stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
        m = torch.zeros(2, 2, 2, device="cuda")
        assert lib_.hook_attn_score(eng._h, m.data_ptr(), 2, 2, 2, 1, m.data_ptr(), stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
        h = torch.zeros(4, 16, dtype=torch.bfloat16, device="cuda")
        v = torch.zeros(16, device="cuda")
        assert lib_.hook_steer_residual(eng._h, h.data_ptr(), v.data_ptr(), 1.0, 4, 16, 16, stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        assert lib_.hook_attn_selftest_wait_limit(eng._h, st.data_ptr(), 1000, None, stream) == binding.HOOK_ATTN_ERR_INVALID_ARG
    finally:
        field[0] = 0
    plan.run()                                                # the handle works again
    torch.cuda.synchronize()


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a GPU")
def test_create_fails_cleanly_without_a_device(lib):
    h = ctypes.c_void_p()
    assert lib.hook_attn_create(ctypes.byref(h), 0) == binding.HOOK_ATTN_ERR_CUDA
    assert not h.value
    with pytest.raises(binding.HookAttnError):
        binding.HookAttn(0)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.load_library()
