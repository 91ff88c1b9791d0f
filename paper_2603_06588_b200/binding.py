"""Thin ctypes binding of ``libhook_attn.so`` (declared in ``include/hook_attn.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels.  PyTorch is used
for device memory and streams.  There is no CPU fallback -- if the compiled library is missing
the import of this module's entry points fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libhook_attn.so")

HOOK_ATTN_OK = 0
HOOK_ATTN_ERR_INVALID_ARG = -1
HOOK_ATTN_ERR_UNSUPPORTED = -2
HOOK_ATTN_ERR_WORKSPACE = -3
HOOK_ATTN_ERR_CUDA = -4
HOOK_ATTN_ERR_TIMEOUT = -5
HOOK_ATTN_ERR_BOUNDS = -6
HOOK_PROBE_ROWS_ALL = 0
HOOK_PROBE_ROWS_LAST = 1

EXPORTS = ("hook_attn_create", "hook_attn_destroy", "hook_attn_workspace_bytes",
           "hook_attn_prefill", "hook_attn_decode", "hook_attn_mixed", "hook_attn_decode_static_scratch",
           "hook_attn_score", "hook_steer_residual", "hook_capture_qk", "hook_attn_selftest_wait_limit",
           "hook_attn_strerror")
HOOK_SCORE_MEAN = 0
HOOK_SCORE_SUM_NORMALIZE = 1
STATIC_SCRATCH_BYTES = 16 << 20   # HOOK_ATTN_STATIC_SCRATCH_BYTES


class HookAttnParams(ctypes.Structure):
    """Mirror of ``hook_attn_params``."""
    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("total_q", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("num_blocks", ctypes.c_int32), ("max_blocks_per_seq", ctypes.c_int32),
        ("num_spans", ctypes.c_int32), ("probe_rows", ctypes.c_int32),
        ("scale", ctypes.c_float), ("max_seq_len", ctypes.c_int32),
        ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("kv_block_stride", ctypes.c_int64), ("kv_token_stride", ctypes.c_int64),
        ("kv_head_stride", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p),
        ("cu_q_lens", ctypes.c_void_p), ("spans", ctypes.c_void_p),
        ("steer_vec", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("span_mass", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("status", ctypes.c_void_p),
        ("head_mask", ctypes.c_void_p), ("alpha", ctypes.c_void_p),
    ]


class HookAttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} (code {code})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Load the compiled CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2603_06588_b200.csrc.build` "
                "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        lib.hook_attn_create.restype = ctypes.c_int
        lib.hook_attn_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int]
        lib.hook_attn_destroy.restype = ctypes.c_int
        lib.hook_attn_destroy.argtypes = [ctypes.c_void_p]
        lib.hook_attn_workspace_bytes.restype = ctypes.c_size_t
        lib.hook_attn_workspace_bytes.argtypes = [ctypes.POINTER(HookAttnParams), ctypes.c_int]
        for name in ("hook_attn_prefill", "hook_attn_decode", "hook_attn_decode_static_scratch"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.c_void_p, ctypes.POINTER(HookAttnParams), ctypes.c_void_p]
        lib.hook_attn_mixed.restype = ctypes.c_int
        lib.hook_attn_mixed.argtypes = [ctypes.c_void_p, ctypes.POINTER(HookAttnParams), ctypes.POINTER(HookAttnParams),
                                        ctypes.c_void_p]
        lib.hook_attn_score.restype = ctypes.c_int
        lib.hook_attn_score.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                        ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        lib.hook_steer_residual.restype = ctypes.c_int
        lib.hook_steer_residual.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                            ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p]
        lib.hook_capture_qk.restype = ctypes.c_int
        lib.hook_capture_qk.argtypes = [ctypes.c_void_p, ctypes.POINTER(HookAttnParams), ctypes.c_int, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.hook_attn_selftest_wait_limit.restype = ctypes.c_int
        lib.hook_attn_selftest_wait_limit.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                                                      ctypes.c_void_p]
        lib.hook_attn_strerror.restype = ctypes.c_char_p
        lib.hook_attn_strerror.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    return load_library().hook_attn_strerror(int(code)).decode()


def _dptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_params(*, q, k_cache, v_cache, block_table, seq_lens, cu_q_lens=None, spans=None,
                head_mask=None, alpha=None, steer_vec=None, scale: float = 0.0,
                probe_rows: int = HOOK_PROBE_ROWS_ALL, out=None, span_mass=None, workspace=None,
                status=None, max_seq_len: int = 0) -> Tuple[HookAttnParams, list]:
    """Marshal tensors into a ``hook_attn_params``.  ``head_mask`` / ``alpha`` are HOST tensors
    (uint8 / float32); everything else lives on the device.  Returns the struct and a list of
    objects that must stay alive until the call has been issued."""
    keep = []
    p = HookAttnParams()
    total_q, hq, d = q.shape
    nb, page, hkv, d2 = k_cache.shape
    assert d2 == d and v_cache.shape == k_cache.shape and v_cache.stride() == k_cache.stride()
    assert k_cache.stride(3) == 1 and q.is_contiguous()
    p.num_seqs = int(seq_lens.shape[0])
    p.total_q = int(total_q)
    p.num_q_heads, p.num_kv_heads, p.head_dim, p.page_size = int(hq), int(hkv), int(d), int(page)
    p.num_blocks = int(nb)
    p.max_blocks_per_seq = int(block_table.shape[1]) if block_table.dim() == 2 else 0
    p.num_spans = 0 if spans is None else int(spans.shape[1])
    p.probe_rows = int(probe_rows)
    p.scale = float(scale)
    p.max_seq_len = int(max_seq_len)
    p.q, p.k_cache, p.v_cache = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr()
    p.kv_block_stride, p.kv_token_stride, p.kv_head_stride = (int(k_cache.stride(0)),
                                                               int(k_cache.stride(1)),
                                                               int(k_cache.stride(2)))
    p.block_table, p.seq_lens = block_table.data_ptr(), seq_lens.data_ptr()
    p.cu_q_lens = _dptr(cu_q_lens)
    p.spans = _dptr(spans)
    p.steer_vec = _dptr(steer_vec)
    p.out = _dptr(out)
    p.span_mass = _dptr(span_mass)
    p.workspace = _dptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    p.status = _dptr(status)
    if head_mask is not None:
        hm = head_mask.detach().to("cpu", torch.uint8).contiguous()
        keep.append(hm)
        p.head_mask = hm.data_ptr()
    if alpha is not None:
        al = alpha.detach().to("cpu", torch.float32).contiguous()
        keep.append(al)
        p.alpha = al.data_ptr()
    return p, keep


class HookAttn:
    """Per-device handle plus the two entry points, taking torch CUDA tensors."""

    def __init__(self, device: int = 0):
        lib = load_library()
        h = ctypes.c_void_p()
        rc = lib.hook_attn_create(ctypes.byref(h), int(device))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_attn_create")
        self._lib = lib
        self._h = h
        self.device = torch.device("cuda", int(device))

    def close(self):
        if getattr(self, "_h", None):
            self._lib.hook_attn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- raw calls -----------------------------------------------------------------------
    def workspace_bytes(self, params: HookAttnParams, is_decode) -> int:
        """``is_decode``: False / True, or 2 for the decode half of a mixed step."""
        return int(self._lib.hook_attn_workspace_bytes(ctypes.byref(params), int(is_decode)))

    def call(self, params: HookAttnParams, is_decode: bool, stream: Optional[int] = None) -> int:
        """Issue the call described by ``params``; returns the library's return code."""
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        fn = self._lib.hook_attn_decode if is_decode else self._lib.hook_attn_prefill
        return int(fn(self._h, ctypes.byref(params), ctypes.c_void_p(stream)))

    def call_decode_static_scratch(self, params: HookAttnParams, stream: Optional[int] = None) -> int:
        """``hook_attn_decode_static_scratch``: decode for callers that cannot allocate or pass
        scratch; the partials go into the library's fixed array (``STATIC_SCRATCH_BYTES``).
        Returns the library's return code."""
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        return int(self._lib.hook_attn_decode_static_scratch(self._h, ctypes.byref(params),
                                                             ctypes.c_void_p(stream)))

    def selftest_wait_limit(self, limit_ns: int = 200_000_000, stream=None):
        """Run the bounded-wait self-test; returns ``(status_code, waited_ns)`` read back from the device."""
        status = torch.zeros(1, dtype=torch.int32, device=self.device)
        waited = torch.zeros(1, dtype=torch.int64, device=self.device)
        rc = int(self._lib.hook_attn_selftest_wait_limit(self._h, status.data_ptr(), int(limit_ns), waited.data_ptr(),
                                                         self._stream(stream)))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_attn_selftest_wait_limit")
        torch.cuda.synchronize(self.device)
        return int(status.item()), int(waited.item())

    def _stream(self, stream):
        return ctypes.c_void_p(torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream)

    def hook_attn_score(self, span_mass: torch.Tensor, mode: int = HOOK_SCORE_SUM_NORMALIZE, scores=None, stream=None):
        """Analyzer reduction: ``span_mass`` fp32 ``[R, P, S]`` (device) -> ``scores`` fp32 ``[R, S]``."""
        rows, nprobed, nspans = span_mass.shape
        assert span_mass.dtype == torch.float32 and span_mass.is_contiguous()
        if scores is None:
            scores = torch.empty((rows, nspans), dtype=torch.float32, device=span_mass.device)
        rc = int(self._lib.hook_attn_score(self._h, span_mass.data_ptr(), rows, nprobed, nspans, int(mode),
                                           scores.data_ptr(), self._stream(stream)))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_attn_score")
        return scores

    def hook_steer_residual(self, hidden: torch.Tensor, steer_vec: torch.Tensor, alpha: float, stream=None):
        """Residual-stream steering in place: ``hidden`` bf16 ``[T, H]`` (device, rows may be strided),
        ``steer_vec`` fp32 ``[H]``."""
        assert hidden.dtype == torch.bfloat16 and hidden.dim() == 2 and hidden.stride(1) == 1
        assert steer_vec.dtype == torch.float32 and steer_vec.is_contiguous()
        rc = int(self._lib.hook_steer_residual(self._h, hidden.data_ptr(), steer_vec.data_ptr(), float(alpha),
                                               hidden.shape[0], hidden.shape[1], hidden.stride(0), self._stream(stream)))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_steer_residual")
        return hidden

    def hook_capture_qk(self, is_decode: bool, *, q, k_cache, v_cache, block_table, seq_lens, cu_q_lens=None,
                        head_mask=None, probe_rows=HOOK_PROBE_ROWS_ALL, status=None, stream=None,
                        q_out=None, k_out=None, cu_k_lens=None, max_seq_len: int = 0, **_ignored):
        """Raw q/k capture of the probed heads.  Returns ``(q_out [rows, P, D], k_out [sum L, P, D], cu_k_lens)``.
        The three outputs are allocated (and the prefix sums computed, with one host sync for the total)
        unless the caller passes them."""
        nprobed = 0 if head_mask is None else int((head_mask != 0).sum())
        total_q, hq, d = q.shape
        last_only = is_decode or probe_rows == HOOK_PROBE_ROWS_LAST
        rows = int(seq_lens.shape[0]) if last_only else int(total_q)
        cu_k = cu_k_lens
        if cu_k is None:
            cu_k = torch.zeros(seq_lens.shape[0] + 1, dtype=torch.int32, device=q.device)
            cu_k[1:] = torch.cumsum(seq_lens, 0)
        if q_out is None:
            q_out = torch.zeros((rows, nprobed, d), dtype=torch.bfloat16, device=q.device)
        if k_out is None:
            k_out = torch.zeros((int(cu_k[-1].item()), nprobed, d), dtype=torch.bfloat16, device=q.device)
        p, keep = make_params(q=q, k_cache=k_cache, v_cache=v_cache, block_table=block_table, seq_lens=seq_lens,
                              cu_q_lens=cu_q_lens, head_mask=head_mask, probe_rows=probe_rows, status=status,
                              max_seq_len=max_seq_len)
        rc = int(self._lib.hook_capture_qk(self._h, ctypes.byref(p), int(bool(is_decode)), q_out.data_ptr(),
                                           k_out.data_ptr(), cu_k.data_ptr(), self._stream(stream)))
        del keep
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_capture_qk")
        return q_out, k_out, cu_k

    # -- convenience ---------------------------------------------------------------------
    def plan(self, is_decode: bool, *, q, k_cache, v_cache, block_table, seq_lens, cu_q_lens=None,
             spans=None, head_mask=None, alpha=None, steer_vec=None, scale=0.0,
             probe_rows=HOOK_PROBE_ROWS_ALL, out=None, span_mass=None, status=None,
             max_seq_len: int = 0, mixed_half: bool = False) -> "HookAttnPlan":
        """Marshal the arguments once (allocating `out`, `span_mass` and scratch when they are not
        given); the returned plan re-issues the same call with one C call per step."""
        total_q, hq, d = q.shape
        if out is None:
            out = torch.empty_like(q)
        nprobed = 0 if head_mask is None else int((head_mask != 0).sum())
        nspans = 0 if spans is None else int(spans.shape[1])
        if span_mass is None and nprobed and nspans:
            rows = seq_lens.shape[0] if (is_decode or probe_rows == HOOK_PROBE_ROWS_LAST) else total_q
            span_mass = torch.zeros((rows, nprobed, nspans), dtype=torch.float32, device=q.device)
        p, keep = make_params(q=q, k_cache=k_cache, v_cache=v_cache, block_table=block_table,
                              seq_lens=seq_lens, cu_q_lens=cu_q_lens, spans=spans,
                              head_mask=head_mask, alpha=alpha, steer_vec=steer_vec, scale=scale,
                              probe_rows=probe_rows, out=out, span_mass=span_mass, status=status,
                              max_seq_len=max_seq_len)
        nbytes = self.workspace_bytes(p, 2 if (is_decode and mixed_half) else is_decode)
        ws = None
        if nbytes:
            ws = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
            p.workspace = ws.data_ptr()
            p.workspace_bytes = nbytes
        keep += [q, k_cache, v_cache, block_table, seq_lens, cu_q_lens, spans, steer_vec, status, ws]
        return HookAttnPlan(self, is_decode, p, out, span_mass, keep)

    def mixed_plan(self, prefill_kw: dict, decode_kw: dict) -> "HookAttnMixedPlan":
        """A step with a decode batch and prefill chunks (``hook_attn_mixed``): marshals both halves once."""
        return HookAttnMixedPlan(self, self.plan(False, **prefill_kw), self.plan(True, mixed_half=True, **decode_kw))

    def hook_attn_mixed(self, prefill_kw: dict, decode_kw: dict):
        """Returns ``((out, span_mass) of the prefill half, (out, span_mass) of the decode half)``."""
        pl = self.mixed_plan(prefill_kw, decode_kw)
        pl.run()
        return (pl.prefill.out, pl.prefill.span_mass), (pl.decode.out, pl.decode.span_mass)

    def hook_attn_prefill(self, **kw):
        """Prefill / chunked prefill.  Returns ``(out, span_mass)``."""
        pl = self.plan(False, **kw)
        pl.run()
        return pl.out, pl.span_mass

    def hook_attn_decode(self, **kw):
        """Decode (one query row per sequence).  Returns ``(out, span_mass)``."""
        pl = self.plan(True, **kw)
        pl.run()
        return pl.out, pl.span_mass


class HookAttnPlan:
    """A marshalled call: ``run()`` enqueues it on the current (or given) CUDA stream."""

    def __init__(self, eng: HookAttn, is_decode: bool, params: HookAttnParams, out, span_mass, keep):
        self.eng, self.is_decode, self.params = eng, is_decode, params
        self.out, self.span_mass, self._keep = out, span_mass, keep
        self._fn = eng._lib.hook_attn_decode if is_decode else eng._lib.hook_attn_prefill
        self._ref = ctypes.byref(params)

    def run(self, stream: Optional[int] = None) -> None:
        if stream is None:
            stream = torch.cuda.current_stream(self.eng.device).cuda_stream
        rc = int(self._fn(self.eng._h, self._ref, ctypes.c_void_p(stream)))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_attn_decode" if self.is_decode else "hook_attn_prefill")


class HookAttnMixedPlan:
    """The two marshalled halves of a mixed step; ``run()`` issues them with one ``hook_attn_mixed`` call."""

    def __init__(self, eng: HookAttn, prefill: HookAttnPlan, decode: HookAttnPlan):
        self.eng, self.prefill, self.decode = eng, prefill, decode

    def run(self, stream: Optional[int] = None) -> None:
        if stream is None:
            stream = torch.cuda.current_stream(self.eng.device).cuda_stream
        rc = int(self.eng._lib.hook_attn_mixed(self.eng._h, self.prefill._ref, self.decode._ref, ctypes.c_void_p(stream)))
        if rc != HOOK_ATTN_OK:
            raise HookAttnError(rc, "hook_attn_mixed")


def case_to_device(case, device="cuda") -> dict:
    """Keyword arguments for :meth:`HookAttn.hook_attn_prefill` / ``hook_attn_decode`` from an
    input-generator case (device copies of the tensors; host copies of head_mask / alpha)."""
    dev = torch.device(device)
    kw = dict(q=case.q.to(dev), k_cache=case.k_cache.to(dev), v_cache=case.v_cache.to(dev),
              block_table=case.block_table.to(dev), seq_lens=case.seq_lens.to(dev),
              scale=case.scale, probe_rows=case.probe_rows)
    if not case.is_decode:
        kw["cu_q_lens"] = case.cu_q_lens.to(dev)
    if case.spans is not None:
        kw["spans"] = case.spans.to(dev)
    if case.steer_vec is not None:
        kw["steer_vec"] = case.steer_vec.to(dev)
    if case.head_mask is not None:
        kw["head_mask"] = case.head_mask
    if case.alpha is not None:
        kw["alpha"] = case.alpha
    return kw
