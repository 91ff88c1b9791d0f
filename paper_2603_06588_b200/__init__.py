"""Hooked paged attention for B200 (sm_100a): causal GQA attention over a paged KV cache
that also returns the attention mass on configured key spans (passive probe) and applies
a per-head steering add (active programming).  The compute lives in the CUDA library
``libhook_attn.so``; this package only marshals arguments."""
from . import inputs  # noqa: F401

__all__ = ["inputs"]
