"""Fused alpha-entmax / ASEntmax attention for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libentmax_attn.so`` (sources under ``csrc/``, declarations in
``include/entmax_attn.h``) plus the thin ctypes binding in :mod:`.binding` (and :mod:`.autograd`, the same calls
as a ``torch.autograd.Function``).  Importing this package
does not load the CUDA library; :mod:`.binding` does, and fails loudly if it is missing.
"""
__all__ = ["inputs"]
