"""Fused chunked KL distillation loss for B200 (sm_100a).

``inputs`` holds the seeded synthetic input generators; ``binding`` is the thin
ctypes layer over the C-ABI library built from ``csrc/``; ``autograd`` wraps the
two calls as a ``torch.autograd.Function`` (``fused_chunked_kl``, ``feature_loss``). Importing the package
does not load the library; calling into ``binding`` does, and fails loudly when
the library has not been built.
"""
__all__ = ["inputs", "binding", "autograd"]
