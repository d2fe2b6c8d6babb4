"""B200-native composed-prefill hot path (gather, RoPE shift, partial-prefill attention).

`workloads` is importable on any machine; `binding` loads the CUDA library and
fails loudly when it is missing (there is no CPU fallback).
"""
__all__ = ["workloads", "binding"]
