"""Carryover drafting round for NVIDIA B200 (sm_100a): hand-written CUDA behind a C ABI.

``synth`` (seeded synthetic inputs) imports without a GPU; ``binding`` loads the
compiled library and raises if it is missing — there is no CPU fallback.
"""
__all__ = ["synth", "binding"]
