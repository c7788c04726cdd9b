"""B200-native verify + recover step of SpecSteer's Draft-Verify-Recover loop.

The product is the C-ABI CUDA library under ``csrc/`` (declared in
``include/specsteer.h``); ``binding`` marshals torch tensors into it and
``synth`` manufactures seeded inputs.  Nothing here computes on the CPU: every
call fails loudly if the CUDA library has not been built.
"""
__all__ = ["binding", "synth", "build", "sharding"]
