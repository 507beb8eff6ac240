"""B200-native imitation-step hot path (reference lookup + FK, observation,
reward, termination/reset, policy forward) behind a C-ABI CUDA library.

`workloads` holds the seeded synthetic input generators; `binding` is the thin
ctypes layer over the CUDA library (loaded on first use, never at import);
`rollout` fills time-major rollout storage through those calls.
"""
__all__ = ["workloads", "binding", "build", "rollout"]
