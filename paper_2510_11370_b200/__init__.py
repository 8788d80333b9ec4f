"""B200-native (sm_100a) kernels for the replayed-routing MoE layer of Rollout Routing Replay.

Sub-modules:
  r3     - thin ctypes binding over the C-ABI CUDA library (loads it on import; raises if the
           library has not been built - there is no CPU fallback)
  synth  - seeded synthetic workloads
  build  - compiles the CUDA library in-tree with nvcc for sm_100a
"""
__all__ = ["r3", "synth", "build"]
