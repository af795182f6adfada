"""B200-native (sm_100a) implementation of the OasisKV per-decode-step hot path.

The compute lives in a C-ABI shared library of hand-written CUDA kernels
(`csrc/`, declared in `include/oasis.h`); `binding` exposes the same calls to Python
with argument marshalling only, and `synth` draws the seeded synthetic workloads.
There is no CPU fallback: calling an operation without the built library raises.
"""
__all__ = ["binding", "synth", "build"]
