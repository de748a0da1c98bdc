"""B200-native MatmulAccum (bf16 x bf16 -> f32, accumulating) behind a C ABI.

``workloads`` holds the seeded input generators; ``binding`` loads the CUDA
shared library and exposes its entry points under the same names.  Nothing in
this package falls back to a CPU implementation: without the built library the
binding raises.
"""
__all__ = ["workloads", "binding"]
