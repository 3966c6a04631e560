"""B200-native SpecPV verification hot path: CUDA kernels behind a C ABI plus a thin binding.

``binding`` loads ``lib/libspecpv.so`` (built by ``build``) and exposes the same call names as
``include/specpv.h``; ``workloads`` holds the seeded synthetic input generators.
"""
__all__ = ["binding", "build", "workloads"]
