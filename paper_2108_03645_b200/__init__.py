"""ONES evolutionary batch-size search on B200: CUDA kernels behind a C ABI.

``inputs`` (seeded synthetic workloads) imports without the CUDA extension;
everything else needs ``libones.so`` and raises if it is missing.
"""
__all__ = ["inputs", "binding", "build"]
