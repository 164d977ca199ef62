"""libgconv for B200: forward grouped 2-D convolution (fp32 NCHW) as hand-written sm_100a CUDA.

Submodules: ``gconv`` (ctypes binding of the C ABI in include/gconv.h), ``synth`` (seeded input
generators), ``workloads`` (layer tables and cost model), ``build`` (nvcc build of the library).
Importing the package loads nothing native; ``gconv`` loads the shared library on first use and
raises if it is missing.
"""
__all__ = ["gconv", "synth", "workloads", "build"]
