"""B200-native PPOW window scoring: C-ABI CUDA library plus a thin ctypes binding.

``workloads`` (input generators) imports without the CUDA library; ``binding`` loads
``libppow.so`` on first use and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
