"""B200-native SurfaceLogicKV prefill KV-cache compression (budgets, window scores, top-k, gather).

The compute lives in the CUDA library `libslkv.so` (C ABI declared in include/slkv.h); `binding` is the
thin ctypes layer over it and `synth` draws the seeded synthetic inputs.  Importing the package loads
nothing; `binding.lib()` loads the shared library and raises if it has not been built.
"""
__all__ = ["binding", "synth"]
