"""B200-native fused int4 KV-cache quantizer (SRFT + lambda + per-group abs-max + nibble pack).

``paper_2605_05699_b200.binding`` is the thin ctypes layer over the C-ABI
library ``libkvq.so`` (see ``include/kvq.h``); ``workloads`` holds the seeded
synthetic input recipes.  Nothing here computes the method on the CPU: every
step of the path runs in the CUDA kernels, and the binding raises if the
library has not been built.
"""
