"""Block-sparse fused prefill attention for NVIDIA B200 (sm_100a).

``inputs`` holds the seeded synthetic workloads; ``binding`` is the ctypes layer over the C ABI
declared in ``include/steel_attn.h``; ``build`` compiles the CUDA library in-tree.  Nothing is
loaded at import time.
"""
