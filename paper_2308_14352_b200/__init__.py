"""B200-native sparse-MoE layer forward on per-expert INT2/INT4/INT8 packed weights.

The compute lives in a C-ABI CUDA library (``csrc/``, declared in ``include/emoe.h``);
``binding`` is the thin ctypes layer over it and ``inputs`` holds the seeded synthetic
workloads.  The library is loaded on first use and there is no CPU fallback: without the
built ``libemoe.so`` every call raises.
"""
