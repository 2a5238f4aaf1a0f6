"""B200-native batch codec and longest-cached-prefix probe for an LSM-backed KV-cache store.

``lsmkv``  -- ctypes binding of the CUDA library (loaded lazily; fails loudly when missing)
``synth``  -- seeded synthetic workloads
``build``  -- nvcc build of the library for sm_100a
"""
__all__ = ["lsmkv", "synth", "build"]
