"""B200-native bounded self-speculative decode step (SpecBound).

``inputs``  -- seeded synthetic workloads (no method arithmetic).
``binding`` -- thin ctypes binding of the C-ABI CUDA library (loaded on first use).
"""
