"""B200-native CoRun hot path: fixed-shape padded decode + isolated prefill.

``corun`` is the thin ctypes binding of the C-ABI library (csrc/); ``synth``
holds the seeded synthetic input generators.
"""
