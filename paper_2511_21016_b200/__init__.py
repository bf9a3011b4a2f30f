"""B200-native (sm_100a) implementation of the Gated KalmaNet hot path.

``gka``   — ctypes binding of the C ABI (``gka_fwd_chunked``, ``gka_decode_step``);
``synth`` — seeded synthetic inputs;  ``build`` — nvcc build step.
Importing the package loads nothing; the CUDA library is loaded on first use and a
missing library is an error (there is no CPU fallback).
"""
