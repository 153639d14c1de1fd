"""B200-native (sm_100a) decode-attention hot path of Hyper-Parallel Decoding.

``synth``    seeded synthetic inputs (no method arithmetic)
``binding``  thin ctypes binding of the C-ABI library ``libhpd.so`` (argument marshalling only)
``build``    compiles the CUDA sources in-tree with nvcc

Importing the package loads nothing; the CUDA library is opened on first use and its
absence is an error (there is no CPU fallback).
"""
