"""B200-native FastMTP draft / verify hot path: hand-written sm_100a CUDA kernels behind a
C ABI (libfastmtp.so), with a thin ctypes binding in `paper_2509_18362_b200.binding`.

Importing the package loads nothing heavy; `binding` loads the shared library and raises if
it is missing (there is no CPU fallback).
"""
