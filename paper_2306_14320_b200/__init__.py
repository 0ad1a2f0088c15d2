"""B200-native im2win: the im2win data transformation and the im2win-based convolution
(hand-written sm_100a CUDA kernels behind a C-ABI library).

``paper_2306_14320_b200.binding`` is the thin ctypes binding (it needs the built shared library and
fails loudly without it); ``paper_2306_14320_b200.workloads`` only names layer shapes and generates
seeded synthetic inputs.  Nothing is loaded at package import.
"""
