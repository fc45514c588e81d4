"""B200-native adaptive dense GEMM (fp16/bf16 in, fp32 accumulate, 16-bit out).

The product is the CUDA library behind ``include/adapt_matmul.h``; ``binding``
marshals arguments to it through ctypes, and ``synth`` draws the seeded
workloads.  Importing this package loads nothing native; the library is loaded
on first use of ``binding`` and its absence is an error, never a fallback.
"""
