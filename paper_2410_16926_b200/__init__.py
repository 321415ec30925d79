"""B200-native group-wise Pyramid Vector Quantization (encode / decode).

`paper_2410_16926_b200.pvq` is the thin binding over the C-ABI CUDA library;
`paper_2410_16926_b200.inputs` makes the seeded synthetic workloads.
Nothing is loaded at import time; the binding raises if the compiled library
is missing.
"""
