"""CPU oracle for group-wise Pyramid Vector Quantization.

Test infrastructure only: a slow, plain reference written from the paper.
It shares no code with the CUDA library and the library never imports it.
"""
