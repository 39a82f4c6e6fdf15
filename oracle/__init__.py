"""CPU oracle of the 3-D U-Net convolution path (TEST INFRASTRUCTURE).

Plain fp64 definitions used to check the CUDA library.  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the CUDA
library and its Python binding never do.
"""
