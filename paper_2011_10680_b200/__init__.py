"""B200-native integer-only inference kernels for HAWQ-V3 (dyadic quantization).

`binding` is the ctypes layer over the CUDA library (libhq.so, built by `build`); `inputs` draws the
seeded synthetic workloads.  Importing the package does not load the library.
"""
