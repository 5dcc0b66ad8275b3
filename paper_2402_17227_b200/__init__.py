"""B200-native sampled backward of a linear layer (VCAS, arXiv 2402.17227).

`inputs` draws the synthetic workloads; `binding` is the ctypes layer over the C ABI of
libvcas.so (built by `build`).  Nothing here computes on the CPU: without the compiled CUDA
library the binding raises on first use.
"""
