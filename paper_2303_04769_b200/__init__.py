"""B200 (sm_100a) implementation of the SMaLL layer set (arXiv 2303.04769) behind a C ABI (include/small.h).

`binding` marshals arguments to libsmall.so; `net` turns a layer list into descriptors for small_run_net.
Nothing here computes: every step of a layer runs in the CUDA kernels under csrc/.  Importing this package
does not load the library; the first use of `binding.lib()` does, and raises if it has not been built.
"""
__all__ = ["binding", "net", "build"]
