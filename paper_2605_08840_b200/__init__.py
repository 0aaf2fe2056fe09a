"""B200-native (sm_100a) implementation of the ReST-KV eviction-scoring hot path.

`inputs`   seeded synthetic workloads (no arithmetic of the method)
`binding`  thin ctypes binding of the C-ABI library `librestkv.so` (argument marshalling
           only; every step of the path runs in the CUDA kernels)
`build`    compiles the CUDA sources in `csrc/` for sm_100a with nvcc

There is no CPU fallback: calling into `binding` without the compiled library raises.
"""
__all__ = ["inputs", "binding", "build"]
