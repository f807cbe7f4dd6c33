"""Lazy update (SGD with Kahan summation, arXiv 1810.05486 Algorithm 1) in dynamic
fixed-point as hand-written CUDA for B200 (sm_100a), behind a C ABI.

  binding    ctypes wrappers with the C ABI's names (kahan_sgd_init / _step / _amax ...)
  workloads  seeded synthetic parameter lists and gradients shaped like the paper's networks
  build      nvcc build of libkahan_sgd.so
"""
