"""B200-native Speculative Jacobi Decoding hot path (arXiv 2410.01699).

  csrc/       CUDA kernels (sm_100a) and the C-ABI of include/sjd.h
  build.py    nvcc build of libsjd.so, in-tree
  binding.py  ctypes binding with the header's names (argument marshalling only)
  inputs.py   seeded synthetic workloads shaped like the paper's
  sharding.py assignment of independent sequences to ranks (no collective on the data path)

Importing this package loads nothing; `binding.lib()` loads the library and raises if it is
missing.  There is no CPU or framework fallback.
"""
