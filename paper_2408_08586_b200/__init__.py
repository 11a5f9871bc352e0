"""B200 (sm_100a) library for the data-parallel hot path of the Rubick scheduler (arXiv 2408.08586).

    build       compiles csrc/*.cu into librubick.so (nvcc)
    binding     ctypes binding of include/rubick.h; device buffers are torch CUDA tensors
    workloads   seeded synthetic jobs, clusters and resource grids
    events      event-driven harness: one full scheduling round per job arrival / completion

Importing the package loads nothing native; `binding.lib()` raises if the library is not built.
"""
