"""PIVOT group-shared indexer for B200 (sm_100a): CUDA kernels behind a C ABI, with a thin
ctypes binding.  `inputs` draws the seeded synthetic tensors used by tests and benchmarks."""
