"""B200-native CNN training-step library (per-replica step of Algorithm 1).

``paper_2503_23186_b200.binding`` is the ctypes layer over ``libb2c.so`` (the C-ABI in
``include/b2c.h``); ``paper_2503_23186_b200.workloads`` builds the seeded synthetic inputs.
Importing the package does not load the CUDA library; ``binding.lib()`` does and raises if
the library has not been built.
"""
