"""B200-native TWA subspace step: C-ABI CUDA library plus a thin binding.

`paper_2205_13104_b200.twa` mirrors the C entry points of include/twa.h;
`paper_2205_13104_b200.inputs` draws the seeded synthetic workloads.
Importing the package does not load the CUDA library; the first call does,
and raises if the library has not been built.
"""
