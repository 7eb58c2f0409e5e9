"""B200-native execution-free CUTLASS kernel selection: featurize -> score -> segmented top-k.

`binding` is the ctypes front end of the C ABI in include/ks.h (needs the built libks.so);
`workloads` holds the seeded synthetic inputs; `build` compiles the library with nvcc.
"""
