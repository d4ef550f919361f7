"""B200-native batched speculative-Jacobi rollout rounds (HB-SJD) behind a C ABI.

`binding` is the ctypes front end of the CUDA library, `synth` the seeded synthetic workloads,
`build` compiles the library in-tree.  Importing the package loads nothing."""
