"""B200-native NUQSGD codec: bucket norm, nonuniform stochastic quantizer,
Elias-recursive encoder and decode+accumulate, as CUDA kernels behind a C ABI.

`from paper_1908_06077_b200 import nuq` gives the thin ctypes binding; the
`inputs` module holds the seeded synthetic workload generators.
"""
