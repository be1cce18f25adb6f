"""B200-native (sm_100a) ISOPO per-linear-layer path behind a C ABI (libisopo.so).

`paper_2512_23353_b200.binding` loads the library (and raises if it has not been built);
`paper_2512_23353_b200.workloads` draws seeded synthetic microbatches; `paper_2512_23353_b200.build`
compiles the CUDA sources in-tree.
"""
