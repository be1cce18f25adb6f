"""B200-native (sm_100a) ISOPO per-linear-layer path behind a C ABI (libisopo.so).

`paper_2512_23353_b200.binding` loads the library (and raises if it has not been built) and mirrors
its entry points one to one; `paper_2512_23353_b200.tp` composes them with one all-reduce of K for a
layer whose output features are split across ranks; `paper_2512_23353_b200.workloads` draws seeded
synthetic microbatches; `paper_2512_23353_b200.build` compiles the CUDA sources in-tree.
"""
