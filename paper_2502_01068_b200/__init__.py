"""B200-native (sm_100a) FastKV token-saliency selection path: score -> select -> compact.

`binding` mirrors the C ABI of libfastkv_b200.so (include/fastkv.h); `workloads` draws the seeded
synthetic inputs; `build` compiles the library in-tree.
"""
