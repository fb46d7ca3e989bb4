"""B200-native WASH population operators (weight shuffle, PAPA EMA, final average).

`binding` mirrors the C ABI of libwash.so (include/wash.h); `workloads` holds seeded
synthetic inputs; `build` compiles the library in-tree for sm_100a.
"""
