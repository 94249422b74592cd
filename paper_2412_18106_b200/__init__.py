"""B200-native hybrid-batch attention meta-kernel (XY-Serve's Meta-Attention, arXiv 2412.18106).

`binding` mirrors the C-ABI of include/xy_attn.h; `workloads` draws seeded synthetic
batches; `build` compiles the CUDA library in-tree for sm_100a.
"""
