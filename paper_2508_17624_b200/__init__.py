"""B200-native adapter-aware MoE layer forward of ExpertWeave (arXiv 2508.17624).

`binding` marshals calls into libexpertweave.so (hand-written CUDA for sm_100a behind a C ABI);
`workloads` draws the seeded synthetic inputs; `build` compiles the library in-tree.
"""
