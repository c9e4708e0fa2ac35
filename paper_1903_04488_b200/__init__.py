"""B200-native Sketched-SGD compression step (CUDA, sm_100a) behind a C-ABI library.

`from paper_1903_04488_b200 import ssgd` gives the thin binding over the library; `workloads` holds the
seeded synthetic gradient generators.
"""
