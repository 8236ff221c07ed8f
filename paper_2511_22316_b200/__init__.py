"""B200-native W4A4 linear hot path of SingleQuant (rotation + INT4 quantisation + INT4 GEMM).

`workloads` (seeded synthetic inputs) imports without CUDA; `binding` loads the C-ABI shared
library and raises if it is missing.
"""
