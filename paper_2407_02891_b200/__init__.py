"""B200-native BCQ (binary-coding-quantised) GEMV / small-batch GEMM for GPTQT inference.

`paper_2407_02891_b200.binding` is the ctypes binding of the C-ABI library declared in
`include/bcq.h`; `paper_2407_02891_b200.synth` generates the seeded synthetic inputs.
Nothing is loaded at import time; the binding raises if the CUDA library is missing.
"""
