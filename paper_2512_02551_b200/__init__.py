"""B200-native half-precision GEMM (C = A * B^T, fp16 in, fp32 accumulate, fp16 out).

``paper_2512_02551_b200.hgemm`` is the thin ctypes binding of the C-ABI library built
from ``csrc/``; ``paper_2512_02551_b200.inputs`` draws the seeded synthetic workloads.
"""
__all__ = ["hgemm", "inputs", "build"]
