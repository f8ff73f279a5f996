"""B200-native bf16 GEMM lineage (C = A.B, fp32 accumulation) behind a C ABI.

``inputs``  - seeded synthetic problem generator (no GEMM arithmetic).
``binding`` - ctypes face of ``libklineage_gemm.so``; importing it fails loudly
              when the CUDA library has not been built.  There is no CPU path.
``build``   - compiles the CUDA library in-tree for sm_100a.
"""
__all__ = ["inputs", "binding", "build"]
