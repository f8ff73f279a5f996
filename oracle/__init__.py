"""CPU oracle for the bf16 GEMM lineage.  Test infrastructure only: never imported by the product."""
