"""CPU oracles of the bf16 GEMM lineage and of the fp16 Conv2d workload.  Test infrastructure only: never imported by the product."""
