"""Column-partitioned multi-GPU GEMM with the all-gather fused into the epilogue (argument marshalling only).

Every rank holds all of A and the column slice ``B[:, n0:n1]`` of the weights, multiplies them with the tcgen05 rung and
lets the kernel's epilogue store the result slice into EVERY rank's full-width C (``klineage_gemm_run_multi_dst``): no
operand crosses NVLink, no collective follows, the only traffic is the result leaving through stores to peer memory.
The paper describes no multi-GPU design; this is the partitioning the GEMM admits without any exchange during compute.

The rendezvous that makes a rank's C addressable by its peers is plumbing and stays outside the library: pass the list
of per-rank C base pointers (for instance the ``buffer_ptrs`` of a ``torch.distributed._symmetric_memory`` rendezvous,
or pointers opened from CUDA IPC handles).  On one GPU the "ranks" may simply be different buffers.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def column_slice(N: int, world: int, rank: int, quantum: int = 8) -> Tuple[int, int]:
    """Half-open column range [n0, n1) of ``rank``: balanced, starts at multiples of ``quantum`` columns.

    With bf16 / fp32 elements a multiple of 8 columns keeps every slice 16-byte aligned inside an aligned C, which the
    TMA-store epilogue needs.  The last ranks may get empty slices when N < world * quantum.
    """
    if world < 1 or not 0 <= rank < world or N < 0 or quantum < 1:
        raise ValueError("bad partition arguments")
    units = -(-N // quantum)                       # ceil
    lo = (units * rank) // world * quantum
    hi = (units * (rank + 1)) // world * quantum
    return min(lo, N), min(hi, N)


def slices(N: int, world: int, quantum: int = 8) -> List[Tuple[int, int]]:
    return [column_slice(N, world, r, quantum) for r in range(world)]


class NPartitionedGemm:
    """One rank's share of ``C = A . B`` partitioned by columns over ``world`` ranks.

    gemm      a ``binding.Gemm`` handle on this rank's GPU
    c_ptrs    base device pointer of every rank's full-width M x N C (index = rank), reachable from this GPU
    ldc       pitch (elements) of those C matrices
    """

    def __init__(self, gemm, world: int, rank: int, N: int, c_ptrs: Sequence[int], ldc: int, quantum: int = 8):
        if len(c_ptrs) != world:
            raise ValueError("one C pointer per rank")
        self.gemm, self.world, self.rank, self.N, self.ldc = gemm, int(world), int(rank), int(N), int(ldc)
        self.n0, self.n1 = column_slice(N, world, rank, quantum)
        celt = 2 if gemm.c_bf16 else 4
        self.dst = [int(p) + self.n0 * celt for p in c_ptrs]      # this rank's slice inside every rank's C

    @property
    def n_local(self) -> int:
        return self.n1 - self.n0

    def run(self, A, B_slice, M: int, K: int, lda: int, ldb: int, variant: int = 4, stream=None) -> None:
        """``B_slice``: this rank's columns of B (row-major K x n_local, or column-major n_local x K)."""
        if self.n_local == 0 or M == 0:
            return
        self.gemm.run_multi_dst(A, B_slice, self.dst, M, self.n_local, K, lda, ldb, [self.ldc] * self.world, variant,
                                stream)
