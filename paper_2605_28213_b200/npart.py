"""Column-partitioned multi-GPU GEMM with the all-gather fused into the epilogue (argument marshalling only).

Every rank holds all of A and the column slice ``B[:, n0:n1]`` of the weights, multiplies them with the tcgen05 rung and
lets the kernel's epilogue store the result slice into EVERY rank's full-width C (``klineage_gemm_run_multi_dst``): no
operand crosses NVLink, no collective follows, the only traffic is the result leaving through stores to peer memory.
The paper describes no multi-GPU design; this is the partitioning the GEMM admits without any exchange during compute.

The rendezvous that makes a rank's C addressable by its peers is plumbing and stays outside the C library, which takes
plain pointers: ``SharedC`` below does it with ``torch.distributed`` (symmetric memory, else CUDA IPC handles passed
over the process group), ``exchange`` is the underlying all-gather of Python objects, and ``partitioned_step`` is one
step of a rank (launch, nothing else: the caller owns barriers and timing).  On one GPU the "ranks" may simply be
different buffers.  The rendezvous has run on CPU ranks only (gloo, with a stand-in for the launch): this build had
one GPU per run.
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


def exchange(obj, world: int, group=None) -> list:
    """Every rank's ``obj`` in rank order (``torch.distributed.all_gather_object``); ``[obj]`` for one rank."""
    if world <= 1:
        return [obj]
    import torch.distributed as dist
    out = [None] * world
    dist.all_gather_object(out, obj, group=group)
    return out


class SharedC:
    """This rank's full-width C plus the address of every rank's C as seen from this GPU.

    how="symm": the buffer comes from ``torch.distributed._symmetric_memory`` and its rendezvous yields the peers'
    mapped addresses.  how="ipc": an ordinary CUDA tensor whose storage is exported as a CUDA IPC handle, gathered
    over the process group and opened on every peer (what ``torch.multiprocessing`` does for shared CUDA tensors).
    how="auto" tries the first and falls back to the second.  Peers are only ever STORED to through these
    addresses (the kernel's epilogue); nothing is loaded from a peer.
    """

    def __init__(self, M: int, ldc: int, dtype, device, world: int, rank: int, group=None, how: str = "auto"):
        import torch
        self.world, self.rank = int(world), int(rank)
        self._keep = []
        self.how = "local"
        if world <= 1:
            self.local = torch.empty((M, ldc), dtype=dtype, device=device)
            self.ptrs = [self.local.data_ptr()]
            return
        import torch.distributed as dist
        group = group if group is not None else dist.group.WORLD
        if how in ("auto", "symm"):
            try:
                import torch.distributed._symmetric_memory as symm
                self.local = symm.empty((M, ldc), dtype=dtype, device=device)
                hdl = symm.rendezvous(self.local, group)
                self.ptrs = [int(p) for p in hdl.buffer_ptrs]
                self._keep.append(hdl)
                self.how = "symm"
                return
            except Exception:
                if how == "symm":
                    raise
        self.local = torch.empty((M, ldc), dtype=dtype, device=device)
        info = self.local.untyped_storage()._share_cuda_()
        offset = self.local.storage_offset() * self.local.element_size()
        infos = exchange((info, offset), world, group)
        self.ptrs = []
        for r, (peer_info, peer_off) in enumerate(infos):
            if r == rank:
                self.ptrs.append(self.local.data_ptr())
                continue
            st = torch.UntypedStorage._new_shared_cuda(*peer_info)
            self._keep.append(st)
            self.ptrs.append(st.data_ptr() + peer_off)
        self.how = "ipc"


def partitioned_step(part: "NPartitionedGemm", A, B_slice, M: int, K: int, lda: int, ldb: int, variant: int = 4,
                     stream=None) -> None:
    """One step of this rank: its column slice of A . B, stored by the epilogue into every rank's C."""
    part.run(A, B_slice, M, K, lda, ldb, variant, stream)
