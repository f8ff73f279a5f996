"""Host logic of the column-partitioned multi-GPU GEMM: the slice arithmetic, and two gloo ranks on CPU that
partition a problem with it, compute their slices with the oracle and assemble C (the exchange the fused epilogue
replaces on GPUs)."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def test_column_slices_cover_disjointly_and_stay_aligned():
    from paper_2605_28213_b200 import npart
    for N in (0, 1, 7, 8, 9, 64, 1000, 1001, 4096, 8192, 12345):
        for world in (1, 2, 3, 4, 8):
            for q in (1, 8, 64):
                sl = npart.slices(N, world, q)
                assert sl[0][0] == 0 and sl[-1][1] == N
                for (a0, a1), (b0, b1) in zip(sl, sl[1:]):
                    assert a1 == b0 and a0 <= a1
                for a0, a1 in sl:
                    assert a0 % q == 0 or a0 == N
                widths = [a1 - a0 for a0, a1 in sl]
                assert max(widths) - min(widths) <= 2 * q or N < world * q
    with pytest.raises(ValueError):
        npart.column_slice(10, 2, 2)
    with pytest.raises(ValueError):
        npart.column_slice(10, 0, 0)


def test_destinations_point_at_the_ranks_slice_in_every_c():
    from paper_2605_28213_b200 import npart

    class FakeGemm:
        c_bf16 = True

        def run_multi_dst(self, A, B, Cs, M, N, K, lda, ldb, ldcs, variant, stream):
            self.call = (A, B, list(Cs), M, N, K, lda, ldb, list(ldcs), variant)

    g = FakeGemm()
    bases = [0x10000000, 0x20000000, 0x30000000]
    p = npart.NPartitionedGemm(g, 3, 1, N=1000, c_ptrs=bases, ldc=1008)
    assert (p.n0, p.n1) == npart.column_slice(1000, 3, 1) and p.n0 % 8 == 0
    p.run(0xA, 0xB, M=64, K=128, lda=128, ldb=p.n_local)
    A, B, Cs, M, N, K, lda, ldb, ldcs, variant = g.call
    assert Cs == [b + p.n0 * 2 for b in bases] and N == p.n_local and ldcs == [1008] * 3 and variant == 4
    g.c_bf16 = False
    p = npart.NPartitionedGemm(g, 3, 2, N=1000, c_ptrs=bases, ldc=1000)
    assert p.dst == [b + p.n0 * 4 for b in bases]
    # an empty slice launches nothing
    g.call = None
    p = npart.NPartitionedGemm(g, 8, 0, N=8, c_ptrs=[0] * 8, ldc=8)      # one 8-column unit: it goes to the last rank
    assert p.n_local == 0
    p.run(0xA, 0xB, M=4, K=4, lda=4, ldb=1)
    assert g.call is None


WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["KL_ROOT"])
    import numpy as np, torch, torch.distributed as dist
    from paper_2605_28213_b200 import inputs as gen, npart
    from oracle import gemm_oracle as orc
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    M, N, K = 37, 203, 64
    case = gen.make_case(M, N, K, seed=5, dist_a="integer", dist_b="integer", name="npart")
    n0, n1 = npart.column_slice(N, world, rank)
    B_slice = np.ascontiguousarray(case.B[:, n0:n1])
    C_slice, _ = orc.gemm(M, n1 - n0, K, case.A, case.lda, B_slice, n1 - n0, False)
    full = torch.zeros(M, N, dtype=torch.float64)
    full[:, n0:n1] = torch.from_numpy(np.asarray(C_slice))
    dist.all_reduce(full)                      # slices are disjoint: the sum assembles C on every rank
    C_ref, _ = orc.gemm(M, N, K, case.A, case.lda, case.B, case.ldb, False)
    ok = bool(np.array_equal(full.numpy(), np.asarray(C_ref)))
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(os.environ["KL_OUT"], f"rank{rank}.json"), "w").write(json.dumps({"ok": ok, "slice": [n0, n1]}))
""")


def test_two_gloo_ranks_assemble_c_from_their_column_slices(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, KL_ROOT=str(ROOT), KL_OUT=str(tmp_path))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    res = [json.loads((tmp_path / f"rank{k}.json").read_text()) for k in range(2)]
    assert all(x["ok"] for x in res)
    assert res[0]["slice"][0] == 0 and res[0]["slice"][1] == res[1]["slice"][0] and res[1]["slice"][1] == 203


DRIVER_WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["KL_ROOT"])
    import numpy as np, torch.distributed as dist
    from paper_2605_28213_b200 import inputs as gen, npart
    from oracle import gemm_oracle as orc
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    out = os.environ["KL_OUT"]
    M, N, K, ldc = 37, 203, 64, 208
    case = gen.make_case(M, N, K, seed=5, dist_a="integer", dist_b="integer", name="npart")
    # every rank's "C" is a file that all ranks can map; its "address" is (rank + 1) << 40
    mine = np.lib.format.open_memmap(os.path.join(out, f"c{rank}.npy"), mode="w+", dtype=np.float32, shape=(M, ldc))
    mine[:] = -1.0
    mine.flush()
    ptrs = npart.exchange((rank + 1) << 40, world)            # the rendezvous: everybody learns everybody's address
    dist.barrier()

    class FileGemm:                                            # stand-in for the launch: stores the slice to every C
        c_bf16 = False
        def run_multi_dst(self, A, B, Cs, M_, N_, K_, lda, ldb, ldcs, variant, stream):
            C_slice, _ = orc.gemm(M_, N_, K_, A, lda, B, ldb, False)
            for dst, ld in zip(Cs, ldcs):
                r, off = (dst >> 40) - 1, (dst & ((1 << 40) - 1)) // 4
                tgt = np.load(os.path.join(out, f"c{r}.npy"), mmap_mode="r+")
                assert ld == ldc and off % 1 == 0
                tgt[:, off:off + N_] = np.asarray(C_slice, dtype=np.float32)
                tgt.flush()

    part = npart.NPartitionedGemm(FileGemm(), world, rank, N, ptrs, ldc)
    B_slice = np.ascontiguousarray(case.B[:, part.n0:part.n1])
    npart.partitioned_step(part, case.A, B_slice, M, K, case.lda, part.n_local)
    dist.barrier()                                             # a step ends when every rank's stores have landed
    got = np.load(os.path.join(out, f"c{rank}.npy"), mmap_mode="r")
    C_ref, _ = orc.gemm(M, N, K, case.A, case.lda, case.B, case.ldb, False)
    ok = bool(np.array_equal(np.asarray(got[:, :N], dtype=np.float64), np.asarray(C_ref))) and bool(np.all(got[:, N:] == -1.0))
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(out, f"drv{rank}.json"), "w").write(json.dumps({"ok": ok, "ptrs": ptrs, "dst": part.dst}))
""")


def test_two_gloo_ranks_drive_the_fused_all_gather_with_a_stand_in_launch(tmp_path):
    """The multi-rank driver's host logic: address exchange over the process group, slice table, every rank's launch
    writing its slice into every rank's C, and each rank finding the whole product in its own C afterwards."""
    script = tmp_path / "driver.py"
    script.write_text(DRIVER_WORKER)
    env = dict(os.environ, KL_ROOT=str(ROOT), KL_OUT=str(tmp_path))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    res = [json.loads((tmp_path / f"drv{k}.json").read_text()) for k in range(2)]
    assert all(x["ok"] for x in res)
    assert res[0]["ptrs"] == res[1]["ptrs"] == [1 << 40, 2 << 40]
    assert res[1]["dst"] == [p + 104 * 4 for p in res[1]["ptrs"]]          # rank 1's slice starts at column 104
