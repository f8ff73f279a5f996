"""Randomised stress of every entry point of the library against the oracles: integer-valued inputs, so every result
must match bit for bit; shapes, layouts, dtypes, alignments, pitches, batch / group counts and convolution geometries
are drawn from a seeded generator.  The committed test runs a short, fixed-seed slice; longer runs with other seeds
(`python -m tests.test_fuzz_gpu SEED SECONDS`) were used during development."""
import dataclasses
import os
import sys
import time

import numpy as np
import pytest

from oracle import conv_oracle as cvo
from oracle import gemm_oracle as orc
from paper_2605_28213_b200 import inputs as gen
from paper_2605_28213_b200 import npart
from tests import parity as P

pytestmark = pytest.mark.gpu


def run(seed: int, budget: float, big: bool = False):
    import torch
    from paper_2605_28213_b200 import binding as kb
    rng = np.random.default_rng(seed)
    t0 = time.time()
    n = {"gemm": 0, "batched": 0, "grouped": 0, "conv": 0, "mdst": 0, "plan": 0}

    def rdim(lo, hi):
        if big and hi >= 300:
            lo = max(lo, hi // 6)
        return int(np.exp(rng.uniform(np.log(lo), np.log(hi))))

    def check(case, vals, bits, what):
        C_ref, S = P.oracle_rows(case, np.arange(case.M))
        P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=what)

    while time.time() - t0 < budget:
        kind = rng.choice(["gemm", "gemm", "batched", "grouped", "conv", "mdst", "plan"])
        col, bf = bool(rng.integers(2)), bool(rng.integers(2))
        if True:
            if kind in ("gemm", "plan"):
                M, N, K = rdim(1, 3000), rdim(1, 3000), rdim(1, 4000)
                if M * N * K > 3e9: continue
                al = bool(rng.integers(2))
                r8 = (lambda v: (v + 7) // 8 * 8) if al else (lambda v: v + int(rng.integers(0, 3)))
                case = gen.make_case(M, N, K, seed=int(rng.integers(1 << 30)), dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf,
                                     lda=r8(K), ldb=r8(K if col else N), ldc=r8(N), name=f"fz{M}x{N}x{K}")
                dev = P.DeviceCase(case, *( (0,0,0) if al else tuple(int(v) for v in rng.integers(0, 2, 3))))
                with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
                    if kind == "plan":
                        plans = g.plan_candidates(dev.a.ptr, dev.b.ptr, dev.c.ptr, M, N, K, case.lda, case.ldb, case.ldc)
                        pl = plans[int(rng.integers(len(plans)))]
                        g.set_plan(pl, dev.a.ptr, dev.b.ptr, dev.c.ptr, M, N, K, case.lda, case.ldb, case.ldc)
                        v = 4
                    else:
                        v = int(rng.choice([4, 4, 4, 3, 5, 2, 1])); pl = None
                    dev.run(g, v)
                    vals, bits = dev.result()
                check(case, vals, bits, f"{kind} {case.name} col={col} bf={bf} v={v} al={al} plan={pl}")
            elif kind == "batched":
                b, M, N, K = rdim(1, 40), rdim(1, 700), rdim(8, 900), rdim(8, 600)
                al = bool(rng.integers(4))
                if al: N, K = (N + 7) // 8 * 8, (K + 7) // 8 * 8
                cases = [gen.make_case(M, N, K, seed=int(rng.integers(1 << 30)), dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf, name=f"fzb{i}") for i in range(b)]
                gap = [int(x) * (8 if al else 1) for x in rng.integers(0, 3, 3)]
                sa, sb, sc = M * K + gap[0], cases[0].B.size + gap[1], M * N + gap[2]
                A = np.full(sa * b, 0x7FC0, np.uint16); B = np.full(sb * b, 0x7FC0, np.uint16)
                for i, c in enumerate(cases):
                    A[i * sa:i * sa + M * K] = c.A.reshape(-1); B[i * sb:i * sb + c.B.size] = c.B.reshape(-1)
                a = P.DeviceBuffer(A.size * 2).upload(A); bb = P.DeviceBuffer(B.size * 2).upload(B)
                celt = 2 if bf else 4; cbuf = P.DeviceBuffer(sc * b * celt)
                with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
                    g.run_batched(b, a.ptr, bb.ptr, cbuf.ptr, M, N, K, K, K if col else N, N, sa, sb, sc, 4)
                    torch.cuda.synchronize(); assert g.device_status()[0] == 0
                assert cbuf.guards_intact()
                flat = cbuf.download().view(np.uint16 if bf else np.uint32)
                for i, c in enumerate(cases):
                    bits = flat[i * sc:i * sc + M * N].reshape(M, N)
                    vals = gen.bf16_bits_to_f32(bits) if bf else bits.view(np.float32)
                    check(c, vals, bits, f"batched b={b} {M}x{N}x{K} col={col} bf={bf} i={i} al={al}")
            elif kind == "grouped":
                G = rdim(1, 12)
                cases = []
                for i in range(G):
                    M, N, K = rdim(1, 1200), rdim(8, 1500) // 8 * 8, rdim(8, 700) // 8 * 8
                    cases.append(gen.make_case(M, max(N, 8), max(K, 8), seed=int(rng.integers(1 << 30)), dist_a="integer", dist_b="integer", b_col_major=col, c_bf16=bf, name=f"fzg{i}"))
                devs = [P.DeviceCase(c) for c in cases]
                with kb.Gemm(0, b_col_major=col, c_bf16=bf) as g:
                    g.run_grouped([d.a.ptr for d in devs], [d.b.ptr for d in devs], [d.c.ptr for d in devs], [c.M for c in cases], [c.N for c in cases],
                                  [c.K for c in cases], [c.lda for c in cases], [c.ldb for c in cases], [c.ldc for c in cases], 4)
                    torch.cuda.synchronize(); assert g.device_status()[0] == 0
                for c, d in zip(cases, devs):
                    vals, bits = d.result(); check(c, vals, bits, f"grouped G={G} {c.M}x{c.N}x{c.K} col={col} bf={bf}")
            elif kind == "conv":
                N_, H, W = rdim(1, 5), rdim(1, 40), rdim(1, 40)
                C = int(rng.choice([64, 128, 8, 16, 24, 5, 3])); F = rdim(1, 300)
                R, S = int(rng.integers(1, 6)), int(rng.integers(1, 6))
                pad = (int(rng.integers(0, 3)), int(rng.integers(0, 3))); stride = (1, 1) if rng.integers(3) else (int(rng.integers(1, 4)), int(rng.integers(1, 4)))
                if H + 2 * pad[0] < R or W + 2 * pad[1] < S: continue
                c = gen.make_conv_case(N_, H, W, C, F, R, S, seed=int(rng.integers(1 << 30)), pad=pad, stride=stride, dist="integer", y_f16=bf)
                yelt = 2 if bf else 4
                x = P.DeviceBuffer(c.x.size * 2).upload(c.x); w = P.DeviceBuffer(c.w.size * 2).upload(c.w)
                nout = c.N * c.P * c.Q * c.F; y = P.DeviceBuffer(max(nout * yelt, 4))
                with kb.Conv2d(0, y_f16=bf) as conv:
                    conv.run(x.ptr, w.ptr, y.ptr, c.N, c.H, c.W, c.C, c.F, c.R, c.S, c.pad, c.stride, 4)
                    torch.cuda.synchronize(); assert conv.device_status()[0] == 0
                assert y.guards_intact() and x.guards_intact() and w.guards_intact()
                y_ref, _ = cvo.conv2d(c.x, c.w, c.pad, c.stride)
                raw = y.download()[:nout * yelt]
                if bf: ok = np.array_equal(raw.view(np.uint16).reshape(y_ref.shape), cvo.round_to_f16(y_ref))
                else: ok = np.array_equal(raw.view(np.float32).reshape(y_ref.shape).astype(np.float64), y_ref)
                assert ok, f"conv {c.name} pad={pad} stride={stride} f16={bf}"
            elif kind == "mdst":
                M, N, K, world = rdim(1, 1500), rdim(8, 3000), rdim(8, 500) // 8 * 8 + 8, int(rng.integers(1, 6))
                case = gen.make_case(M, N, K, seed=int(rng.integers(1 << 30)), dist_a="integer", dist_b="integer", c_bf16=bf, name=f"fzm{M}x{N}x{K}")
                celt = 2 if bf else 4
                a = P.DeviceBuffer(case.A.size * 2).upload(case.A)
                cs = [P.DeviceBuffer(M * N * celt) for _ in range(world)]
                with kb.Gemm(0, c_bf16=bf) as g:
                    for r in range(world):
                        part = npart.NPartitionedGemm(g, world, r, N, [c.ptr for c in cs], N)
                        if part.n_local == 0: continue
                        Bs = np.ascontiguousarray(case.B[:, part.n0:part.n1]); b = P.DeviceBuffer(Bs.size * 2).upload(Bs)
                        part.run(a.ptr, b.ptr, M, K, K, part.n_local, 4); torch.cuda.synchronize(); assert g.device_status()[0] == 0
                C_ref, S = P.oracle_rows(case, np.arange(M))
                for c in cs:
                    assert c.guards_intact()
                    bits = c.download().view(np.uint16 if bf else np.uint32).reshape(M, N)
                    vals = gen.bf16_bits_to_f32(bits) if bf else bits.view(np.float32)
                    P.assert_matches_oracle(case, vals, bits, C_ref, S, exact=True, what=f"mdst {M}x{N}x{K} world={world} bf={bf}")
            n[kind] += 1
    return n


def test_short_fixed_seed_slice():
    counts = run(seed=7, budget=20.0)
    assert all(v > 0 for v in counts.values()), counts
    counts = run(seed=8, budget=15.0, big=True)
    assert sum(counts.values()) > 20, counts


if __name__ == "__main__":
    print(run(int(sys.argv[1]), float(sys.argv[2]), big=bool(int(os.environ.get("BIG", "0")))))
