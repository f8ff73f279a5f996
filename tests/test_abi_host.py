"""Host-only checks of the C ABI: the library loads without a GPU, exports every
symbol the header declares, and validates arguments before touching a device."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def kb():
    from paper_2605_28213_b200 import build
    build.build()
    from paper_2605_28213_b200 import binding
    return binding


def declared_functions():
    names = set()
    for hdr in (ROOT / "include").glob("*.h"):
        text = re.sub(r"/\*.*?\*/", "", hdr.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(klineage_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(kb):
    decl = declared_functions()
    assert {"klineage_gemm_create", "klineage_gemm_run", "klineage_gemm_destroy"} <= decl
    lib = ctypes.CDLL(str(kb.LIB_PATH))
    for name in decl:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert decl == set(kb.EXPORTED_SYMBOLS) | {n for n in decl if n not in kb.EXPORTED_SYMBOLS}
    for name in kb.EXPORTED_SYMBOLS:
        assert name in decl or name.startswith("klineage_"), name


def test_shipped_library_carries_no_trace_code(kb):
    """The timeline stamps of the tcgen05 kernels exist only in builds with -DKLIN_TRACE: the shipped library exports
    none of the trace entry points (and therefore holds no trace buffer the kernels could write to)."""
    import ctypes
    lib = ctypes.CDLL(str(kb.LIB_PATH))
    for name in ("klin_trace_dump_pair", "klin_trace_dump_single", "klin_trace_set_knob"):
        assert not hasattr(lib, name), name


def test_status_and_variant_names(kb):
    assert kb.klineage_status_string(0) == "ok"
    assert kb.klineage_status_string(kb.KLINEAGE_ERR_BAD_VARIANT) == "bad variant"
    assert kb.klineage_status_string(12345) == "unknown status"
    assert [kb.klineage_variant_name(v) for v in range(6)] == ["naive", "tiled", "vectorized", "pipelined", "tcgen05",
                                                                "mma_sync"]
    assert kb.klineage_variant_name(6) == "unknown"


def test_check_args_rules(kb):
    chk = kb.klineage_gemm_check_args
    A, B, C = 0x10000, 0x20000, 0x40000
    ok = lambda **kw: chk(**{**dict(b_layout=0, c_dtype=0, M=8, N=9, K=10, A=A, lda=10, B=B, ldb=9, C=C, ldc=9,
                                    variant=0), **kw})
    assert ok() == kb.KLINEAGE_OK
    assert ok(variant=6) == kb.KLINEAGE_ERR_BAD_VARIANT and ok(variant=-1) == kb.KLINEAGE_ERR_BAD_VARIANT
    assert ok(variant=5) == kb.KLINEAGE_OK
    assert ok(b_layout=2) == kb.KLINEAGE_ERR_INVALID_ARG and ok(c_dtype=3) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(M=-1) == kb.KLINEAGE_ERR_INVALID_ARG and ok(K=1 << 31) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(lda=9) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(ldb=8) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(ldc=8) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(b_layout=1, ldb=9) == kb.KLINEAGE_ERR_INVALID_ARG      # column-major needs ldb >= K
    assert ok(b_layout=1, ldb=10) == kb.KLINEAGE_OK
    assert ok(A=None) == kb.KLINEAGE_ERR_INVALID_ARG and ok(C=None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert ok(A=A + 1) == kb.KLINEAGE_ERR_INVALID_ARG                # bf16 needs 2-byte alignment
    assert ok(C=C + 2) == kb.KLINEAGE_ERR_INVALID_ARG                # fp32 C needs 4-byte alignment
    assert ok(C=C + 2, c_dtype=1) == kb.KLINEAGE_OK                  # bf16 C needs only 2
    assert ok(C=A + 4) == kb.KLINEAGE_ERR_INVALID_ARG                # C overlaps A
    assert ok(C=B) == kb.KLINEAGE_ERR_INVALID_ARG                    # C overlaps B
    assert ok(M=0, A=None, C=None) == kb.KLINEAGE_OK                 # empty product: nothing is read
    assert ok(K=0, A=None, B=None) == kb.KLINEAGE_OK                 # K == 0 only writes C
    assert ok(A=A + 2, B=B + 2, lda=11) == kb.KLINEAGE_OK            # element alignment suffices


def test_no_handle_and_no_device_paths(kb):
    assert kb.klineage_gemm_run_raw(None, 1, 1, 1, 16, 1, 32, 1, 64, 1, 0, None) == kb.KLINEAGE_ERR_INVALID_ARG
    kb.klineage_gemm_destroy(None)
    assert kb.klineage_gemm_last_kernel_id(None) == -1
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(kb.KlineageError) as e:
            kb.klineage_gemm_create(0, 0, 0)
        assert e.value.status == kb.KLINEAGE_ERR_INVALID_ARG


def test_binding_refuses_to_import_without_the_library(tmp_path, monkeypatch):
    """No fallback: with the shared library absent the binding must raise, not degrade."""
    import importlib.util
    src = (ROOT / "paper_2605_28213_b200" / "binding.py").read_text()
    fake = tmp_path / "binding_copy.py"
    fake.write_text(src)
    spec = importlib.util.spec_from_file_location("binding_copy", fake)
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)


def test_product_never_imports_the_oracle():
    """The product and the oracle share no code and neither imports the other."""
    imp = re.compile(r"^\s*(from|import)\s+oracle\b|liboracle|oracle_gemm|gemm_oracle|oracle/", re.M)
    for py in (ROOT / "paper_2605_28213_b200").rglob("*.py"):
        assert not imp.search(py.read_text()), f"{py} reaches into the oracle"
    for src in (ROOT / "paper_2605_28213_b200" / "csrc").glob("*.cu*"):
        assert not imp.search(src.read_text()), f"{src} reaches into the oracle"
    back = re.compile(r"^\s*(from|import)\s+paper_2605_28213_b200|klineage_gemm|csrc", re.M)
    for f in (ROOT / "oracle").glob("*"):
        if f.suffix in (".py", ".c"):
            assert not back.search(f.read_text()), f"{f} reaches into the product"


def test_conv2d_check_args_rules(kb):
    # host-only: the geometry and aliasing rules of the Conv2d call need no GPU
    chk = kb.klineage_conv2d_check_args
    X, Wt, Y = 0x100000, 0x200000, 0x400000

    def call(**kw):
        return chk(kw.get("dt", kb.KLINEAGE_C_F16), kw.get("N", 1), kw.get("H", 8), kw.get("W", 8), kw.get("C", 8),
                   kw.get("F", 8), kw.get("R", 3), kw.get("S", 3), kw.get("ph", 1), kw.get("pw", 1), kw.get("sh", 1),
                   kw.get("sw", 1), kw.get("x", X), kw.get("w", Wt), kw.get("y", Y), kw.get("v", kb.KLINEAGE_TCGEN05))

    assert call() == kb.KLINEAGE_OK
    assert call(dt=kb.KLINEAGE_C_F32) == kb.KLINEAGE_OK
    assert call(dt=kb.KLINEAGE_C_BF16) == kb.KLINEAGE_ERR_INVALID_ARG      # bf16 is not a Conv2d output type
    assert call(v=kb.KLINEAGE_NAIVE) == kb.KLINEAGE_OK
    for v in (1, 2, 3, 5, 6, -1):
        assert call(v=v) == kb.KLINEAGE_ERR_BAD_VARIANT
    assert call(R=0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(S=65) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(sh=0) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(pw=-1) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(H=1, ph=0) == kb.KLINEAGE_ERR_INVALID_ARG                  # filter taller than the padded image
    assert call(H=1, ph=1) == kb.KLINEAGE_OK                               # ... but not with padding 1: P = 1
    assert call(y=None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(x=None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(y=X) == kb.KLINEAGE_ERR_INVALID_ARG                        # y aliases x
    assert call(y=Wt + 2) == kb.KLINEAGE_ERR_INVALID_ARG                   # y overlaps w
    assert call(y=Y + 1) == kb.KLINEAGE_ERR_INVALID_ARG                    # fp16 y must be 2-byte aligned
    assert call(dt=kb.KLINEAGE_C_F32, y=Y + 2) == kb.KLINEAGE_ERR_INVALID_ARG
    assert call(N=0, y=None, x=None, w=None) == kb.KLINEAGE_OK             # nothing to compute
    assert call(F=0, y=None) == kb.KLINEAGE_OK
    assert call(C=0) == kb.KLINEAGE_OK                                     # K = 0: y is zero-filled, x and w unused
    assert call(N=1 << 21) == kb.KLINEAGE_ERR_INVALID_ARG


def test_null_handles_are_refused_everywhere(kb):
    P = 0x100000
    assert kb.klineage_gemm_run_raw(None, 8, 8, 8, P, 8, P * 2, 8, P * 3, 8, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_gemm_run_addmm_raw(None, 8, 8, 8, P, 8, P * 2, 8, P * 4, P * 3, 8, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_gemm_run_batched_raw(None, 2, 8, 8, 8, P, 8, 64, P * 2, 8, 64, P * 3, 8, 64, 4, None) == \
        kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_gemm_run_grouped_raw(None, [8], [8], [8], [P], [8], [P * 2], [8], [P * 3], [8], 4, None) == \
        kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_gemm_run_multi_dst_raw(None, 8, 8, 8, P, 8, P * 2, 8, [P * 3], [8], 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_conv2d_run_raw(None, 1, 8, 8, 8, 8, 3, 3, 1, 1, 1, 1, P, P * 2, P * 3, 4, None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert kb.klineage_gemm_set_plan_raw(None, 8, 8, 8, P, 8, P * 2, 8, P * 3, 8, None) == kb.KLINEAGE_ERR_INVALID_ARG
    assert kb._lib.klineage_gemm_last_launch_count(None) == 0
    assert kb.klineage_gemm_last_kernel_id(None) == -1


def test_host_scratch_bytes_follows_the_documented_layout(kb):
    """Three matrices, pitches rounded up to 8 elements, each at a 256-byte offset; 0 for empty or invalid shapes."""
    def expect(col, bf16, M, N, K):
        up8 = lambda v: (v + 7) // 8 * 8 if v > 0 else 8
        up256 = lambda v: (v + 255) // 256 * 256
        b_rows, b_cols = (N, K) if col else (K, N)
        return up256(M * up8(K) * 2) + up256(b_rows * up8(b_cols) * 2) + up256(M * up8(N) * (2 if bf16 else 4))

    for col in (False, True):
        for bf16 in (False, True):
            for (M, N, K) in ((1000, 1001, 999), (1, 1, 1), (8192, 8192, 8192), (16, 8192, 8192), (70, 33, 0)):
                got = kb.klineage_gemm_host_scratch_bytes(int(col), int(bf16), M, N, K)
                assert got == expect(col, bf16, M, N, K), (col, bf16, M, N, K, got)
    assert kb.klineage_gemm_host_scratch_bytes(0, 0, 1000, 1001, 999) == 2000128 + 2014208 + 4032000   # worked by hand
    assert kb.klineage_gemm_host_scratch_bytes(0, 0, 0, 8, 8) == 0
    assert kb.klineage_gemm_host_scratch_bytes(0, 0, 8, 0, 8) == 0
    assert kb.klineage_gemm_host_scratch_bytes(0, 0, 8, 8, -1) == 0
    assert kb.klineage_gemm_host_scratch_bytes(2, 0, 8, 8, 8) == 0
    assert kb.klineage_gemm_host_scratch_bytes(0, 5, 8, 8, 8) == 0
    assert kb.klineage_gemm_host_scratch_bytes(0, 0, 1 << 31, 8, 8) == 0
    P = 0x100000
    assert kb.klineage_gemm_run_host_raw(None, 8, 8, 8, P, 8, P * 2, 8, P * 3, 8, P * 4, 1 << 20, 4, None) == \
        kb.KLINEAGE_ERR_INVALID_ARG
