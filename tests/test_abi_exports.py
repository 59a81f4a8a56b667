"""CPU-only: the C-ABI library builds, loads and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "gptq2d.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gptq2d_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    from paper_2607_27042_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    syms = _declared_symbols()
    assert "gptq2d_round" in syms and "gptq2d_factor" in syms and "gptq2d_objective" in syms
    for s in syms:
        assert hasattr(lib, s), s
    from paper_2607_27042_b200 import gptq2d
    assert sorted(gptq2d.EXPORTS) == [s for s in syms]
    for s in syms:
        if s != "gptq2d_status_string":
            assert callable(getattr(gptq2d, s)), "binding lacks " + s


def test_workspace_queries_and_status_strings_need_no_gpu():
    from paper_2607_27042_b200 import gptq2d
    assert gptq2d.status_string(0) == "ok"
    assert "positive definite" in gptq2d.status_string(5)
    assert gptq2d.gptq2d_round_workspace_bytes(0, 5) == 0
    w = gptq2d.gptq2d_round_workspace_bytes(8192, 8192)
    assert 2 * 8192 * 8192 * 8 <= w < 2 * 8192 * 8192 * 8 + (1 << 20)
    assert gptq2d.gptq2d_round_workspace_bytes(100, 130) >= 2 * 128 * 256 * 8
    assert gptq2d.gptq2d_round_host_workspace_bytes(64, 64) > gptq2d.gptq2d_round_workspace_bytes(64, 64)
    assert gptq2d.gptq2d_factor_workspace_bytes(64, 256) >= 3 * 256 * 256 * 8
    assert gptq2d.gptq2d_objective_workspace_bytes(64, 256) >= 2 * 64 * 256 * 8


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_27042_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f


def test_batched_entry_argument_checks_need_no_gpu():
    """Host-side validation of the batched call: made-up (never dereferenced) device addresses."""
    import ctypes as c
    from paper_2607_27042_b200 import gptq2d as g
    lib = g._lib

    def probs(shapes):
        arr = (g.Problem * len(shapes))()
        for b, (m, n) in enumerate(shapes):
            arr[b] = g.Problem(m, n, 0x1000, n, 0x2000, m, 0x3000, n, 0x4000, n, None, 0)
        return arr

    shapes = [(64, 64), (200, 330), (1, 9)]
    arr = probs(shapes)
    total = lib.gptq2d_round_batched_workspace_bytes(3, c.cast(arr, c.c_void_p))
    # at least the padded E and C buffers of every matrix; no more than that plus bookkeeping
    bufs = sum(2 * 8 * (-(-m // 128) * 128) * (-(-n // 128) * 128) for m, n in shapes)
    assert bufs <= total < bufs + (1 << 16)
    one = [lib.gptq2d_round_batched_workspace_bytes(1, c.cast(probs([s]), c.c_void_p)) for s in shapes]
    assert total <= sum(one)
    assert lib.gptq2d_round_batched_workspace_bytes(0, c.cast(arr, c.c_void_p)) == 0
    # invalid descriptors are rejected before any CUDA call
    ws = c.c_void_p(0x100000)
    assert lib.gptq2d_round_batched(0, c.cast(arr, c.c_void_p), None, ws, 1 << 40, None, None) == 1
    assert lib.gptq2d_round_batched(3, None, None, ws, 1 << 40, None, None) == 1
    bad = probs(shapes)
    bad[1].ldx = 100                                   # leading dimension below n
    assert lib.gptq2d_round_batched(3, c.cast(bad, c.c_void_p), None, ws, 1 << 40, None, None) == 1
    bad = probs(shapes)
    bad[2].Z = None
    assert lib.gptq2d_round_batched(3, c.cast(bad, c.c_void_p), None, ws, 1 << 40, None, None) == 1
    big = probs([(g.BATCH_MAX_DIM + 1, 8)])
    assert lib.gptq2d_round_batched(1, c.cast(big, c.c_void_p), None, ws, 1 << 40, None, None) == 9
    many = probs([(8, 8)] * (g.BATCH_MAX_COUNT + 1))
    assert lib.gptq2d_round_batched(len(many), c.cast(many, c.c_void_p), None, ws, 1 << 40, None, None) == 9
    # workspace too small / missing
    assert lib.gptq2d_round_batched(3, c.cast(arr, c.c_void_p), None, ws, total - 1, None, None) == 2
    assert lib.gptq2d_round_batched(3, c.cast(arr, c.c_void_p), None, None, total, None, None) == 2


def test_batched_setup_argument_checks_need_no_gpu():
    """Host-side validation of gptq2d_factor_batched: made-up (never dereferenced) device addresses."""
    import ctypes as c
    from paper_2607_27042_b200 import gptq2d as g
    lib = g._lib

    def probs(shapes, a=0x1000):
        arr = (g.FactorProblem * len(shapes))()
        for b, (m, n) in enumerate(shapes):
            arr[b] = g.FactorProblem(m, n, a, m, 0x2000, n, 0x3000, m, 0x4000, n, None, None)
        return arr

    small = probs([(64, 64), (1, 128), (100, 7)])
    table = lib.gptq2d_factor_batched_workspace_bytes(3, c.cast(small, c.c_void_p))
    assert 0 < table <= 4096                                    # descriptors only: no blocked route needed
    mixed = probs([(64, 64), (300, 90)])
    total = lib.gptq2d_factor_batched_workspace_bytes(2, c.cast(mixed, c.c_void_p))
    assert total >= g.gptq2d_factor_workspace_bytes(300, 90)    # the blocked route's own workspace on top
    assert lib.gptq2d_factor_batched_workspace_bytes(0, c.cast(small, c.c_void_p)) == 0
    assert lib.gptq2d_factor_batched(0, c.cast(small, c.c_void_p), None, 0, None, None) == 1      # INVALID_ARG
    bad = probs([(64, 64)])
    bad[0].ldl = 10                                             # leading dimension below m
    assert lib.gptq2d_factor_batched(1, c.cast(bad, c.c_void_p), None, 0, None, None) == 1
    assert lib.gptq2d_factor_batched(3, c.cast(small, c.c_void_p), None, 0, None, None) == 2      # WORKSPACE
