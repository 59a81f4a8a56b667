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
