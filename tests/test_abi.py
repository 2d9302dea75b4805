"""Host-side checks that need no GPU: the shared library loads, exports every symbol the public
header declares, and its shape arithmetic / validation behaves."""
import ctypes
import os
import re

import pytest

from paper_2506_07366_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding._lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moegps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"MOEGPS_API\s+[\w\s\*]+?\b(moegps_\w+)\s*\(", text)))


def test_header_declares_the_six_steps():
    names = declared_symbols()
    for step in ("route", "histogram", "plan", "dispatch", "expert_ffn", "combine"):
        assert f"moegps_{step}" in names
    assert len(names) >= 12


def test_library_exports_every_declared_symbol(lib):
    raw = ctypes.CDLL(binding.library_path())
    for name in declared_symbols():
        assert hasattr(raw, name), f"{name} is declared in moegps.h but not exported"
    assert set(binding.EXPORTS) == set(declared_symbols())


def test_rcap_and_workspace(lib):
    s = binding.Shape(T=256, D=512, F=1024, E=8, K=2, S=8, row_align=128)
    assert binding.rcap(s) == 256 * 2 + 8 * 127 == s.Rcap
    assert binding.workspace_bytes(s) >= (512 // 256) * 8 * 4
    s1 = binding.Shape(T=4096, D=7168, F=2048, E=256, K=8, S=288, gate_mode=1, row_align=1)
    assert binding.rcap(s1) == 4096 * 8
    assert binding.workspace_bytes(s1) >= (32768 // 256) * 256 * 4
    assert binding.workspace_bytes(s1) % 16 == 0


@pytest.mark.parametrize("bad", [
    dict(K=9, E=16, S=16), dict(K=3, E=2, S=2), dict(E=257, S=257), dict(S=7), dict(S=1025),
    dict(D=516), dict(F=1020), dict(row_align=3), dict(row_align=512), dict(T=-1), dict(gate_mode=2),
    dict(c_max=-1),
])
def test_invalid_shapes_are_rejected(lib, bad):
    base = dict(T=256, D=512, F=1024, E=8, K=2, S=8, gate_mode=0, row_align=128, c_max=0)
    base.update(bad)
    s = binding.Shape(**base)
    assert binding.rcap(s) == -1
    assert binding.workspace_bytes(s) == 0


def test_error_strings(lib):
    seen = set()
    for code in range(0, -9, -1):
        msg = binding.error_string(code)
        assert msg and msg not in seen
        seen.add(msg)
    assert "unknown" in binding.error_string(-99)


def test_null_context_is_an_error_not_a_crash(lib):
    assert lib.moegps_destroy(None) == binding.ERR_INVALID_ARG
    assert lib.moegps_histogram(None, None, None, None) == binding.ERR_INVALID_ARG
    assert lib.moegps_launch_count(None) == -1


def test_context_needs_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.Context(binding.Shape(T=8, D=64, F=64, E=2, K=1, S=2))


def test_missing_library_fails_loudly(tmp_path):
    # there is no fallback path: a missing shared library must raise, in a fresh interpreter
    import subprocess
    import sys
    code = ("import os, sys; sys.path.insert(0, %r); os.environ['MOEGPS_LIBRARY'] = %r; "
            "from paper_2506_07366_b200 import binding; binding._lib()") % (ROOT, str(tmp_path / "nope.so"))
    proc = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True)
    assert proc.returncode != 0
    assert "ImportError" in proc.stderr and "no fallback" in proc.stderr
