"""CPU-side checks of the boundary: the C-ABI library builds for sm_100a, loads, exports
every symbol that include/tsenor.h declares, and rejects bad arguments on the host
(no kernel is launched here)."""
import os
import re

import pytest

from paper_2505_23949_b200 import binding as ts
from paper_2505_23949_b200 import build as ts_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ts_build.build()
    return ts.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "tsenor.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b(tsenor_[a-z_0-9]+)\s*\(", text))


def test_library_exports_every_declared_symbol(lib):
    declared = _declared_functions()
    assert declared == set(ts.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_checked_flavour_builds_and_exports_the_same_symbols():
    import ctypes
    checked = ctypes.CDLL(ts_build.build(bounds=True))
    for name in _declared_functions():
        assert getattr(checked, name) is not None


def test_host_arithmetic_and_messages(lib):
    assert [lib.tsenor_mask_words_per_row(c) for c in (0, 1, 32, 33, 4096)] == [0, 1, 1, 2, 128]
    for code in (0, -1, -2, -3, -4, -5):
        assert len(lib.tsenor_strerror(code)) > 1
    assert lib.tsenor_strerror(-99) == b"unknown status"


def test_argument_errors_are_decided_on_the_host(lib):
    n0 = lib.tsenor_launch_count()
    assert lib.tsenor_solve(None, 8, 8, 8, 2, 5, 1.0, 1, -1, None, None, None) == ts.ERR_NM
    assert lib.tsenor_solve(None, 8, 8, 8, 5, 4, 1.0, 1, -1, None, None, None) == ts.ERR_NM
    assert lib.tsenor_solve(None, 6, 8, 8, 2, 4, 1.0, 1, -1, None, None, None) == ts.ERR_SHAPE
    assert lib.tsenor_solve(None, 8, 8, 4, 2, 4, 1.0, 1, -1, None, None, None) == ts.ERR_SHAPE
    assert lib.tsenor_solve(None, 8, 8, 8, 2, 4, 1.0, -1, -1, None, None, None) == ts.ERR_ARG
    assert lib.tsenor_solve(None, 8, 8, 8, 2, 4, 1.0, 1, -1, None, None, None) == ts.ERR_NULL
    assert lib.tsenor_solve(None, 0, 8, 8, 2, 4, 1.0, 1, -1, None, None, None) == ts.OK
    assert lib.tsenor_dykstra(None, 8, 8, 8, 4, 4, 1.0, 1, None, 8, 0, None, None) == ts.ERR_NM
    assert lib.tsenor_dykstra(None, 8, 8, 8, 2, 4, 1.0, 1, None, 4, 0, None, None) == ts.ERR_SHAPE
    assert lib.tsenor_round(None, 8, None, 8, 8, 8, 2, 4, -1, None, None, None) == ts.ERR_NULL
    assert lib.tsenor_check(None, 8, 8, 2, 4, None, None) == ts.ERR_NULL
    assert lib.tsenor_objective(None, 8, None, 8, 8, None, None) == ts.ERR_NULL
    assert lib.tsenor_max_abs(None, 8, 8, 4, None, None) == ts.ERR_SHAPE
    assert lib.tsenor_launch_count() == n0


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(TypeError):
        ts.solve(torch.zeros(8, 8), 2, 4, 1.0)


def test_layout_setting_is_validated_and_returns_the_previous_value(lib):
    assert lib.tsenor_set_layout(7) == ts.ERR_ARG and lib.tsenor_set_layout(-1) == ts.ERR_ARG
    assert ts.set_layout(ts.LAYOUT_LATENCY) == ts.LAYOUT_AUTO
    assert ts.set_layout(ts.LAYOUT_THROUGHPUT) == ts.LAYOUT_LATENCY
    assert ts.set_layout(ts.LAYOUT_AUTO) == ts.LAYOUT_THROUGHPUT
    with pytest.raises(ts.TsenorError):
        ts.set_layout(3)


def test_output_tensor_checks_raise_before_anything_reaches_the_library():
    """The binding rejects outputs of the wrong kind on the host (no CUDA call is made)."""
    import torch
    cpu = torch.zeros(8, 1, dtype=torch.int32)
    for bad, kw in [(cpu, dict(dtype=torch.int32, device="cuda:0")),]:
        with pytest.raises(TypeError):
            ts._out(bad, "mask_out", kw["dtype"], kw["device"])
    assert ts._out(None, "status", torch.int32, "cuda:0") is None


def test_header_is_plain_c(tmp_path):
    """include/tsenor.h compiles as C11 and as C++ on its own (no CUDA headers needed by a caller)."""
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "tsenor.h"\n'
                   '#include <string.h>\n'
                   'int use(void) { tsenor_scores_t s; memset(&s, 0, sizeof s); s.kind = TSENOR_SCORES_ABS; '
                   'return (int)tsenor_mask_words_per_row(64) + s.kind + TSENOR_LAYOUT_AUTO; }\n')
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-I", inc, "-c", str(src), "-o",
                    str(tmp_path / "c.o")], check=True)
    subprocess.run(["g++", "-std=c++17", "-Wall", "-Wextra", "-Werror", "-x", "c++", "-I", inc, "-c", str(src), "-o",
                    str(tmp_path / "cc.o")], check=True)
