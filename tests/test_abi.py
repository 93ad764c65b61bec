"""The C-ABI library loads, exports every function include/evo.h declares, and fails loudly
instead of falling back when there is no device (CPU only, no compute calls)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_03760_b200 import build
    return C.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "evo.h")).read()
    return re.findall(r"EVO_API\s+[\w\s\*]+?\b(evo_\w+)\s*\(", text)


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"evo_create", "evo_destroy", "evo_strerror", "evo_last_error", "evo_gen_inputs", "evo_validate",
            "evo_validate_host", "evo_fitness", "evo_fitness_host", "evo_plan_inspect", "evo_launch_count",
            "evo_set_timing_events", "evo_validate_static", "evo_validate_static_error", "evo_check",
            "evo_selftest_wait", "evo_fitness_ex", "evo_summary", "evo_select_elite", "evo_mismatch_sample", "evo_validate_exact", "evo_validate_f64"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_record_layouts_match_the_header():
    from paper_2510_03760_b200 import binding
    assert binding.RESULT_DTYPE.itemsize == 40 and binding.FIT_DTYPE.itemsize == 16
    assert [binding.RESULT_DTYPE.fields[k][1] for k in ("n_mismatch", "n_nonfinite", "sse", "max_abs", "max_rel", "flags", "pass")] \
        == [0, 8, 16, 24, 28, 32, 36]
    assert [binding._DESC_DTYPE.fields[k][1] for k in ("n", "ref", "dtype", "group")] == [0, 8, 16, 20]


def test_status_strings(lib):
    lib.evo_strerror.restype = C.c_char_p
    seen = {lib.evo_strerror(s) for s in range(0, -7, -1)}
    assert len(seen) == 7 and b"unknown status" not in seen
    assert lib.evo_strerror(-99) == b"unknown status"


def test_null_context_is_rejected_before_any_cuda_call(lib):
    for name, nargs in [("evo_gen_inputs", 7), ("evo_validate", 12), ("evo_validate_host", 12), ("evo_fitness", 9),
                        ("evo_fitness_host", 9)]:
        fn = getattr(lib, name)
        fn.restype = C.c_int
        assert fn(*([None] * nargs)) == -1, name
    assert lib.evo_create(None, 0) == -1


@pytest.mark.skipif(torch.cuda.is_available(), reason="needs a machine without a CUDA device")
def test_no_device_means_an_error_not_a_fallback(lib):
    h = C.c_void_p()
    assert lib.evo_create(C.byref(h), 0) == -4 and not h.value
    from paper_2510_03760_b200 import Context, EvoError
    with pytest.raises(EvoError):
        Context(0)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2510_03760_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "libevo.so"))
    with pytest.raises(ImportError):
        binding.load_library()


def test_product_does_not_reach_into_the_oracle():
    pkg = os.path.join(ROOT, "paper_2510_03760_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2510_03760_b200" not in text and "libevo.so" not in text, f


def test_the_header_is_plain_c(tmp_path):
    """include/evo.h is the boundary: it must compile as C99 without warnings, no C++ needed."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("gcc not found")
    src = tmp_path / "use_evo.c"
    src.write_text('#include "evo.h"\nint main(void) { evo_result r; evo_desc d; (void)r; (void)d; return EVO_OK; }\n')
    p = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                        "-fsyntax-only", str(src)], capture_output=True, text=True)
    assert p.returncode == 0, p.stderr
