"""Host-side checks of the C ABI that need no GPU: the library builds, loads and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_06641_b200 import api, build
    build.build_library()
    return api.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "sneakpeek.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2505_06641_b200 import api
    names = _declared()
    assert len(names) >= 16 and set(names) == set(api.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_record_layouts_match_the_header(lib):
    from paper_2505_06641_b200 import api
    assert api.ROUND_DTYPE.itemsize == 64 and api.REQ_DTYPE.itemsize == 24
    assert api.ROUND_DTYPE.fields["t_start_ns"][1] == 32 and api.ROUND_DTYPE.fields["utility"][1] == 48
    assert api.REQ_DTYPE.fields["order"][1] == 16


def test_no_silent_fallback_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2505_06641_b200 import api, runner, synth
    with pytest.raises(api.SpError) as e:
        api.sp_create(0, 0)
    assert e.value.status == api.SP_ECUDA
    with pytest.raises(RuntimeError):
        runner.Session(synth.make_workload("C1"))


def test_default_options_need_no_gpu(lib):
    from paper_2505_06641_b200 import api
    o = api.sp_default_options()
    assert o == dict(trace_mode=0, timing=0, guard_utility=2e-5, guard_priority=2e-6)
    lib.sp_default_options(None)


def test_null_context_is_rejected(lib):
    assert lib.sp_reset(None) == 1 and lib.sp_check(None) == 1
    assert lib.sp_last_error(None) == b"null context"
    lib.sp_destroy(None)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_06641_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "synth.py", f
    text = open(os.path.join(pkg, "synth.py")).read()
    assert "import oracle" not in text and "from oracle" not in text
