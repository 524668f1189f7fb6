"""The C-ABI library loads without a GPU and exports every function that
include/omnidraft.h declares (no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "omnidraft.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(od_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_step_functions():
    names = _declared()
    for n in ("od_map_proposals", "od_verify", "od_sample_residual", "od_create", "od_destroy",
              "od_set_vocab_map", "od_cache_build", "od_step_host"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_2507_02659_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for n in _declared():
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2507_02659_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    lib = binding.lib()
    assert lib.od_version() >= 100
    assert lib.od_status_string(0) == b"ok"
    assert b"inject" in lib.od_status_string(-3)


def test_binding_constants_match_the_header():
    from paper_2507_02659_b200 import binding
    text = open(os.path.join(ROOT, "include", "omnidraft.h")).read()
    def macro(name):
        m = re.search(rf"#define\s+{name}\s+(\S+)", text)
        return m.group(1)
    assert int(macro("OD_VF_BOUNDARY_MASK").rstrip("u"), 16) == binding.OD_VF_BOUNDARY_MASK
    assert int(macro("OD_VF_BAD_TEMPERATURE").rstrip("u"), 16) == binding.OD_VF_BAD_TEMPERATURE
    assert int(macro("OD_VF_NONFINITE").rstrip("u"), 16) == binding.OD_VF_NONFINITE
    assert int(macro("OD_SF_BOUNDARY").rstrip("u"), 16) == binding.OD_SF_BOUNDARY
    assert int(macro("OD_SF_ZERO_MASS").rstrip("u"), 16) == binding.OD_SF_ZERO_MASS
    assert int(macro("OD_SF_BONUS").rstrip("u"), 16) == binding.OD_SF_BONUS
    assert float(macro("OD_TAU_ACCEPT").rstrip("f")) == binding.OD_TAU_ACCEPT
    assert float(macro("OD_TAU_SAMPLE")) == binding.OD_TAU_SAMPLE
    assert int(macro("OD_MAX_K")) == binding.OD_MAX_K


def test_no_cuda_device_means_a_loud_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for the CPU-only box")
    from paper_2507_02659_b200 import binding
    with pytest.raises(Exception):
        binding.Context("cuda:0", 10, 10, 1, 1)
