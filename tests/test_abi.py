"""The C-ABI library loads without a GPU and exports every symbol include/ks.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_35587_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ks.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ks_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15 and "ks_select" in names and "ks_featurize" in names and "ks_score" in names
    for n in names:
        assert hasattr(lib, n), n
    from paper_2609_35587_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_introspection_calls_need_no_gpu(lib):
    lib.ks_feature_name.restype = ctypes.c_char_p
    lib.ks_status_string.restype = ctypes.c_char_p
    assert lib.ks_feature_count() == 63
    names = [lib.ks_feature_name(i).decode() for i in range(63)]
    assert len(set(names)) == 63 and names[30] == "waves" and names[31] == "eta_last"
    assert lib.ks_feature_name(63) is None and lib.ks_feature_name(-1) is None
    assert lib.ks_status_string(0) == b"ok" and b"invalid" in lib.ks_status_string(1)


def test_create_rejects_bad_arguments_without_touching_a_gpu(lib):
    from paper_2609_35587_b200 import workloads as wl
    h = ctypes.c_void_p()
    assert lib.ks_create(None, 0, None) == 1
    assert lib.ks_create(ctypes.byref(h), 0, None) == 1
    bad = wl.gpu_desc().copy()
    bad["num_sms"] = 0
    assert lib.ks_create(ctypes.byref(h), 0, ctypes.c_void_p(bad.reshape(1).ctypes.data)) == 1
    assert h.value is None
    assert lib.ks_destroy(None) == 0 and lib.ks_model_destroy(None) == 0


def test_record_layouts_match_the_header():
    from paper_2609_35587_b200 import workloads as wl
    assert wl.PROBLEM_DT.itemsize == 16 and wl.CANDIDATE_DT.itemsize == 16
    assert wl.GPU_DESC_DT.itemsize == 80 and wl.NODE_DT.itemsize == 12
    assert wl.GPU_DESC_DT.fields["l2_bytes"][1] == 32
    assert wl.CANDIDATE_DT.fields["stages"][1] == 8 and wl.NODE_DT.fields["left"][1] == 8
