"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports every symbol
declared in include/ee.h; the binding's struct layouts match the header's field order."""
import ctypes
import os
import re

import pytest

from paper_2209_13443_b200 import binding as eb
from paper_2209_13443_b200 import build as ebuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "ee.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ee_[a-z_0-9]+)\s*\(", src)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    so = ebuild.build()
    lib = ctypes.CDLL(so)
    names = _declared()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in ee.h but not exported"
    assert sorted(eb.EXPORTS) == names


def test_status_strings_without_a_device():
    lib = eb.load_library()
    assert lib.ee_status_string(0) == b"ok"
    assert b"capacity" in lib.ee_status_string(3)
    assert lib.ee_last_cuda_error() == b""


def test_wait_count_returns_the_value_or_times_out():
    """ee_wait_count is host-only: it polls a word until it leaves the sentinel (here a thread plays the GPU's copy)."""
    import threading
    import time

    lib = eb.load_library()
    word = ctypes.c_int32(-1)
    out = ctypes.c_int32(-7)
    assert lib.ee_wait_count(ctypes.addressof(word), -1, 0.05, ctypes.byref(out)) == eb.STATUS_NAMES.index("EE_ERR_TIMEOUT")
    assert out.value == -7                                   # untouched on timeout
    t = threading.Thread(target=lambda: (time.sleep(0.02), setattr(word, "value", 5)))
    t.start()
    assert lib.ee_wait_count(ctypes.addressof(word), -1, 5.0, ctypes.byref(out)) == 0 and out.value == 5
    t.join()
    assert lib.ee_wait_count(None, -1, 1.0, ctypes.byref(out)) == eb.STATUS_NAMES.index("EE_ERR_INVALID_ARG")


def test_binding_structs_follow_the_header():
    src = open(os.path.join(ROOT, "include", "ee.h")).read()

    def fields(struct_name):
        end = re.search(r"\}\s*" + struct_name + r"\s*;", src).start()
        body = src[src.rindex("typedef struct {", 0, end) + len("typedef struct {"):end]
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        out = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            for part in decl.split(","):
                out.append(re.findall(r"[A-Za-z_][A-Za-z_0-9]*", part)[-1])
        return out

    for cname, cls in [("ee_layer_desc_t", eb.LayerDesc), ("ee_stage_desc_t", eb.StageDesc), ("ee_model_desc_t", eb.ModelDesc),
                       ("ee_stage_info_t", eb.StageInfo), ("ee_stage_in_t", eb.StageIn), ("ee_stage_out_t", eb.StageOut),
                       ("ee_layer_plan_t", eb.LayerPlan)]:
        assert fields(cname) == [f for f, _ in cls._fields_], cname


def test_no_cpu_fallback():
    import torch

    if torch.cuda.is_available():
        pytest.skip("GPU present")
    from paper_2209_13443_b200 import workloads as wl

    with pytest.raises(RuntimeError):
        eb.EEModel(wl.tiny_ee_cnn())
