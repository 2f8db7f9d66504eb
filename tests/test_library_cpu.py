"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol that
include/octo.h declares, validates configurations before touching CUDA, and the ctypes
mirrors of the public structs have the C layout."""
import ctypes
import os
import re

import pytest

import paper_2502_01277_b200 as octo
from paper_2502_01277_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "octo.h")).read()
    return sorted(set(re.findall(r"OCTO_API\s+[\w\s\*]+?\b(octo_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = octo.load_library()
    names = _declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in octo.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_version_and_strerror():
    lib = octo.load_library()
    assert re.fullmatch(rb"\d+\.\d+", lib.octo_version())
    seen = set()
    for code in range(0, -8, -1):
        s = lib.octo_strerror(code)
        assert s and s != b"unknown status code"
        seen.add(s)
    assert len(seen) == 8
    assert lib.octo_strerror(-99) == b"unknown status code"


def test_struct_layouts_match_header():
    assert ctypes.sizeof(binding.BranchCfg) == 56
    assert ctypes.sizeof(binding.StageConfig) == 15 * 4 + 4 * 56
    assert ctypes.sizeof(binding.Frame) == 24
    assert binding.DET_DTYPE.itemsize == 32 and binding.ITEM_DTYPE.itemsize == 32
    assert ctypes.sizeof(binding.StageStats) == 40


@pytest.mark.parametrize("field,value", [
    ("net_size", 0), ("net_size", 641), ("net_size", 8192), ("max_batch", 0), ("max_batch", 513),
    ("num_anchors", 0), ("num_anchors", (1 << 24) + 1), ("num_classes", 0), ("num_classes", 129),
    ("head_is_logits", 2), ("conf_thresh", -0.1), ("conf_thresh", float("nan")), ("iou_thresh", 1.5),
    ("max_det", 0), ("pad_value", 256), ("pad_value", -1), ("swap_rb", 3), ("num_branches", 0),
    ("num_branches", 5), ("device", -1), ("head_layout", 2), ("multi_label", 2), ("class_agnostic", 2),
])
def test_create_rejects_bad_config_before_any_cuda_call(field, value):
    cfg = octo.make_config()
    setattr(cfg, field, value)
    with pytest.raises(octo.OctoError) as ei:
        octo.octo_stage_create(cfg)
    assert ei.value.code == binding.OCTO_E_INVALID_ARG


@pytest.mark.parametrize("ow,oh", [(0, 8), (12, 8), (4096, 8), (8, 0), (8, 4096)])
def test_create_rejects_bad_branch(ow, oh):
    cfg = octo.make_config(branches=((ow, oh),))
    with pytest.raises(octo.OctoError) as ei:
        octo.octo_stage_create(cfg)
    assert ei.value.code == binding.OCTO_E_INVALID_ARG


def test_null_arguments_are_rejected():
    lib = octo.load_library()
    assert lib.octo_stage_create(None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_stage_destroy(None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_preprocess_batch(None, None, 1, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_postprocess_batch(None, None, 1, None, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_crop_batch(None, 0, 0, 0, None, None, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_stage_workspace_bytes(None) == 0
    assert lib.octo_adopt_regions(None, None, 1, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_adopt_items_device(None, None, 0, 0, 1, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_stage_selftest_wait(None, 10, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_static_status(0, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_static_status(-1, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_queue_push(None, None, 0, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_queue_pop_due(None, 1, 0, None, None, None, None) == binding.OCTO_E_INVALID_ARG
    assert lib.octo_strerror(binding.OCTO_E_NO_MEMORY) == b"out of host or device memory"


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(ImportError):
        octo.load_library(str(tmp_path / "nope.so"))


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_01277_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("no cpu fallback", ""), f
