"""The shared library loads without a GPU, exports every symbol the header declares, and its
host-side logic (sizes, argument checks, bucket function) behaves as documented."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    from paper_2312_11462_b200 import build
    build.build()
    from paper_2312_11462_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "csd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(csd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(b):
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(b.lib, n), n


def test_struct_sizes_match_header(b):
    assert C.sizeof(b.ModelConfig) == 15 * 4
    assert C.sizeof(b.CascadeStats) == 8 * (1 + 32 + 2 + 1) + 3 * 8


def test_weight_bytes_match_blob_layout(b):
    for name, s in workloads.SHAPES.items():
        cfg = b.config_from_shape(s)
        _, total = workloads.blob_layout(s)
        assert b.lib.csd_model_weight_bytes(C.byref(cfg)) == 2 * total, name
        assert b.lib.csd_model_workspace_bytes(C.byref(cfg)) > 0


def test_config_validation(b):
    s = workloads.SHAPES["tiny_target"]
    cfg = b.config_from_shape(s)
    cfg.d_head = 48
    assert b.lib.csd_model_weight_bytes(C.byref(cfg)) == 0
    h = C.c_void_p()
    assert b.lib.csd_model_create(C.byref(cfg), 256, 1 << 20, 256, 1 << 20, None, C.byref(h)) == 2   # SHAPE
    cfg = b.config_from_shape(s)
    assert b.lib.csd_model_create(C.byref(cfg), None, 0, None, 0, None, C.byref(h)) == 1            # INVALID_ARG
    assert b.lib.csd_model_create(C.byref(cfg), 256, 16, 256, 16, None, C.byref(h)) == 3            # CAPACITY


def test_argument_checks_return_before_any_launch(b):
    L = b.lib
    assert L.csd_spec_accept(None, None, None, None, 1, 1, 8, 1.0, 1.0, 0, 0, None, None, None, 0, None) == 1
    assert L.csd_spec_accept(256, None, None, 256, 1, 1, 8, 1.0, 0.5, 0, 0, 256, 256, 256, 1 << 20, None) == 1
    assert L.csd_spec_accept(256, None, None, 256, 1, 1, 8, -1.0, 1.0, 0, 0, 256, 256, 256, 1 << 20, None) == 1
    assert L.csd_spec_accept(256, None, None, 256, 1, 65, 8, 1.0, 1.0, 0, 0, 256, 256, 256, 1 << 20, None) == 1
    assert L.csd_spec_accept(256, None, None, 256, 1, 1, 8, 1.0, 1.0, 0, 0, 256, 256, 256, 16, None) == 3
    assert L.csd_spec_accept(256, None, None, 256, 0, 1, 8, 1.0, 1.0, 0, 0, 256, 256, 256, 16, None) == 0  # no rows
    assert L.csd_linear(256, 8, 12, 256, 1, 256, 256, 1 << 20, None) == 1      # K not a multiple of 8
    assert L.csd_linear(256, 8, 16, 256, 129, 256, 256, 1 << 20, None) == 1    # too many rows
    assert L.csd_linear(256, 8, 16, 256, 18, 256, 256, 1 << 20, None) == 8     # a wide block needs a large matrix
    assert L.csd_prefill(None, 256, 4, 0, None) == 1
    assert L.csd_mag_draft(None, 256, 1, 1, 256, None) == 1
    assert L.csd_spec_accept_workspace_bytes(64, 16, 128256) > 0
    assert L.csd_cascade_workspace_bytes(32000, 4, 448, 128, 16) > 0
    assert L.csd_cascade_workspace_bytes(32000, 17, 448, 128, 16) == 0
    assert L.csd_status_string(3) == b"capacity exceeded"


def test_rel_bucket_agrees_with_oracle(b, orc):
    for bidir in (False, True):
        for rel in range(-400, 401):
            assert b.csd_rel_bucket(rel, bidir, 32, 128) == orc.rel_bucket(rel, bidir, 32, 128), (bidir, rel)
    for rel in range(-70, 71):
        assert b.csd_rel_bucket(rel, True, 16, 64) == orc.rel_bucket(rel, True, 16, 64)
