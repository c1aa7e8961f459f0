"""CPU-side checks of the boundary: the shared library builds for sm_100a, loads, and exports every entry
point that include/graft.h declares; without a CUDA device it refuses to work instead of falling back."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "graft.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(graft_[a-z_]+)\s*\(", text)))


def test_header_and_library_agree():
    from paper_2608_20375_b200 import binding
    lib = binding.load_library()
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in graft.h but not exported"
    assert sorted(binding.ENTRY_POINTS) == names
    assert lib.graft_version().decode().startswith("graft-b200")
    assert lib.graft_status_str(2).decode() != lib.graft_status_str(1).decode()


def test_binding_exposes_the_same_names():
    from paper_2608_20375_b200 import Graft
    for n in ("build_trees", "accept", "vocab_pass", "tdes_edges", "tdes_precompute", "set_saba", "set_tdes_tables",
              "build_trees_host", "launch_count", "set_timing", "read_timing"):
        assert hasattr(Graft, n)


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a GPU")
def test_no_cpu_fallback():
    from paper_2608_20375_b200 import Graft, GraftError, binding
    with pytest.raises(GraftError):
        Graft(1000, 4, 4, 16, 8, 1, 8, 8)
    lib = binding.load_library()
    cfg = binding._Config(1000, 4, 4, 16, 8, 1, 8, 8, 8, 0.2, 1, 0, 0)
    ctx = C.c_void_p()
    assert lib.graft_create(C.byref(cfg), C.byref(ctx)) == 3 and not ctx.value  # GRAFT_ERR_CUDA
    cfg.K = 64
    assert lib.graft_create(C.byref(cfg), C.byref(ctx)) == 2  # limits are checked before the device


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2608_20375_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f"{f} mentions the oracle"
    assert "paper_2608_20375_b200" not in open(os.path.join(ROOT, "oracle", "__init__.py")).read()
    assert "include" not in open(os.path.join(ROOT, "oracle", "graft_oracle.c")).read().replace("#include <", "")
