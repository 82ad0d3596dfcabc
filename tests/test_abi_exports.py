"""The C-ABI library builds for sm_100a, loads, and exports every symbol the public header declares.
No compute call is made here (there is no GPU on the CPU test box)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for m in re.finditer(r"\b(rm_[a-z_0-9]+)\s*\(", text):
            names.add(m.group(1))
    return sorted(names)


@pytest.fixture(scope="module")
def libpath():
    from paper_2609_19104_b200.build import build_library
    return build_library()


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for required in ("rm_mask_compact", "rm_sparse_mlp", "rm_action_expert_step"):
        assert required in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"


def test_binding_lists_the_same_names(libpath):
    import paper_2609_19104_b200 as rm
    assert sorted(rm.EXPORTS) == declared_functions()
    rm.load_library()
    assert rm.status_string(0) == "ok"
    assert "index" in rm.status_string(rm.RM_ERR_INDEX)


def test_no_gpu_means_a_loud_failure(libpath):
    import torch
    import paper_2609_19104_b200 as rm
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        rm.Context(1, 64, 8, 4)


def test_product_does_not_reach_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_19104_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text and "rm_oracle" not in text, fn
