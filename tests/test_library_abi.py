"""The C-ABI shared library builds, loads without a GPU and exports every function that
include/niti.h declares (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2009_13108_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "niti.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(niti_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared()
    for must in ["niti_linear_fwd", "niti_linear_bwd", "niti_conv_fwd", "niti_conv_dgrad",
                 "niti_conv_wgrad", "niti_int_xent", "niti_int_sgd_update"]:
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_library_is_built_from_the_sources_in_the_tree(lib_path):
    """build() records the digest of the sources next to the binary and rebuilds when they differ; the
    binding warns when it loads a library built from other sources."""
    from paper_2009_13108_b200 import build
    assert build.built_from_current_sources() is True
    assert len(build.source_digest()) == 64


def test_binding_lists_the_same_names(lib_path):
    from paper_2009_13108_b200 import api
    assert sorted(api.EXPORTS) == _declared()


def test_workspace_query_needs_no_gpu(lib_path):
    lib = ctypes.CDLL(lib_path)
    lib.niti_workspace_bytes.restype = ctypes.c_size_t
    dims = (ctypes.c_int64 * 3)(64, 256, 784)
    assert lib.niti_workspace_bytes(0, dims, 3) >= 64 * 256 * 4
    assert lib.niti_workspace_bytes(0, dims, 2) == 0
    assert lib.niti_workspace_bytes(99, dims, 3) == 0


def test_no_cpu_fallback_without_cuda():
    import torch
    from paper_2009_13108_b200 import Niti, NitiError
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(NitiError):
        Niti(0)


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2009_13108_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, os.path.join(dirpath, f)
