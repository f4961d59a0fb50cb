"""The C-ABI library builds, loads and exports every function include/rtma.h declares.
No compute calls: this runs without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2305_09887_b200 import build
    return ctypes.CDLL(build.build_library())


def _declared():
    text = open(os.path.join(ROOT, "include", "rtma.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rtma_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_named_calls():
    names = _declared()
    for must in ("rtma_partition", "rtma_build_induced_csr", "rtma_local_steps", "rtma_aggregate"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2305_09887_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_param_count_and_struct_layout(lib):
    from paper_2305_09887_b200 import binding, inputs
    assert ctypes.sizeof(binding.ModelDesc) == 4 + 4 * 9 + 4 + 4 + 3 * 4
    for dims in [(64, 64, 8), (128, 256, 256, 47), (100, 256, 256, 47), (128, 256, 2), (512, 512, 512, 47)]:
        assert binding.param_count(dims) == inputs.param_count(dims)
    assert binding.param_count((128, 256, 256, 47)) == 221231   # the Medium model
    assert binding.param_count((512, 512, 512, 47)) == 1097775  # the sweep model
    # variants: GCN has one weight matrix per layer; hidden layers add gamma, beta (norm) and a slope (PReLU)
    assert binding.param_count((128, 256, 256, 47), (1, 0, 0)) == 129 * 256 + 257 * 256 + 257 * 47
    assert binding.param_count((128, 256, 256, 47), (1, 1, 1)) == 129 * 256 + 257 * 256 + 257 * 47 + 2 * (2 * 256 + 1)
    assert binding.param_count((128, 256, 256, 47), (0, 1, 0)) == 221231 + 2


def test_no_cpu_fallback_without_a_device():
    import torch
    from paper_2305_09887_b200 import binding
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.RtmaError):
        binding.Context(0)


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2305_09887_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
