"""The C-ABI library builds for sm_100a, loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "omnitide.h")


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_34653_b200 import build
    return build.build()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(omni(?:tide|page)_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_hot_path_calls():
    names = _declared_functions()
    for required in ("omnitide_score_units", "omnitide_select_units", "omnipage_compact", "omnitide_chunk_attention"):
        assert required in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_entry_points(lib_path):
    torch = pytest.importorskip("torch")
    from paper_2609_34653_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_functions()
    binding.load_library()          # sets argtypes for every export


def test_struct_layouts_match_the_header():
    from paper_2609_34653_b200 import binding
    assert ctypes.sizeof(binding.Geometry) == 28
    assert ctypes.sizeof(binding.SelectParams) == 20
    assert ctypes.sizeof(binding.StructuralParams) == 28
    assert ctypes.sizeof(binding.CompactInfo) == 32
    assert ctypes.sizeof(binding.ClassInfo) == 32


def test_create_without_gpu_fails_loudly(lib_path):
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2609_34653_b200 import binding
    with pytest.raises(binding.OmniTideError):
        binding.Context(4, 1, 64, "fp32", 128, 8, 16)
