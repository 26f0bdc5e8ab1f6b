"""The C boundary on a box without a GPU: the library builds, loads, and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    import importlib.util
    spec = importlib.util.spec_from_file_location(
        "hotline_build", os.path.join(ROOT, "paper_2204_05436_b200", "csrc", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod.build_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hotline.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"HL_API[^;(]*?\b(hl_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_seven_path_calls():
    names = declared_functions()
    for required in ("hl_profile_hot", "hl_build_remap", "hl_fragment", "hl_embbag_fwd", "hl_embbag_bwd_sgd",
                     "hl_gather_cold", "hl_scatter_cold"):
        assert required in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol(lib_path):
    import paper_2204_05436_b200 as hl
    for name in declared_functions():
        assert name in hl.binding.EXPORTS
        assert callable(getattr(hl, name if name != "hl_strerror" else "strerror"))


def test_host_side_argument_checks(lib_path):
    """Calls that fail on the host before touching a device."""
    import paper_2204_05436_b200 as hl
    assert hl.strerror(hl.HL_EBOUNDS).startswith("index outside")
    geom = hl.make_geometry([10, 20], 16, 1)
    assert hl.hl_workspace_bytes(geom, 64, 128, 10, 10) > 0
    with pytest.raises(hl.HotlineError):
        hl.hl_workspace_bytes(hl.make_geometry([10, 20], 6, 1), 64, 128, 10, 10)       # dim not a multiple of 4
    with pytest.raises(hl.HotlineError):
        hl.hl_workspace_bytes(hl.make_geometry([2 ** 31], 16, 1), 64, 128, 10, 10)     # row ids must fit int32
    with pytest.raises(hl.HotlineError):
        hl.hl_create(geom, 64, 128, 10, 10, None, 0)                                   # no workspace
    big = hl.hl_workspace_bytes(hl.make_geometry([40_000_000] * 6, 64, 1), 16384, 16384 * 6, 4_194_304, 100_000)
    assert big < 4 << 30
