"""The C-ABI library builds, loads without a GPU and exports every call the header declares."""
import ctypes
import os
import re

from paper_2207_09682_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "qgbdt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qgbdt_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_call():
    lib = ctypes.CDLL(build.build())
    names = header_functions()
    assert "qgbdt_build_histograms" in names and "qgbdt_train" in names and len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_header_sizes():
    # int32 x5, double x4, uint64, int32 x2 -> 72 bytes; split record 72 bytes; model: 8 pointers
    assert ctypes.sizeof(binding.Params) == 72
    assert ctypes.sizeof(binding.Split) == 72
    assert ctypes.sizeof(binding.Model) == 8 * ctypes.sizeof(ctypes.c_void_p)


def test_null_arguments_are_rejected_without_a_device():
    lib = ctypes.CDLL(build.build())
    assert lib.qgbdt_create(None, None) == binding.ERR_ARG
    assert lib.qgbdt_destroy(None) == binding.ERR_ARG
    assert lib.qgbdt_train(None, None, None, 0, 0, None, None) == binding.ERR_ARG
    assert lib.qgbdt_build_histograms(None, 0, None, None) == binding.ERR_ARG
    bad = binding.make_params(bits=9)
    h = ctypes.c_void_p()
    assert lib.qgbdt_create(ctypes.byref(h), ctypes.byref(bad)) == binding.ERR_ARG


def test_product_path_does_not_reach_the_checker():
    pkg = os.path.join(ROOT, "paper_2207_09682_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "qo_" not in text, f
