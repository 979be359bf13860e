"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_1412_1576_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names += re.findall(r"\b(lda_[a-z_0-9]+)\s*\(", src)
    return sorted(set(names))


def test_library_builds_and_exports_declared_symbols():
    path = build.build_library()
    lib = ctypes.CDLL(path)
    declared = _declared()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    for name in binding.EXPORTS:
        assert name in declared


def test_argument_checks_need_no_gpu():
    L = binding.load_library()
    h = ctypes.c_void_p()
    assert L.lda_create(0, 4, 0.1, 0.1, ctypes.byref(h)) == binding.LDA_EINVAL
    assert L.lda_create(4, 4, -1.0, 0.1, ctypes.byref(h)) == binding.LDA_EINVAL
    assert L.lda_create(4, 4, float("nan"), 0.1, ctypes.byref(h)) == binding.LDA_EINVAL
    assert L.lda_create(4, 1 << 20, 0.1, 0.1, ctypes.byref(h)) == binding.LDA_ERANGE
    assert L.lda_create(4, 4, 0.1, 0.1, None) == binding.LDA_EINVAL
    assert L.lda_sweep(None, 1, 2) == binding.LDA_EINVAL
    assert L.lda_init(None, 0) == binding.LDA_EINVAL


def test_no_product_module_touches_the_oracle():
    """The product path must not import or call anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_1412_1576_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in src.lower() or fn == "synth.py", fn
                assert "ldaref" not in src
