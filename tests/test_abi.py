"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

from conftest import ROOT

HEADER = os.path.join(ROOT, "include", "sketched_amsgrad.h")


def _declared():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(sk_[a-z_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = _declared()
    for must in ("sk_create", "sk_step", "sk_destroy"):
        assert must in names
    assert len(names) >= 12


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2210_07454_b200 import binding, build
    path = build.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(L, name), f"{name} declared in the header but not exported"
    assert sorted(binding.EXPORTS) == _declared()
    L.sk_version.restype = ctypes.c_char_p
    assert b"sm_100a" in L.sk_version()


def test_no_cpu_fallback_without_a_device():
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2210_07454_b200 import binding
    with pytest.raises(binding.SkError):
        binding.SketchedAMSGrad(1024, 2, 5, 256, 16)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2210_07454_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".inc")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "sk_oracle" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2210_07454_b200" not in text and "sketched_amsgrad.h" not in text, f


def test_every_option_the_library_parses_is_documented_in_the_header():
    # the option names are string literals on both sides: a name sk_set_option / sk_get_option compares against must
    # appear, quoted, in the header's description of the options
    import re
    src = open(os.path.join(ROOT, "paper_2210_07454_b200", "csrc", "sk_api.cu")).read()
    names = set(re.findall(r'strcmp\(key, "([A-Za-z_0-9]+)"\)', src))
    assert {"log2g", "window_lines", "chained_launches", "timing"} <= names
    header = open(os.path.join(ROOT, "include", "sketched_amsgrad.h")).read()
    missing = sorted(n for n in names if f'"{n}"' not in header)
    assert not missing, missing
