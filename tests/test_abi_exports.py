"""The CUDA library builds for sm_100a, loads without a GPU and exports every function that
include/disc.h declares.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "disc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(disc_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared()
    for must in ("disc_build_set", "disc_mask", "disc_step", "disc_resample"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2504_09135_b200 import binding
    L = binding.lib()
    for name in _declared():
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTS) == _declared()
    assert L.disc_error_string(-4).decode().startswith("a member is a proper prefix")


def test_no_cpu_fallback_without_a_device():
    import numpy as np
    import torch
    from paper_2504_09135_b200 import disc_build_set
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(RuntimeError):
        disc_build_set(np.array([0, 1], np.int32), np.array([0, 2], np.int64), 4)


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_09135_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "disc_oracle" not in text, f
