"""The C-ABI library loads without a GPU and exports every function the header declares."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "reader_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(reader_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2508_09072_b200 import binding, build
    build.build()
    lib = binding.load_library()
    names = declared_functions()
    assert "reader_verify_attn" in names and "reader_accept" in names and "reader_kv_commit" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names
    assert binding.status_string(0) == "ok"
    assert "tree" in binding.status_string(binding.ERR_BAD_TREE)


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2508_09072_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f
    osrc = open(os.path.join(ROOT, "oracle", "__init__.py")).read() + open(os.path.join(ROOT, "oracle", "reader_oracle.c")).read()
    assert "paper_2508_09072_b200" not in osrc and "libreader_verify" not in osrc and "csrc" not in osrc
    assert "reader_verify.h" not in osrc


def test_no_gpu_means_a_loud_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2508_09072_b200 import binding
    with pytest.raises(RuntimeError):
        binding.Reader(0)
