"""The C ABI without a GPU: the library loads, exports every declared symbol, and the
header and the binding agree on names."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pac_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2408_10746_b200 import build, binding
    build.build()
    lib = binding.load_library()
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_no_cpu_fallback_without_a_device():
    import torch
    import paper_2408_10746_b200 as pac
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(pac.PacError) as e:
        pac.PacContext(0)
    assert e.value.status_name == "PAC_ERR_CUDA"


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2408_10746_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("no CPU fallback", ""), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2408_10746_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
