"""The C-ABI library builds, loads, and exports every symbol include/omse.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_1902_06822_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_header_symbols_are_exported_and_bound():
    hdr = open(os.path.join(ROOT, "include", "omse.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(omse_[a-z0-9_]+)\s*\(", hdr))
    assert {"omse_quantize_weights", "omse_activation_scale", "omse_residual_quantize", "omse_pack_int4"} <= declared
    lib = ctypes.CDLL(build.build())
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_status_strings_need_no_device():
    assert binding.status_string(0) == "ok"
    assert "invalid" in binding.status_string(binding.EINVAL)


def test_header_limits_match_binding_constants():
    hdr = open(os.path.join(ROOT, "include", "omse.h")).read()
    for name, val in [("OMSE_MAX_CANDIDATES", binding.MAX_CANDIDATES), ("OMSE_MAX_KERNEL_LEN", binding.MAX_KERNEL_LEN),
                      ("OMSE_MAX_KERNEL_LEN_MULTISWEEP", binding.MAX_KERNEL_LEN_MULTISWEEP),
                      ("OMSE_MAX_TENSORS", binding.MAX_TENSORS)]:
        assert int(re.search(rf"#define {name}\s+(\d+)", hdr).group(1)) == val


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    """No fallback of any kind: without libomse.so the binding raises instead of computing elsewhere."""
    import pytest
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(build, "LIB_PATH", str(tmp_path / "libomse.so"))
    with pytest.raises(FileNotFoundError):
        binding.load_library()


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_1902_06822_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
