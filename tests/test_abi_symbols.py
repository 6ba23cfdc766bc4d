"""CPU-only checks of the boundary: the library builds, loads, and exports what include/precc.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_34054_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "precc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(precc_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_named_entry_points():
    names = _declared()
    for n in ("precc_lr_precompute", "precc_lr_attend_decode", "precc_lr_attend_prefill", "precc_rebase_project"):
        assert n in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), f"{name} declared in precc.h but not exported"


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2609_34054_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    binding.load_library()


def test_host_only_calls_work_without_a_gpu(lib_path):
    from paper_2609_34054_b200 import binding, inputs as I
    lib = binding.load_library()
    assert lib.precc_error_name(0) == b"PRECC_OK" and lib.precc_error_name(2) == b"PRECC_ERR_UNSUPPORTED"
    d = binding.layer_desc(I.C2)
    n = lib.precc_decode_workspace_bytes(ctypes.byref(d), 1, 8192, 148)
    assert n > 0 and n % 4 == 0
    n2 = lib.precc_decode_workspace_bytes(ctypes.byref(d), 64, 32768, 148)
    assert n2 > n
    bad = binding.layer_desc(I.Geometry(128, 8, 2, 96, 2, 16, 16, 1.0))
    assert lib.precc_decode_workspace_bytes(ctypes.byref(bad), 1, 128, 148) == 0


def test_product_path_fails_loudly_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    from paper_2609_34054_b200.binding import Precc, PreccError
    with pytest.raises(PreccError):
        Precc(0)


def test_product_package_never_imports_the_oracle():
    imp = re.compile(r"^\s*(from|import)\s+([\w\.]+)", re.M)
    pkg = os.path.join(ROOT, "paper_2609_34054_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith(".py"):
                mods = [m[1] for m in imp.findall(open(os.path.join(dirpath, f)).read())]
                assert not any(m.split(".")[0] == "oracle" for m in mods), f"{f} imports the oracle"
            if f.endswith((".cu", ".cuh")):
                assert "oracle/" not in open(os.path.join(dirpath, f)).read()
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            mods = [m[1] for m in imp.findall(open(os.path.join(ROOT, "oracle", f)).read())]
            assert not any("paper_2609_34054_b200" in m or m == "torch" or m == "ctypes" for m in mods)
