"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol, and
rejects bad arguments on the host before anything would be launched."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2504_05346_b200 import build as B
    import paper_2504_05346_b200 as T

    B.build()
    return T.load_library()


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            src = open(os.path.join(inc, f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names.update(re.findall(r"\b(thanos_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert "thanos_hessian_accumulate" in names and "thanos_prune_layer" in names
    assert "thanos_prepare_inverse" in names and len(names) >= 8
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_version(lib):
    import paper_2504_05346_b200 as T

    assert T.version() >= 100
    seen = {T.status_string(i) for i in range(9)}
    assert len(seen) == 9 and T.status_string(0) == "ok"
    assert T.status_string(99) == "unknown status"


def test_workspace_queries(lib):
    import paper_2504_05346_b200 as T

    assert T.workspace_bytes(1, 0, 4096, 0, T.F32) >= 4096 * 4096 * 4
    f32 = T.workspace_bytes(2, 4096, 4096, 128, T.F32)
    bf16 = T.workspace_bytes(2, 4096, 4096, 128, T.BF16)
    assert bf16 >= f32 + 4096 * 4096 * 4  # fp32 working copy for 16-bit weights
    assert T.workspace_bytes(2, 4096, 4097, 128, T.F32) == 0  # b % 8 != 0
    assert T.workspace_bytes(7, 1, 8, 8, T.F32) == 0
    assert T.workspace_bytes(3, 64, 64, 32, T.BF16) > T.workspace_bytes(2, 64, 64, 32, T.BF16)


def test_host_side_argument_checks_need_no_gpu(lib):
    # null pointers / bad shapes are rejected before any CUDA call
    vp = ctypes.c_void_p
    assert lib.thanos_hessian_accumulate(None, 64, None, 0, 16, 64, None, 0, None) == 1
    buf = (ctypes.c_char * 4096)()
    addr = ctypes.addressof(buf)
    addr = (addr + 255) // 256 * 256
    assert lib.thanos_hessian_accumulate(vp(addr), 60, vp(addr), 0, 16, 64, vp(addr), 256, None) == 2
    assert lib.thanos_hessian_accumulate(vp(addr), 64, vp(addr), 5, 16, 64, vp(addr), 256, None) == 3
    assert lib.thanos_hessian_accumulate(vp(addr), 64, vp(addr + 4), 0, 16, 64, vp(addr), 256, None) == 4
    assert lib.thanos_hessian_accumulate(vp(addr), 64, vp(addr), 0, 16, 60, vp(addr), 256, None) == 4
    assert lib.thanos_hessian_accumulate(vp(addr), 64, vp(addr), 0, 0, 64, vp(addr), 256, None) == 0
    assert lib.thanos_prepare_inverse(vp(addr), 64, ctypes.c_float(0.01), vp(addr), vp(addr),
                                      vp(addr), 16, vp(addr), None) == 5
    assert lib.thanos_prepare_inverse(vp(addr), 64, ctypes.c_float(-1.0), vp(addr), vp(addr),
                                      vp(addr), 1 << 30, vp(addr), None) == 1
    assert lib.thanos_prune_layer(vp(addr), vp(addr), vp(addr), 0, 8, 64, vp(addr), vp(addr), 1,
                                  ctypes.c_double(0.0), 2, 4, 30, vp(addr), 1 << 30, vp(addr),
                                  None) == 2
    assert lib.thanos_prune_layer(vp(addr), vp(addr), vp(addr), 0, 8, 64, vp(addr), vp(addr), 0,
                                  ctypes.c_double(1.5), 0, 0, 32, vp(addr), 1 << 30, vp(addr),
                                  None) == 1
    assert lib.thanos_prune_layer(vp(addr), vp(addr), vp(addr), 0, 8, 64, vp(addr), vp(addr), 0,
                                  ctypes.c_double(0.5), 0, 0, 32, vp(addr), 64, vp(addr),
                                  None) == 5


def test_missing_library_is_a_loud_error(monkeypatch, tmp_path):
    from paper_2504_05346_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_HERE", str(tmp_path))
    with pytest.raises(FileNotFoundError):
        binding.load_library()
    monkeypatch.setattr(binding, "_lib", None)


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_05346_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2504_05346_b200" not in src and "ctypes" not in src
