"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
before touching the GPU (so these run on a box without one)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2602_02711_b200 import build, binding
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dmr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dmr_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"dmr_quantize", "dmr_lowbit_linear", "dmr_routed_linear", "dmr_dense_linear"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_size_queries(L):
    from paper_2602_02711_b200 import QFormat
    f = QFormat(4, 128)
    assert L.dmr_qweight_bytes(512, 512, f) == 512 * 512 // 2
    assert L.dmr_scales_bytes(512, 512, f) == 512 * 4 * 2
    assert L.dmr_zeros_bytes(512, 512, f) == 512 * 4
    assert L.dmr_qweight_bytes(8, 256, QFormat(8, 0)) == 8 * 256
    assert L.dmr_scales_bytes(8, 256, QFormat(8, 0)) == 8 * 2
    assert L.dmr_qweight_bytes(8, 96, QFormat(4, 64)) == 0      # g does not divide K
    assert L.dmr_qweight_bytes(8, 256, QFormat(3, 128)) == 8 * 256 * 3 // 8   # 32 codes in three words
    assert L.dmr_qweight_bytes(8, 256, QFormat(2, 128)) == 0    # unsupported width
    for op in (0, 1, 2):
        b = L.dmr_workspace_bytes(op, 64, 5120, 5120, f)
        assert b >= 256 and b % 256 == 0


def test_status_strings(L):
    seen = set()
    for code in range(8):
        s = L.dmr_status_string(code)
        assert s and s not in seen
        seen.add(s)


def test_argument_errors_are_reported_before_any_launch(L):
    from paper_2602_02711_b200 import QFormat
    f = QFormat(4, 128)
    buf = ctypes.create_string_buffer(4096 + 64)
    base = (ctypes.addressof(buf) + 63) // 64 * 64
    p = ctypes.c_void_p(base)
    odd = ctypes.c_void_p(base + 2)
    n0 = L.dmr_launch_count()
    # null pointers / bad sizes
    assert L.dmr_quantize(None, 8, 128, f, p, p, p, None, None) == 1
    assert L.dmr_quantize(p, 8, 96, QFormat(4, 64), p, p, p, None, None) == 1
    assert L.dmr_quantize(p, 8, 128, QFormat(2, 128), p, p, p, None, None) == 2
    assert L.dmr_quantize(odd, 8, 128, f, p, p, p, None, None) == 3
    assert L.dmr_lowbit_linear(p, -1, p, p, p, 8, 128, f, p, 0, p, 4096, None) == 1
    assert L.dmr_lowbit_linear(p, 1, None, p, p, 8, 128, f, p, 0, p, 4096, None) == 1
    assert L.dmr_lowbit_linear(p, 1, p, p, p, 8, 128, f, p, 5, p, 4096, None) == 1
    assert L.dmr_lowbit_linear(odd, 1, p, p, p, 8, 128, f, p, 0, p, 4096, None) == 3
    assert L.dmr_lowbit_linear(p, 1, p, p, p, 8, 128, f, p, 0, None, 0, None) == 4
    assert L.dmr_lowbit_linear(p, 1, p, p, p, 8, 128, f, p, 0, p, 16, None) == 4
    assert L.dmr_dense_linear(p, 1, None, 8, 128, p, 0, p, 4096, None) == 1
    assert L.dmr_routed_linear(p, 4, None, p, p, p, p, 8, 128, f, p, 0, p, 4096, None) == 1
    assert L.dmr_routed_linear(p, 4, p, p, p, p, p, 8, 128, f, p, 0, p, 256, None) == 4
    # M = 0 is a no-op that succeeds without launching
    assert L.dmr_lowbit_linear(p, 0, p, p, p, 8, 128, f, p, 0, p, 4096, None) == 0
    assert L.dmr_dense_linear(p, 0, p, 8, 128, p, 0, p, 4096, None) == 0
    assert L.dmr_routed_linear(p, 0, p, p, p, p, p, 8, 128, f, p, 0, p, 4096, None) == 0
    assert L.dmr_launch_count() == n0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2602_02711_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "libdmr.so"))
    with pytest.raises(binding.DmrError):
        binding.lib()


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2602_02711_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text, fn
                assert "liboracle" not in text and "dmr_oracle" not in text, fn
