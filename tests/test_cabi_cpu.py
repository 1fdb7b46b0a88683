"""CPU checks of the boundary: the C-ABI library loads without a GPU, exports every function include/enec.h
declares, and its pure host function agrees with the oracle's closed-form size."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libenec():
    from paper_2604_03298_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "enec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(enec_[a-z_]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for want in ("enec_max_compressed_size", "enec_compress", "enec_compress_with_params", "enec_decompress",
                 "enec_compress_batched", "enec_decompress_batched", "enec_compress_noalloc", "enec_compress_blockwise",
                 "enec_decompress_blockwise", "enec_max_compressed_size_blockwise", "enec_launch_count", "enec_allocation_count",
                 "enec_version"):
        assert want in names


def test_library_exports_every_declared_symbol(libenec):
    for name in declared_functions():
        assert hasattr(libenec, name), name


def test_max_compressed_size_matches_oracle(libenec, oracle):
    f = libenec.enec_max_compressed_size
    f.argtypes = [ctypes.c_int, ctypes.c_size_t]
    f.restype = ctypes.c_size_t
    for dt in (0, 1, 2):
        for count in (0, 1, 15, 16, 17, 4096, 16383, 16384, 16385, 123457, 1 << 20, 128256 * 4096, (1 << 36) - 1):
            assert f(dt, count) == oracle.max_compressed_size(dt, count)
    assert f(3, 100) == 0 and f(0, 1 << 36) == 0
    f = libenec.enec_max_compressed_size_blockwise
    f.argtypes = [ctypes.c_int, ctypes.c_size_t]
    f.restype = ctypes.c_size_t
    for dt in (0, 1, 2):
        for count in (0, 1, 15, 16, 17, 4096, 16383, 16384, 16385, 123457, 1 << 20, 128256 * 4096, (1 << 36) - 1):
            assert f(dt, count) == oracle.max_compressed_size_blockwise(dt, count)
    assert f(3, 100) == 0 and f(0, 1 << 36) == 0


def test_binding_has_the_same_names():
    import paper_2604_03298_b200 as enec
    for name in declared_functions():
        if name in ("enec_version",):
            continue
        assert hasattr(enec, name), name


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2604_03298_b200 import binding
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        binding.lib()
