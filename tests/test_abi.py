"""The C-ABI library builds for sm_100a, loads without a GPU, exports every declared symbol, and rejects bad
arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_23553_b200 import build
    build.build()
    from paper_2608_23553_b200 import binding
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "chimera.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(chimera_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_two_named_entry_points():
    names = declared_symbols()
    assert "chimera_build_index" in names and "chimera_search" in names
    assert len(names) >= 10


def test_every_declared_symbol_is_exported(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_version_and_error_text(lib):
    assert lib.chimera_version() >= 100
    assert lib.chimera_last_error() is not None


def test_null_arguments_are_rejected_without_a_device(lib):
    out = ctypes.c_void_p()
    assert lib.chimera_build_index(None, None, None, None, None, None, ctypes.byref(out)) == 1
    assert out.value is None
    assert b"NULL" in lib.chimera_last_error()
    n = ctypes.c_size_t()
    assert lib.chimera_workspace_bytes(None, 1, 32, 4, 16, 10, ctypes.c_int64(0), ctypes.byref(n)) == 1
    assert lib.chimera_search(None, None, 1, 32, 4, 16, 10, ctypes.c_int64(0), None, ctypes.c_size_t(0), None, None,
                              None) == 1
    assert lib.chimera_destroy_index(None) == 0
    st = ctypes.c_int32()
    assert lib.chimera_workspace_status(None, None, ctypes.byref(st)) == 1


def test_unsupported_descriptions_are_rejected_before_device_use(lib):
    from paper_2608_23553_b200.binding import _Desc
    out = ctypes.c_void_p()
    fake = ctypes.c_void_p(256)          # non-NULL, aligned; never dereferenced on these paths
    for desc, code in [(_Desc(100, 2, -0.25, 0.25, 4, 4, 4), 6), (_Desc(128, 3, -0.25, 0.25, 4, 4, 4), 6),
                       (_Desc(128, 2, 0.25, -0.25, 4, 4, 4), 1), (_Desc(128, 2, -0.25, 0.25, 0, 4, 4), 1)]:
        rc = lib.chimera_build_index(ctypes.byref(desc), fake, fake, fake, fake, None, ctypes.byref(out))
        assert rc == code, (desc.dim, desc.nbits, rc)


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    from paper_2608_23553_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libchimera.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_probe_sampling_rule_on_the_configurations_sizes(lib):
    """chimera_probe_sample_stride is plain arithmetic (no device): every 128 / max(nprobe, 4)-th tile of 128 centroids
    is a sample tile when there are at least 8 of them, nprobe <= 32 and q_len is a multiple of 4; 0 = table scan."""
    f = lib.chimera_probe_sample_stride
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]
    assert f(262144, 32, 4) == 32 and f(65536, 32, 4) == 32          # Large, Mid
    assert f(32768, 64, 8) == 16                                     # long documents
    assert f(1024, 32, 4) == 0                                       # Tiny: 8 tiles in all
    assert f(262144, 32, 1) == 32 and f(262144, 32, 16) == 8 and f(262144, 32, 32) == 4
    assert f(262144, 32, 33) == 0 and f(262144, 30, 4) == 0 and f(262144, 32, 0) == 0
    for nprobe in range(1, 33):
        s = f(1 << 20, 32, nprobe)
        assert s == 128 // max(nprobe, 4)
        k_min = 8 * s * 128 - 127                                    # fewest centroids with 8 * s tiles
        assert f(k_min, 32, nprobe) == s and f(k_min - 1, 32, nprobe) == 0
