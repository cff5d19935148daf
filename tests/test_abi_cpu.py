"""The C-ABI library loads without a GPU and exports every symbol include/rkv.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2411_05787_b200 import build
    build.build()
    from paper_2411_05787_b200 import rkv
    return rkv


def _declared_symbols():
    with open(os.path.join(ROOT, "include", "rkv.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(rkv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib.lib, n), n
    assert sorted(lib.EXPORTS) == names


def test_workspace_bytes_and_config_validation(lib):
    ok = lib.RkvConfig(1, 32, 8, 128, 32768, 2560, 0, 1, 0.0)
    nbytes = lib.lib.rkv_workspace_bytes(ctypes.byref(ok))
    # logits scratch alone is B*Hkv*G*stride*4 bytes
    assert nbytes >= 32 * 32768 * 4
    for bad in (lib.RkvConfig(1, 32, 8, 64, 32768, 2560, 0, 1, 0.0),      # head_dim
                lib.RkvConfig(1, 36, 4, 128, 32768, 2560, 0, 1, 0.0),     # G = 9
                lib.RkvConfig(1, 32, 5, 128, 32768, 2560, 0, 1, 0.0),     # Hq % Hkv
                lib.RkvConfig(0, 32, 8, 128, 32768, 2560, 0, 1, 0.0),
                lib.RkvConfig(1, 32, 8, 128, 32768, 2560, 3, 1, 0.0)):    # unknown aggregation
        assert lib.lib.rkv_workspace_bytes(ctypes.byref(bad)) == 0
        h = ctypes.c_void_p(1234)
        rc = lib.lib.rkv_create(ctypes.byref(bad), ctypes.byref(h))
        assert rc in (1, 2) and not h.value
    assert lib.lib.rkv_status_string(0) == b"ok"
    assert lib.lib.rkv_status_string(2) == b"unsupported configuration"


def test_null_arguments_are_rejected_before_any_launch(lib):
    assert lib.lib.rkv_destroy(None) == 1
    assert lib.lib.rkv_launch_count(None) == 0
    assert lib.lib.rkv_small_step(None, None, None, None, None, 0, None) == 1
    assert lib.lib.rkv_append(None, None, None, None, None, None) == 1
    assert lib.lib.rkv_should_refresh(None, None, None, 0.5, None, None, None, None) == 1


def test_harness_library_exports_every_declared_symbol():
    """libllama_harness.so (decoder kernels of the end-to-end workload) against include/rkv_harness.h."""
    from paper_2411_05787_b200 import build
    build.build()
    from paper_2411_05787_b200 import harness
    with open(os.path.join(ROOT, "include", "rkv_harness.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    names = sorted(set(re.findall(r"\b(llh_[a-z_]+)\s*\(", text)))
    assert len(names) == 6 and sorted(harness.EXPORTS) == names
    for n in names:
        assert hasattr(harness.lib, n), n
    assert harness.lib.llh_gemv(None, None, 0, None, 1e-5, None, None, 8, 256, None) == -1      # null pointers: rejected on the host
    assert harness.lib.llh_rmsnorm(None, None, 1e-5, None, 4096, None) == -1
