"""Host-side checks of the CUDA library that need no GPU: it loads, exports every
symbol the public header declares, and its pure host entry points behave."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def qesgd():
    from paper_1901_03040_b200 import build
    build.build()
    from paper_1901_03040_b200 import qesgd as mod
    return mod


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "qesgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qesgd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(qesgd):
    names = _declared_symbols()
    assert len(names) >= 16
    for name in names:
        assert hasattr(qesgd.lib, name), f"{name} is declared in qesgd.h but not exported"
        assert name in qesgd.SIGNATURES, f"{name} has no ctypes signature"
    assert sorted(qesgd.SIGNATURES) == names


def test_size_helpers(qesgd):
    assert qesgd.num_buckets(0, 512) == 0
    assert qesgd.num_buckets(1, 512) == 1
    assert qesgd.num_buckets(11_689_512, 512) == 22_832
    assert qesgd.num_buckets(25_557_032, 256) == 99_833
    assert qesgd.num_buckets(1 << 30, 128) == 8_388_608
    assert qesgd.num_buckets(100, 100) == 0            # not a power of two
    assert qesgd.code_bytes(1 << 24, 512, 2) == 4 << 20
    assert qesgd.code_bytes(1 << 24, 512, 8) == 16 << 20
    assert qesgd.code_bytes(11_689_512, 512, 4) == 22_832 * 256
    assert qesgd.code_bytes(1000, 512, 3) == 0
    for bucket in (64, 128, 8192):
        for bits in (2, 4, 8):
            assert qesgd.code_bytes(12345, bucket, bits) % 16 == 0


def test_null_context_and_strerror(qesgd):
    lib = qesgd.lib
    assert lib.qesgd_destroy(None) == qesgd.EINVAL
    assert lib.qesgd_encode(None, None, None, 10, 512, 7, 4, 0, 0.0, 0, 0, 0, None, None) == qesgd.EINVAL
    assert lib.qesgd_decode(None, None, None, 10, 512, 7, 4, None) == qesgd.EINVAL
    assert lib.qesgd_status(None, None) == qesgd.EINVAL
    assert lib.qesgd_launch_count(None) == 0
    assert lib.qesgd_strerror(0) == b"ok"
    assert b"invalid" in lib.qesgd_strerror(qesgd.EINVAL)
    assert lib.qesgd_create(None, 0, None) == qesgd.EINVAL
    assert lib.qesgd_set_wait_limit(None, 1000) == qesgd.EINVAL
    assert lib.qesgd_debug_drop_signal(None, 0) == qesgd.EINVAL


def test_create_without_a_device_fails_cleanly(qesgd):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    handle = C.c_void_p()
    rc = qesgd.lib.qesgd_create(C.byref(handle), 0, None)
    assert rc in (qesgd.ECUDA, qesgd.EINVAL) and not handle.value
