"""CPU-side checks of the C ABI: the library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_03383_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    with open(os.path.join(ROOT, "include", "uniql.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(uniql_[a-z0-9_]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert "uniql_qlinear" in names and "uniql_qk_rope_proj" in names and len(names) >= 11
    for n in names:
        assert hasattr(lib, n), "missing export " + n


def test_status_strings_and_version(lib):
    lib.uniql_status_string.restype = ctypes.c_char_p
    assert lib.uniql_status_string(0) == b"ok"
    assert lib.uniql_status_string(7) == b"device-side wait timed out"
    assert lib.uniql_version() >= 100


def test_argument_errors_are_caught_on_the_host(lib):
    vp = ctypes.c_void_p
    fake = vp(0x10000)         # never dereferenced: every call below must fail validation first
    odd = vp(0x10001)
    ql = lib.uniql_qlinear
    ql.argtypes = [vp, vp, vp, vp] + [ctypes.c_int] * 5 + [vp, vp]
    assert ql(None, fake, fake, fake, 1, 128, 16, 128, 16, fake, None) == 1       # NULL
    assert ql(fake, fake, fake, fake, 1, 100, 16, 100, 16, fake, None) == 2       # K % 128
    assert ql(fake, fake, fake, fake, 0, 128, 16, 128, 16, fake, None) == 2       # M < 1
    assert ql(fake, fake, fake, fake, 1, 128, 16, 256, 16, fake, None) == 2       # k_in > K
    assert ql(fake, fake, fake, fake, 1, 128, 16, 128, 17, fake, None) == 2       # k_out > N
    assert ql(odd, fake, fake, fake, 1, 128, 16, 128, 16, fake, None) == 3        # x misaligned
    assert ql(fake, vp(0x10008), fake, fake, 1, 128, 16, 128, 16, fake, None) == 3  # weights not 16-byte aligned
    assert lib.uniql_set_path(9) == 2
    pk = lib.uniql_pack_u4
    pk.argtypes = [vp, ctypes.c_int64, ctypes.c_int64, vp, vp]
    assert pk(fake, 4, 7, fake, None) == 2
    assert pk(None, 4, 8, fake, None) == 1
    lib.uniql_workspace_bytes.restype = ctypes.c_size_t
    assert lib.uniql_workspace_bytes(1, 4096, 4096) > 0
    assert lib.uniql_workspace_bytes(0, 4096, 4096) == 0
