"""The C-ABI library loads without a GPU and exports every function include/gdn.h declares;
host-side argument validation rejects bad calls before any CUDA work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gdn.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2607_17979_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gdn_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for n in ("gdn_decode", "gdn_prefill", "gdn_prefill_workspace_bytes", "gdn_status_string",
              "gdn_version"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    for n in declared_functions():
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2607_17979_b200 import api
    assert set(declared_functions()) <= set(api.EXPORTS) | {n for n in dir(api) if n.startswith("gdn_")}


def test_status_strings_and_version(lib):
    lib.gdn_status_string.restype = ctypes.c_char_p
    assert lib.gdn_status_string(0) == b"ok"
    for code in range(-7, 0):
        assert lib.gdn_status_string(code) not in (b"", b"ok", b"unknown status")
    assert lib.gdn_status_string(-99) == b"unknown status"
    assert lib.gdn_version() >= 100


def _decode(lib, ptr=0x1000, B=1, Hqk=1, Hv=1, dk=128, dv=128, slots=1, null=None, mis=None):
    P = ctypes.c_void_p
    args = [P(ptr)] * 8
    if null is not None:
        args[null] = P(0)
    if mis is not None:
        args[mis] = P(ptr + 8)
    lib.gdn_decode.argtypes = [P] * 8 + [ctypes.c_int32] * 6 + [ctypes.c_float, P, P]
    return lib.gdn_decode(*args, B, Hqk, Hv, dk, dv, slots, 1.0, P(0), P(0))


def test_decode_validation_rejects_before_launch(lib):
    assert _decode(lib, B=0) == 0                       # empty batch: no-op
    assert _decode(lib, B=-1) == -2
    assert _decode(lib, slots=0) == -2
    assert _decode(lib, dk=64) == -3
    assert _decode(lib, Hqk=3, Hv=4) == -3
    assert _decode(lib, null=0) == -1
    assert _decode(lib, null=5) == -1                   # state pool
    assert _decode(lib, mis=7) == -4                    # o misaligned
    assert _decode(lib, null=6) != -1                   # slot_idx may be NULL (rejected later or ok)


def test_prefill_validation_rejects_before_launch(lib):
    P, I32 = ctypes.c_void_p, ctypes.c_int32
    lib.gdn_prefill.argtypes = [P] * 10 + [I32] * 9 + [ctypes.c_float, P, ctypes.c_size_t, P, P]
    lib.gdn_prefill_workspace_bytes.restype = ctypes.c_size_t
    lib.gdn_prefill_workspace_bytes.argtypes = [I32] * 7

    def call(T=64, N=1, Hqk=1, Hv=1, dk=128, dv=128, chunk=64, slots=1, ws=0x2000, ws_bytes=1 << 40,
             null=None):
        a = [P(0x1000)] * 10
        if null is not None:
            a[null] = P(0)
        return lib.gdn_prefill(*a, T, N, 0, Hqk, Hv, dk, dv, chunk, slots, 1.0, P(ws), ws_bytes,
                               P(0), P(0))

    assert call(T=0) == 0 and call(N=0) == 0
    assert call(T=-5) == -2
    assert call(chunk=32) == -3
    assert call(dv=256) == -3
    assert call(null=1) == -1
    assert call(null=7) == -1                           # final_state
    assert call(ws=0) == -1
    assert call(ws=0x2010) == -4
    need = lib.gdn_prefill_workspace_bytes(64, 1, 1, 1, 128, 128, 64)
    assert need > 0 and call(ws_bytes=need - 1) == -5
    assert lib.gdn_prefill_workspace_bytes(64, 1, 1, 1, 64, 128, 64) == 0


def test_prefill_routing_rules_are_pure_host_arithmetic():
    """gdn_prefill_route needs no GPU: it answers from the shapes and the two device facts it is
    given which variant gdn_prefill would launch."""
    from paper_2607_17979_b200 import api
    r = api.gdn_prefill_route
    assert r(0, 0, 0, 32) == "none" and r(100, 0, 0, 32) == "none"
    # longest sequence (hint, else the bound T) up to 16 tokens: token by token
    assert r(16, 1, 0, 32) == "recurrent" and r(4000, 400, 12, 32) == "recurrent"
    assert r(17, 1, 0, 32) != "recurrent" and r(4000, 400, 17, 8) != "recurrent"
    # a hint larger than T is ignored
    assert r(10, 1, 5000, 32) == "recurrent"
    # few long units: one cooperative launch, if the device can
    assert r(32768, 1, 0, 32) == "fused" and r(32768, 1, 0, 32, 148, False) == "stream"
    assert r(1025, 1, 0, 32) == "fused" and r(1024, 1, 0, 32) == "stream"
    assert r(32768, 1, 0, 49) == "fused" and r(32768, 1, 0, 50) == "stream"       # 148 // 3 = 49 units
    # everything else that is chunked: the three launches with the persistent state pass
    assert r(7680, 4, 0, 32) == "stream" and r(129, 1, 0, 32) == "stream"
    assert r(128, 1, 0, 32) == "stream" and r(400, 4, 100, 32) == "stream"
    assert r(1600, 16, 100, 4) == "stream" and r(1700, 17, 100, 4) == "stream"
    assert r(8192, 128, 64, 32) == "stream" and r(296, 37, 8, 4) == "recurrent"
    assert r(1184, 37, 32, 4) == "stream" and r(1216, 38, 32, 4) == "stream"
    # the caller says how long the longest sequence is, chains of at least 40 chunks, more units
    # than the cooperative launch takes and at most half as many as SMs: the two-part production
    assert r(8192, 2, 4096, 32) == "overlap" and r(4000, 2, 3000, 32) == "overlap"
    assert r(8192, 2, 0, 32) == "stream" and r(5118, 2, 2559, 32) == "stream"
    assert r(8192, 2, 4096, 37) == "overlap" and r(8192, 2, 4096, 38) == "stream"   # 74 / 76 units
    assert r(8192, 2, 4096, 24) == "fused" and r(8192, 2, 4096, 25) == "overlap"    # 48 / 50 units
    assert r(7680, 4, 4096, 32) == "stream" and r(6144, 3, 2048, 32) == "stream"
    # the thresholds follow the SM count given
    assert r(1184, 37, 32, 4, 100) == "stream"
