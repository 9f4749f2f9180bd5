"""Host-side checks of the C-ABI library that need no GPU: the library loads,
exports every function the header declares, and rejects bad layer descriptions
before touching a device (Algorithm 1's reject list turned into status codes)."""
import ctypes
import os
import re

import pytest

import paper_2609_31938_b200 as ccv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "ccv3d.h")


def _declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ccv3d_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_function():
    names = _declared_functions()
    assert "ccv3d_create" in names and "ccv3d_forward" in names and "ccv3d_destroy" in names
    lib = ctypes.CDLL(ccv._build.LIB)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in ccv3d.h but not exported"
    assert set(names) == set(ccv.EXPORTS)


def test_struct_layouts_match_the_header():
    # ccv3d_desc: 12 scalars + two int32[3] = 18 x 4 bytes; ccv3d_counters: 11 x uint64
    assert ctypes.sizeof(ccv.Desc) == 18 * 4
    assert ctypes.sizeof(ccv.Counters) == 11 * 8
    src = open(HEADER).read()
    body = src[src.index("typedef struct {", src.index("Layer description")):src.index("} ccv3d_desc;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b([a-z_]+)\b(?=(?:\[3\])?[,;])", body)
    assert fields == [f for f, _ in ccv.Desc._fields_]


def test_status_strings():
    assert ccv.status_string(ccv.OK) == "CCV3D_OK"
    assert ccv.status_string(ccv.ERR_DEVICE_TIMEOUT) == "CCV3D_ERR_DEVICE_TIMEOUT"
    assert ccv.status_string(1234) == "CCV3D_ERR_UNKNOWN"
    src = open(HEADER).read()
    for i, name in enumerate(re.findall(r"\b(CCV3D_(?:OK|ERR_[A-Z_]+)) = (\d+)", src)):
        assert ccv.status_string(int(name[1])) == name[0]


@pytest.mark.parametrize("kwargs,expected", [
    (dict(stride=(9, 1, 1)), ccv.ERR_UNSUPPORTED),
    (dict(stride=(1, 9, 1)), ccv.ERR_UNSUPPORTED),       # beyond what a TMA traversal stride can express
    (dict(stride=(1, 0, 1)), ccv.ERR_INVALID_ARG),
    (dict(dilation=(1, 0, 1)), ccv.ERR_INVALID_ARG),
    (dict(dilation=(9, 1, 1)), ccv.ERR_UNSUPPORTED),
    (dict(groups=2), ccv.ERR_UNSUPPORTED),               # groups != 1 (Algorithm 1, validation)
    (dict(k=(3, 9, 9)), ccv.ERR_UNSUPPORTED),
    (dict(pad=(1, -1, 1)), ccv.ERR_INVALID_ARG),
    (dict(pad=(1, 40, 1)), ccv.ERR_UNSUPPORTED),
    (dict(pad=(0, 1, 1)), ccv.ERR_UNSUPPORTED),          # temporal padding that is not the causal total 2 pad_t = d_t (kt-1)
    (dict(dilation=(2, 1, 1), pad=(1, 1, 1)), ccv.ERR_UNSUPPORTED),
    (dict(dtype=ccv.F32, out_dtype=ccv.BF16), ccv.ERR_UNSUPPORTED),
    (dict(dtype=7), ccv.ERR_INVALID_ARG),
    (dict(cin=0), ccv.ERR_INVALID_ARG),
    (dict(cout=-3), ccv.ERR_INVALID_ARG),
])
def test_create_rejects_bad_descriptions_on_the_host(kwargs, expected):
    base = dict(cin=16, cout=16)
    base.update(kwargs)
    d = ccv.make_desc(base.pop("cin"), base.pop("cout"), **base)
    s, h = ccv.ccv3d_create(d, 4096, None)     # the fake weight address is never dereferenced: validation comes first
    assert s == expected and h is None


def test_null_and_misaligned_arguments():
    d = ccv.make_desc(16, 16)
    assert ccv.ccv3d_create(d, None, None)[0] == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_create(d, 4100, None)[0] == ccv.ERR_ALIGNMENT
    assert ccv.lib.ccv3d_create(None, ctypes.byref(d), 4096, None, None) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_destroy(None) == ccv.OK
    assert ccv.ccv3d_forward(None, 4096, None, 8192, None, 1, 1, 8, 8) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_forward_host(None, 4096, None, 8192, None, 1, 1, 8, 8) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_forward_host_stream(None, 4096, 8192, 1, 1, 1, 8, 8) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_rows_copy(None, 4, 0, 4096, 4, 0, 1, 1, 16) == ccv.ERR_INVALID_ARG          # no destination
    assert ccv.ccv3d_rows_copy(4096, 4, 3, 8192, 4, 0, 1, 2, 16) == ccv.ERR_INVALID_ARG          # rows leave the plane
    assert ccv.ccv3d_workspace_bytes(None, 1, 1, 8, 8)[0] == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_set_workspace(None, 4096, 1 << 20) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_device_status(None)[0] == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_add_bf16(None, None, None, 16) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_upsample_bf16(None, None, 1, 1, 1, 1, 1, 1) == ccv.ERR_INVALID_ARG
    with pytest.raises(ccv.Ccv3dError):
        ccv.ccv3d_get_counters(None)


def test_ring_geometry_and_argument_checks_need_no_device():
    """Frame rings: the block-size rule, the byte count, and every rejection that happens before a launch."""
    assert [ccv.ccv3d_ring_kb(c) for c in (0, 16, 32, 64, 96, 100, 192, 384)] == [0, 0, 32, 64, 32, 0, 64, 64]
    assert ctypes.sizeof(ccv.Ring) == 8 + 6 * 4
    r = ccv.Ring(4096, 2, 96, 5, 7, 9, 32)
    assert ccv.ccv3d_ring_bytes(r) == 2 * 5 * 96 * 7 * 9 * 2
    assert ccv.ccv3d_ring_bytes(ccv.Ring(4096, 1, 96, 5, 7, 9, 64)) == 0          # 96 channels do not split into 64s
    assert ccv.ccv3d_ring_bytes(ccv.Ring(4096, 1, 64, 0, 7, 9, 64)) == 0
    big = ccv.Ring(1 << 20, 1, 64, 4, 8, 8, 64)
    assert ccv.ccv3d_ring_load(big, 0, None, 1) == ccv.ERR_INVALID_ARG             # no source
    assert ccv.ccv3d_ring_load(big, 4, 1 << 24, 1) == ccv.ERR_INVALID_ARG          # slot out of range
    assert ccv.ccv3d_ring_load(big, 0, 1 << 24, 5) == ccv.ERR_INVALID_ARG          # more frames than slots
    assert ccv.ccv3d_ring_load(big, 0, (1 << 24) + 4, 1) == ccv.ERR_ALIGNMENT
    assert ccv.ccv3d_ring_load(big, 0, (1 << 20) + 256, 1) == ccv.ERR_ALIAS        # source inside the ring
    assert ccv.ccv3d_ring_store(ccv.Ring(None, 1, 64, 4, 8, 8, 64), 0, 1 << 24, 1) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_ring_store(big, 0, (1 << 20) + 256, 1) == ccv.ERR_ALIAS
    twice = ccv.Ring(1 << 26, 1, 64, 4, 16, 16, 64)
    assert ccv.ccv3d_upsample_ring(big, 0, twice, 0, 2, 3) == ccv.ERR_INVALID_ARG  # 2 x 3 frames > 4 slots
    assert ccv.ccv3d_upsample_ring(big, 0, big, 0, 1, 1) == ccv.ERR_INVALID_ARG    # not twice the size
    assert ccv.ccv3d_upsample_ring(big, 0, ccv.Ring(1 << 26, 1, 32, 4, 16, 16, 32), 0, 1, 1) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_forward_ring(None, big, 0, 0, None, 0, twice, 0, None, 1) == ccv.ERR_INVALID_ARG
