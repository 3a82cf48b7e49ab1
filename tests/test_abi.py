"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol that
include/fh.h declares, validates arguments, and its size formulas agree with the oracle's."""
import ctypes as C
import os
import re

import pytest

from oracle import fho
from paper_2510_11400_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "fh.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(fh_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.fh_version() == 1


def test_struct_sizes_match_header_layout():
    assert C.sizeof(api.fh_tensor_desc) == 32
    assert C.sizeof(api.fh_params) == 56
    assert C.sizeof(api.fh_sched_entry) == 56
    assert C.sizeof(api.fh_sched_report) == 40


def test_default_params(lib):
    p = api.default_params()
    assert (p.bits, p.salient_mode, p.rho_num, p.rho_den, p.block, p.tau_num, p.tau_den, p.dense_bits,
            p.rounding) == (2, 0, 1, 32, 8, 1, 4, 8, 0)
    assert p.eps == 0.0625


@pytest.mark.parametrize("shape,dtype", [((32, 16, 32, 32), 0), ((2, 3, 7, 7), 1), ((64, 64, 112, 112), 0),
                                         ((1, 1, 1, 1), 0), ((5, 9, 13, 3), 1)])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_size_formulas_agree_with_oracle(lib, shape, dtype, bits):
    for which in (0, 1):
        a = api.compressed_bytes(api.desc(shape, dtype), api.default_params(bits=bits), which)
        b = fho.compressed_bytes(fho.desc(shape, dtype), fho.params(bits=bits), which)
        assert a == b > 0
    assert api.compressed_bytes(api.desc((32, 16, 32, 32)), api.default_params(bits=2), 0) == 139328


def test_argument_errors_are_returned_before_any_cuda_call(lib):
    d = api.desc((1, 2, 8, 8))
    p = api.default_params()
    buf = (C.c_uint8 * 4096)()
    addr = (C.addressof(buf) + 255) & ~255
    # bad parameters
    assert lib.fh_compress(C.byref(d), C.byref(api.default_params(bits=3)), addr, addr, 4096, None, None) == api.FH_ERR_UNSUPPORTED
    assert lib.fh_compress(C.byref(d), C.byref(api.default_params(eps=0.0)), addr, addr, 4096, None, None) == api.FH_ERR_ARG
    assert lib.fh_compress(C.byref(d), C.byref(api.default_params(block=4)), addr, addr, 4096, None, None) == api.FH_ERR_UNSUPPORTED
    assert lib.fh_compress(C.byref(d), C.byref(api.default_params(rounding=2)), addr, addr, 4096, None, None) == api.FH_ERR_UNSUPPORTED
    # bad tensor
    assert lib.fh_compress(C.byref(api.desc((1, 0, 8, 8))), C.byref(p), addr, addr, 4096, None, None) == api.FH_ERR_ARG
    assert lib.fh_compress(C.byref(api.desc((1, 1, 1, 70000))), C.byref(p), addr, addr, 4096, None, None) == api.FH_ERR_UNSUPPORTED
    assert lib.fh_compress(C.byref(api.desc((1, 1, 8, 8), 7)), C.byref(p), addr, addr, 4096, None, None) == api.FH_ERR_ARG
    # null / misaligned pointers, capacity below header + table
    assert lib.fh_compress(C.byref(d), C.byref(p), None, addr, 4096, None, None) == api.FH_ERR_ARG
    assert lib.fh_compress(C.byref(d), C.byref(p), addr + 4, addr, 4096, None, None) == api.FH_ERR_ARG
    assert lib.fh_compress(C.byref(d), C.byref(p), addr, addr, 64 + 16 * 2 - 1, None, None) == api.FH_ERR_CAPACITY
    assert lib.fh_decompress(None, 100, C.byref(d), addr, None, None) == api.FH_ERR_ARG
    assert lib.fh_decompress(addr, 100, C.byref(api.desc((0, 1, 1, 1))), addr, None, None) == api.FH_ERR_ARG
    assert api.compressed_bytes(api.desc((1, 0, 8, 8)), p) == 0
    rep = api.fh_sched_report()
    assert lib.fh_run_schedule(None, 1, C.byref(p), addr, 4096, C.byref(rep), None) == api.FH_ERR_ARG


def test_planes_too_large_for_shared_memory_are_unsupported(lib):
    d = api.desc((1, 1, 512, 512))
    buf = (C.c_uint8 * 4096)()
    addr = (C.addressof(buf) + 255) & ~255
    assert lib.fh_compress(C.byref(d), C.byref(api.default_params()), addr, addr, 4096, None, None) == api.FH_ERR_UNSUPPORTED


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        api.lib()
