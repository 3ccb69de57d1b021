"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2609_24433_b200 import build as fq_build
from paper_2609_24433_b200 import fq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fq_build.build()
    return fq.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fq_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_list_the_same_entry_points():
    assert declared_symbols() == sorted(fq.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_status_strings(lib):
    seen = {fq.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert fq.status_string(99) == "unknown status"


def test_workspace_bytes_is_a_host_computation(lib):
    assert fq.workspace_bytes(0, 1024, 1024, 4) == 256
    w = fq.workspace_bytes(816, 2048, 2560, 4)
    assert w >= 816 * 2048 + 4 * 816 and w % 256 == 0
    assert fq.workspace_bytes(64, 1024, 1024, 8) >= 64 * 1024


def test_argument_checks_run_before_any_device_work(lib):
    out = ctypes.c_void_p()
    null = ctypes.c_void_p(0)
    i64 = ctypes.c_int64

    def fold(N, K, ldw, block, bits):
        return lib.fq_fold_weights(null, 0, i64(N), i64(K), i64(ldw), null, null, block, bits, null, ctypes.byref(out))

    assert fold(8, 1024, 1024, 128, 5) == fq.ERR_INVALID_ARG          # bits
    assert fold(-8, 1024, 1024, 128, 4) == fq.ERR_INVALID_ARG         # negative size
    assert fold(8, 1024, 1024, 96, 4) == fq.ERR_UNSUPPORTED           # block not a power of two
    assert fold(8, 1024, 1024, 512, 4) == fq.ERR_UNSUPPORTED          # block too large
    assert fold(8, 1056, 1056, 64, 4) == fq.ERR_UNSUPPORTED           # block does not divide K
    assert fold(8, 48, 48, 16, 4) == fq.ERR_UNSUPPORTED               # K not a multiple of 32
    assert fold(12, 1024, 1024, 128, 4) == fq.ERR_UNSUPPORTED         # N not a multiple of 8
    assert fold(8, 262144, 262144, 128, 8) == fq.ERR_UNSUPPORTED      # accumulator bound
    assert fold(8, 1024, 1024, 128, 4) == fq.ERR_INVALID_ARG          # NULL weights
    assert lib.fq_fold_weights(null, 0, i64(8), i64(1024), i64(1024), null, null, 128, 4, null, null) == fq.ERR_INVALID_ARG

    def quant(M, K, block, bits, clip):
        return lib.fq_quantize_act(null, 0, i64(M), i64(K), i64(K), null, block, bits, ctypes.c_float(clip), null,
                                   null, null)

    assert quant(4, 1024, 128, 3, 1.0) == fq.ERR_INVALID_ARG
    assert quant(4, 1024, 128, 4, 0.0) == fq.ERR_INVALID_ARG
    assert quant(4, 1024, 128, 4, 1.5) == fq.ERR_INVALID_ARG
    assert quant(4, 1024, 48, 4, 1.0) == fq.ERR_UNSUPPORTED
    assert quant(0, 1024, 128, 4, 1.0) == fq.OK                        # empty batch is a no-op
    assert quant(4, 1024, 128, 4, 1.0) == fq.ERR_INVALID_ARG          # NULL data
    assert lib.fq_gemm_w4a4(null, null, i64(4), null, null, 0, i64(8), null, ctypes.c_size_t(0), null) == fq.ERR_INVALID_ARG
    assert lib.fq_linear_w8a8(null, 0, i64(4), i64(8), null, ctypes.c_float(1.0), null, 0, i64(8), null,
                              ctypes.c_size_t(0), null) == fq.ERR_INVALID_ARG
    assert lib.fq_weights_destroy(null) == fq.OK


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(fq, "_lib", None)
    monkeypatch.setattr(fq, "LIB_PATH", "/nonexistent/libfq_b200.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        fq.lib()
