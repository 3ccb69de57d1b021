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


def test_planner_splits_k_only_where_it_measured_faster(lib):
    """The workspace a shape asks for tells whether the planner would split K (scratch for the partial sums beyond the
    codes and steps).  On operands from HBM a split costs a call 16-25 thousand cycles, so short batches on square
    matrices and the backbone's sites run unsplit; a few tiles on a very long K still split.  (Without a device the
    planner assumes 148 SMs.)"""
    def base(M, K):
        return (M * K + 255) // 256 * 256 + (4 * M + 255) // 256 * 256

    for M, K, N, bits in [(64, 4096, 4096, 8), (50, 4096, 1024, 8), (16, 8192, 8192, 8), (50, 4096, 1024, 4),
                          (816, 16384, 2048, 8), (816, 2048, 32768, 4), (16384, 8192, 8192, 4)]:
        assert fq.workspace_bytes(M, K, N, bits) == base(M, K), (M, K, N, bits)
    for M, K, N, bits in [(50, 16384, 1024, 8), (100, 16384, 256, 4), (208, 16384, 384, 8)]:
        assert fq.workspace_bytes(M, K, N, bits) > base(M, K), (M, K, N, bits)


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


def test_argument_checks_of_the_widened_entry_points(lib):
    out = ctypes.c_void_p()
    null = ctypes.c_void_p(0)
    i64 = ctypes.c_int64
    f32 = ctypes.c_float
    # weight-only projection: a NULL handle, a negative batch
    assert lib.fq_linear_w4a16(null, 0, i64(1), i64(1024), null, null, 0, i64(8), null) == fq.ERR_INVALID_ARG
    # block 1 is the identity rotation and a legal block everywhere (NULL data is what is refused here)
    assert lib.fq_fold_weights(null, 0, i64(8), i64(1024), i64(1024), null, null, 1, 4, null, ctypes.byref(out)) == fq.ERR_INVALID_ARG
    assert lib.fq_quantize_act(null, 0, i64(0), i64(1024), i64(1024), null, 1, 4, f32(1.0), null, null, null) == fq.OK

    def fold_c(K, block, perm, blocks):
        return lib.fq_fold_weights_composite(null, 0, i64(8), i64(K), i64(K), null, null, perm, blocks, block, 4, null,
                                             ctypes.byref(out))

    one = ctypes.c_void_p(16)           # any non-NULL address: the checks below return before it is touched
    assert fold_c(1024, 8, one, one) == fq.ERR_UNSUPPORTED           # stored blocks below 16 channels
    assert fold_c(1024, 48, one, one) == fq.ERR_UNSUPPORTED
    assert fold_c(1024, 64, null, one) == fq.ERR_INVALID_ARG         # no permutation
    assert fold_c(1024, 64, one, null) == fq.ERR_INVALID_ARG         # no matrices

    def quant_c(M, K, block, ws_bytes):
        return lib.fq_quantize_act_composite(one, 0, i64(M), i64(K), i64(K), null, one, one, block, 4, f32(1.0), one, one,
                                             one, ctypes.c_size_t(ws_bytes), null)

    assert quant_c(0, 1024, 64, 0) == fq.OK                          # empty batch
    assert quant_c(4, 1024, 8, 1 << 20) == fq.ERR_UNSUPPORTED
    assert quant_c(4, 1024, 64, 4 * 4 * 1024 - 1) == fq.ERR_NOMEM     # scratch for the rotated rows too small

    def gptq(K, Mc, calib, damp):
        return lib.fq_fold_weights_gptq(one, 0, i64(8), i64(K), i64(K), null, null, calib, 0, i64(Mc), i64(K), 64, 4,
                                        f32(damp), null, ctypes.byref(out))

    assert gptq(32768, 16, one, 0.01) == fq.ERR_UNSUPPORTED           # K beyond the factorisation's limit
    assert gptq(1024, 16, null, 0.01) == fq.ERR_INVALID_ARG           # no calibration tokens
    assert gptq(1024, 0, one, 0.01) == fq.ERR_INVALID_ARG
    assert gptq(1024, 16, one, -1.0) == fq.ERR_INVALID_ARG
    assert lib.fq_weights_composite(null) == 0


def test_reference_arm_lines_of_the_extra_workloads():
    """`bench.py --impl reference` runs on the host alone; its JSON line keeps the contract's keys."""
    import json
    import subprocess
    import sys
    for workload in ("w4a16:1,256,64", "gptq:16,128,64,32"):
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", workload,
                            "--steps", "1"], capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr[-500:]
        line = json.loads(r.stdout.strip().splitlines()[-1])
        for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                    "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline", "impl"):
            assert key in line, (workload, key)
        assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(fq, "_lib", None)
    monkeypatch.setattr(fq, "LIB_PATH", "/nonexistent/libfq_b200.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        fq.lib()
