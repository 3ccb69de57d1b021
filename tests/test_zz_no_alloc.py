"""The workspace-free W4A4 entry point (fq_linear_w4a4_static) against the regular one.

Some callers cannot hand the library a workspace because they cannot allocate device memory
when they call it (a plugin's enqueue callback, a control loop that must not stall on an
allocation, a process whose memory was all given out at start-up).  For them the library keeps
the scratch inside its own image.  This file is collected last on purpose: a run that stops at
the first failure has then already gone through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from helpers import assert_close, to_dev, to_np
from paper_2609_24433_b200 import fq, synth

pytestmark = pytest.mark.gpu


def _site(M, K, N, dtype, seed):
    site = synth.Site("t", M, K, [("p", N)], beta=128, bits=4, x_dtype=dtype, y_dtype=dtype)
    return synth.make_site(site, seed)


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    # two calls in a row through the C ABI: the second is smaller and must not see the first's leftovers
    for M, K, N, dtype, seed in [(816, 2048, 520, "bf16", 1), (50, 1024, 264, "f32", 2)]:
        data = _site(M, K, N, dtype, seed)
        x = to_dev(data.x, dtype)
        h = fq.fold_weights(to_dev(data.W["p"]), None, to_dev(data.bias["p"]), 128, 4)
        ydt = torch.float32 if dtype == "f32" else torch.bfloat16
        want = fq.linear_w4a4(x, h, 1.0, ydt)
        got = torch.full((M + 1, N), 77.0, dtype=ydt, device="cuda")
        fq.linear_w4a4_static(x, h, 1.0, y=got[:M])
        torch.cuda.synchronize()
        assert_close(to_np(got[:M]), to_np(want), dtype, f"static vs workspace, M={M}")
        assert torch.equal(got[:M], want)                  # same kernels, same inputs: identical bits
        assert (got[M] == 77.0).all()                      # rows beyond M untouched
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


def test_static_scratch_rejects_what_does_not_fit_and_bad_arguments():
    K, N = 16384, 264
    W = torch.zeros((N, K), dtype=torch.float32, device="cuda")
    h4 = fq.fold_weights(W, None, None, 256, 4)
    x = torch.zeros((816, K), dtype=torch.bfloat16, device="cuda")       # 816 * 16384 bytes > 4 MiB
    assert 816 * K > fq.STATIC_MAX_CODE_BYTES
    with pytest.raises(fq.FqError) as e:
        fq.linear_w4a4_static(x, h4)
    assert e.value.status == fq.ERR_NOMEM
    y = fq.linear_w4a4_static(x[:256], h4, out_dtype=torch.bfloat16)      # exactly at the limit: accepted
    assert y.shape == (256, N) and not y.any()
    h8 = fq.fold_weights(W[:, :1024].contiguous(), None, None, 128, 8)
    with pytest.raises(fq.FqError) as e:
        fq.linear_w4a4_static(x[:8, :1024], h8)
    assert e.value.status == fq.ERR_UNSUPPORTED
    null = ctypes.c_void_p(0)
    assert fq.lib().fq_linear_w4a4_static(null, 0, ctypes.c_int64(4), ctypes.c_int64(K), h4.handle,
                                          ctypes.c_float(1.0), null, 0, ctypes.c_int64(N), null) == fq.ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_static_scratch_calls_leave_the_device_memory_as_it_was():
    """After the start-up call (zero tokens: it loads the module that holds the scratch), calls of the workspace-free
    entry point take no device memory: the free-memory figure the driver reports is the same before and after."""
    data = _site(200, 1024, 264, "bf16", 3)
    x = to_dev(data.x, "bf16")
    h = fq.fold_weights(to_dev(data.W["p"]), None, to_dev(data.bias["p"]), 128, 4)
    y = torch.empty((200, 264), dtype=torch.bfloat16, device="cuda")
    fq.linear_w4a4_static(x[:0], h, 1.0, y=y[:0])          # start-up call
    fq.linear_w4a4_static(x, h, 1.0, y=y)                  # and one full call, so that every kernel's module is resident
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        fq.linear_w4a4_static(x, h, 1.0, y=y)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert torch.equal(y, fq.linear_w4a4(x, h, 1.0, torch.bfloat16))
