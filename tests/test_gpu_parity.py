"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer stages (packed codes, per-token steps, folded weight codes and scales,
int32 accumulators) must match bit for bit; floating-point outputs within 1e-3 (fp32) or
1e-2 (bf16) relative."""
import numpy as np
import pytest
import torch

import oracle
from helpers import as_f64, assert_close, concat_consumers, oracle_smooth, to_dev, to_np
from paper_2609_24433_b200 import fq, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _watchdog_clean():
    yield
    st, word = fq.device_status()
    assert st == fq.OK, f"device wait watchdog fired: {word:#x}"


def fused_workspace(ws: torch.Tensor, M: int, K: int, bits: int):
    """What the one-call entry points leave in the caller's workspace between their two kernels: the
    activation codes as one int8 per code ([M, K]; at 4 bits every group of 8 channels is stored even
    channels first: c0 c2 c4 c6 c1 c3 c5 c7) and, 256-byte aligned behind them, the per-token steps.
    Returns (codes [M, K] int32 in natural channel order, steps as uint32 bit patterns)."""
    raw = ws[:M * K].view(torch.int8).view(M, K).cpu().numpy().astype(np.int32)
    if bits == 4:
        g = raw.reshape(M, K // 8, 8)
        nat = np.empty_like(g)
        nat[:, :, 0::2] = g[:, :, 0:4]
        nat[:, :, 1::2] = g[:, :, 4:8]
        raw = nat.reshape(M, K)
    off = (M * K + 255) // 256 * 256
    delta = ws[off:off + 4 * M].view(torch.float32).cpu().numpy()
    return raw, delta.view(np.uint32)


def assert_fused_stages(x_dev, h, clip, ydt, want_codes, want_delta, what=""):
    """The one-call path (its own prologue instantiations: int8 codes in the GEMM's channel order) against the
    oracle's codes and steps bit for bit, and its output against the two-call route bit for bit: the same
    integer sums scaled by an exact power of two, so nothing may differ."""
    M, K = x_dev.shape
    ws = torch.zeros(fq.workspace_bytes(M, h.K, h.N, h.bits), dtype=torch.uint8, device="cuda")
    y = fq.linear(x_dev, h, clip, ydt, workspace=ws)
    codes, delta = fused_workspace(ws, M, K, h.bits)
    assert np.array_equal(delta, want_delta.view(np.uint32)), f"{what}: fused steps differ"
    assert np.array_equal(codes, oracle.unpack(want_codes, K, h.bits)), f"{what}: fused codes differ"
    c2, d2 = fq.quantize_act(x_dev, h, h.block, h.bits, clip)
    y2 = (fq.gemm_w4a4 if h.bits == 4 else fq.gemm_w8a8)(c2, d2, h, ydt)
    assert torch.equal(y, y2), f"{what}: one-call and two-call outputs differ"
    return y


def make_x(M, K, dtype, seed, frac=0.01):
    site = synth.Site("t", M, K, [("p", 8)], beta=32, bits=4, x_dtype=dtype, outlier_frac=frac)
    return synth.make_site(site, seed, with_weights=False).x


# ----------------------------------------------------------------- prologue ----
ACT_CASES = [
    # M, K, block, bits, dtype, smooth, clip
    (64, 1024, 128, 4, "f32", True, 1.0),
    (50, 1024, 64, 4, "bf16", False, 1.0),
    (50, 4096, 64, 4, "bf16", False, 1.0),
    (816, 2048, 128, 4, "bf16", True, 1.0),
    (816, 2048, 128, 8, "bf16", False, 1.0),
    (203, 16384, 256, 8, "bf16", False, 1.0),
    (131, 16384, 256, 4, "f32", True, 0.8),
    (5, 32, 32, 4, "f32", False, 1.0),
    (3, 64, 2, 8, "bf16", False, 1.0),
    (9, 96, 32, 4, "bf16", True, 1.0),
    (33, 256, 4, 4, "f32", False, 1.0),
    (33, 512, 8, 8, "bf16", False, 0.5),
    (17, 3072, 16, 4, "bf16", False, 1.0),
    (7, 3072, 128, 8, "f32", True, 0.9),
    (300, 8192, 32, 4, "bf16", False, 1.0),
    (19, 8192, 256, 8, "f32", False, 1.0),
    (4, 32768, 256, 4, "bf16", True, 1.0),
    (3, 32768, 64, 8, "f32", False, 0.75),
    (1, 2048, 128, 4, "bf16", False, 1.0),
    (2500, 1024, 64, 4, "bf16", False, 1.0),
    (600, 2048, 128, 4, "f32", True, 0.8),
    (400, 4096, 256, 8, "f32", False, 1.0),
    (333, 3072, 128, 4, "bf16", True, 1.0),
    (1000, 16384, 256, 4, "bf16", True, 1.0),
    (700, 8192, 32, 8, "bf16", False, 0.6),
    # identity rotation (block 1): scale-only sites
    (64, 1024, 1, 4, "f32", True, 1.0),
    (816, 2048, 1, 8, "bf16", False, 1.0),
    (300, 8192, 1, 4, "bf16", True, 0.8),
    (2500, 1024, 1, 4, "bf16", False, 1.0),
]


@pytest.mark.parametrize("M,K,block,bits,dtype,smooth,clip", ACT_CASES)
def test_quantize_act_bit_exact(M, K, block, bits, dtype, smooth, clip):
    x = make_x(M, K, dtype, seed=M + K + block)
    rng = np.random.default_rng(K)
    s = np.exp(rng.uniform(-2, 2, K)).astype(np.float32) if smooth else None
    g = oracle.multiplier(s, K, block, False) if smooth else None
    want_codes, want_delta = oracle.quantize_act(x, dtype, g, block, bits, clip)
    codes, delta = fq.quantize_act(to_dev(x, dtype), to_dev(g), block, bits, clip)
    assert np.array_equal(to_np(delta).view(np.uint32), want_delta.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)


@pytest.mark.parametrize("bits", [4, 8])
def test_quantize_act_zero_tiny_and_strided_rows(bits):
    M, K, block = 37, 1024, 128
    x = make_x(M, K, "f32", seed=1).copy()
    x[3] = 0.0
    x[11] = np.float32(1e-42)
    x[20] = np.float32(-3e-39)
    want_codes, want_delta = oracle.quantize_act(x, "f32", None, block, bits)
    assert want_delta[3] == 0 and want_delta[11] == 0
    wide = torch.full((M, K + 64), 7.0, dtype=torch.float32, device="cuda")   # leading dimension > K
    wide[:, :K] = to_dev(x)
    codes = torch.full((M + 1, K * bits // 8), 0xAB, dtype=torch.uint8, device="cuda")
    delta = torch.full((M + 1,), -1.0, dtype=torch.float32, device="cuda")
    fq.quantize_act(wide[:, :K], None, block, bits, 1.0, codes=codes[:M], delta=delta[:M])
    assert np.array_equal(to_np(codes[:M]), want_codes)
    assert np.array_equal(to_np(delta[:M]).view(np.uint32), want_delta.view(np.uint32))
    assert (codes[M] == 0xAB).all() and delta[M] == -1.0      # nothing written past row M


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("M,K,dtype", [(40, 1024, "f32"), (600, 2048, "bf16"), (700, 4096, "f32"), (333, 1024, "bf16"),
                                       (1200, 2048, "bf16"), (1300, 4096, "f32"), (300, 8192, "bf16")])
def test_quantize_act_exact_ties_round_to_even(bits, M, K, dtype):
    """Every scaled value is an exact half-integer: a fused multiply-add or a different tie rule in
    any kernel variant (register kernel for short batches, streaming kernel for long ones) shows up
    in thousands of codes.  One-hot inputs per 32-channel block give z = +-a on the whole block; one
    block per token carries 2q so that the step is exactly 2 and z/2 is a tie for odd a."""
    q = 7 if bits == 4 else 127
    rng = np.random.default_rng(M + K + bits)
    nb = K // 32
    a = 2 * rng.integers(0, q, size=(M, nb)) + 1                  # odd amplitudes below 2q
    a[np.arange(M), rng.integers(0, nb, size=M)] = 2 * q          # sets max|z| = 2q  ->  step 2
    x = np.zeros((M, K), np.float32)
    pos = rng.integers(0, 32, size=(M, nb))
    x[np.arange(M)[:, None], np.arange(nb)[None, :] * 32 + pos] = a
    xs = synth.as_dtype(x, dtype)                                  # small integers: exact in bf16
    g = np.ones(K, np.float32)
    want_codes, want_delta = oracle.quantize_act(xs, dtype, g, 32, bits)
    assert np.all(want_delta == 2.0)
    c = oracle.unpack(want_codes, K, bits)
    assert np.all((np.abs(c) % 2 == 0) | (np.abs(c) == q))        # ties went to even
    codes, delta = fq.quantize_act(to_dev(xs, dtype), to_dev(g), 32, bits)
    assert np.array_equal(to_np(delta), want_delta)
    assert np.array_equal(to_np(codes), want_codes)
    # the same ties through the one-call path, whose prologue instantiations (int8 codes in the GEMM's channel
    # order) are compiled separately from the canonical-format ones above
    wq = rng.integers(-q, q + 1, size=(8, K)).astype(np.int32)
    h = fq.weights_import(to_dev(oracle.pack(wq, bits)), to_dev(np.ones(8, np.float32)), to_dev(g), None, K, 32, bits)
    assert_fused_stages(to_dev(xs, dtype), h, 1.0, torch.float32, want_codes, want_delta, "exact ties")


def test_quantize_act_amplitude_invariance_on_device():
    x = make_x(64, 2048, "f32", seed=4)
    c0, d0 = fq.quantize_act(to_dev(x), None, 64, 4)
    for k in (-7, 5):
        c1, d1 = fq.quantize_act(to_dev(x * np.float32(2.0 ** k)), None, 64, 4)
        assert torch.equal(c0, c1) and torch.equal(d1, d0 * (2.0 ** k))


def test_quantize_act_empty_batch():
    x = torch.empty((0, 1024), dtype=torch.bfloat16, device="cuda")
    codes, delta = fq.quantize_act(x, None, 128, 4)
    assert codes.shape == (0, 512) and delta.shape == (0,)


# --------------------------------------------------------------------- fold ----
FOLD_CASES = [
    # N, K, block, bits, wdtype, smooth
    (1024, 1024, 128, 4, "f32", True),
    (256, 2048, 128, 8, "f32", False),
    (264, 4096, 64, 4, "bf16", True),
    (8, 32, 32, 4, "f32", False),
    (24, 16384, 256, 8, "bf16", False),
    (16, 16384, 256, 4, "f32", True),
    (40, 96, 32, 8, "f32", True),
    (264, 1536, 1, 4, "bf16", False),       # identity transform: plain RTN of W
    (64, 2048, 1, 8, "f32", True),
]


@pytest.mark.parametrize("N,K,block,bits,wdtype,smooth", FOLD_CASES)
def test_fold_weights_bit_exact(N, K, block, bits, wdtype, smooth):
    rng = np.random.default_rng(N + K)
    W = synth.as_dtype(synth.draw_weights(rng, N, K), wdtype)
    if N > 2:
        W[2] = 0                                                   # zero output channel
    bias = rng.standard_normal(N).astype(np.float32)
    s = np.exp(rng.uniform(-2, 2, K)).astype(np.float32) if smooth else None
    want_codes, want_scale, want_g = oracle.fold_weights(W, wdtype, s, block, bits)
    h = fq.fold_weights(to_dev(W, wdtype), to_dev(s), to_dev(bias), block, bits)
    assert (h.N, h.K, h.block, h.bits) == (N, K, block, bits)
    codes, scale, g, b = h.export()
    assert np.array_equal(to_np(g).view(np.uint32), want_g.view(np.uint32))
    assert np.array_equal(to_np(scale).view(np.uint32), want_scale.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)
    assert np.array_equal(to_np(b), bias)
    # import of the exported pack behaves like the original handle
    h2 = fq.weights_import(codes, scale, g, b, K, block, bits)
    c2, s2, g2, b2 = h2.export()
    assert torch.equal(c2, codes) and torch.equal(s2, scale) and torch.equal(g2, g) and torch.equal(b2, b)


# ------------------------------------------------- fold-after variant (T = P^-1 R) ----
AFTER_CASES = [
    # M, K, block, bits, dtype, clip      (register kernel: short batches / small K; ring kernel: the rest)
    (50, 1024, 64, 4, "bf16", 1.0),
    (64, 1024, 128, 4, "f32", 1.0),
    (9, 96, 32, 8, "bf16", 0.9),
    (33, 512, 8, 8, "f32", 1.0),
    (131, 16384, 256, 4, "f32", 0.8),
    (816, 2048, 128, 4, "bf16", 1.0),
    (816, 2048, 128, 8, "bf16", 1.0),
    (600, 4096, 64, 8, "f32", 1.0),
    (1000, 16384, 256, 8, "bf16", 1.0),
    (700, 8192, 32, 4, "bf16", 0.6),
    (333, 3072, 128, 4, "bf16", 1.0),
]


@pytest.mark.parametrize("M,K,block,bits,dtype,clip", AFTER_CASES)
def test_quantize_act_after_bit_exact(M, K, block, bits, dtype, clip):
    x = make_x(M, K, dtype, seed=M + K + block + 1)
    rng = np.random.default_rng(K + 1)
    gpost = (np.float32(1.0) / np.exp(rng.uniform(-2, 2, K)).astype(np.float32)).astype(np.float32)
    want_codes, want_delta = oracle.quantize_act_after(x, dtype, gpost, block, bits, clip)
    codes, delta = fq.quantize_act(to_dev(x, dtype), to_dev(gpost), block, bits, clip, fold_after=True)
    assert np.array_equal(to_np(delta).view(np.uint32), want_delta.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)
    # the same vector ahead of the rotation is a different transform: the flag must matter
    other, _ = fq.quantize_act(to_dev(x, dtype), to_dev(gpost), block, bits, clip, fold_after=False)
    assert not torch.equal(other, codes)


@pytest.mark.parametrize("N,K,block,bits,wdtype", [(40, 1024, 128, 4, "f32"), (136, 2048, 64, 8, "bf16"),
                                                    (304, 4096, 256, 4, "f32"), (24, 96, 32, 8, "f32")])
def test_fold_weights_after_bit_exact_and_linear(N, K, block, bits, wdtype):
    rng = np.random.default_rng(N + K)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    if wdtype == "bf16":
        W = synth.f32_to_bf16_bits(W)
    bias = (rng.standard_normal(N) * 0.02).astype(np.float32)
    p = np.exp(rng.uniform(-1.5, 1.5, K)).astype(np.float32)
    want_codes, want_scale, want_g = oracle.fold_weights_after(W, wdtype, p, block, bits)
    h = fq.fold_weights_after(to_dev(W, wdtype), to_dev(p), to_dev(bias), block, bits)
    assert h.fold_after and (h.N, h.K, h.block, h.bits) == (N, K, block, bits)
    codes, scale, g, b = h.export()
    assert np.array_equal(to_np(g).view(np.uint32), want_g.view(np.uint32))
    assert np.array_equal(to_np(scale).view(np.uint32), want_scale.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)
    # whole runtime path on that handle (prologue behind the rotation, GEMM, epilogue) against the oracle
    M = 70
    x = make_x(M, K, "bf16", seed=5)
    ac, ad = oracle.quantize_act_after(x, "bf16", want_g, block, bits)
    want_y = oracle.epilogue(oracle.gemm_i32(ac, want_codes, K, bits), ad, want_scale, bias, "f32")
    y = fq.linear(to_dev(x, "bf16"), h, 1.0)
    assert_close(to_np(y), want_y, "f32", "fold-after linear")
    gc, gd = fq.quantize_act(to_dev(x, "bf16"), h, block, bits)          # picks the mode up from the handle
    assert np.array_equal(to_np(gc), ac) and np.array_equal(to_np(gd).view(np.uint32), ad.view(np.uint32))
    # an imported copy keeps the mode
    h2 = fq.weights_import(codes, scale, g, b, K, block, bits, fold_after=True)
    assert h2.fold_after
    assert torch.equal(fq.linear(to_dev(x, "bf16"), h2, 1.0), y)


def test_exact_folds_set_multiplier_and_scale_outputs():
    """Eq. 4 helpers: a replaced runtime multiplier (RMS gain absorbed: gamma * g) and scaled output channels
    (1/s absorbed by the up rows of a gate/up handle) against the oracle with the same vectors."""
    rng = np.random.default_rng(31)
    M, K, N, block = 120, 1024, 256, 64
    x = make_x(M, K, "bf16", seed=9)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.02).astype(np.float32)
    s = np.exp(rng.uniform(-1, 1, K)).astype(np.float32)
    gamma = (rng.random(K) + 0.5).astype(np.float32)
    wc, wsc, g = oracle.fold_weights(W, "f32", s, block, 4)
    h = fq.fold_weights(to_dev(W), to_dev(s), to_dev(bias), block, 4)
    # (1) gain absorbed by the multiplier
    g2 = gamma * g
    h.set_multiplier(to_dev(g2))
    want = oracle.linear(x, "bf16", g2, block, 4, 1.0, wc, wsc, bias, "f32")
    y = fq.linear(to_dev(x, "bf16"), h, 1.0)
    assert_close(to_np(y), want[0], "f32", "replaced multiplier")
    codes, delta = fq.quantize_act(to_dev(x, "bf16"), h, block, 4)
    assert np.array_equal(to_np(codes), want[1]) and np.array_equal(to_np(delta).view(np.uint32), want[2].view(np.uint32))
    # (2) constant multiplier (diagonal absorbed upstream)
    h.set_multiplier(None)
    want = oracle.linear(x, "bf16", None, block, 4, 1.0, wc, wsc, bias, "f32")
    assert_close(to_np(fq.linear(to_dev(x, "bf16"), h, 1.0)), want[0], "f32", "constant multiplier")
    # (3) output channels 64..191 scaled by d
    d = np.exp(rng.uniform(-1, 1, 128)).astype(np.float32)
    h.scale_outputs(64, to_dev(d))
    _, sc, _, b = h.export()
    wsc2, bias2 = wsc.copy(), bias.copy()
    wsc2[64:192] *= d
    bias2[64:192] *= d
    assert np.array_equal(to_np(sc).view(np.uint32), wsc2.view(np.uint32))
    assert np.array_equal(to_np(b).view(np.uint32), bias2.view(np.uint32))
    want = oracle.linear(x, "bf16", None, block, 4, 1.0, wc, wsc2, bias2, "f32")
    assert_close(to_np(fq.linear(to_dev(x, "bf16"), h, 1.0)), want[0], "f32", "scaled outputs")


# ------------------------------------------------------------ integer GEMM ----
def random_codes(rng, rows, K, bits):
    q = 7 if bits == 4 else 127
    return oracle.pack(rng.integers(-q, q + 1, size=(rows, K)).astype(np.int32), bits)


def import_codes(wc, K, bits, block=32, scale=None, bias=None):
    N = wc.shape[0]
    scale = np.ones(N, np.float32) if scale is None else scale
    return fq.weights_import(to_dev(wc), to_dev(scale), None, to_dev(bias), K, block, bits)


GEMM_CASES = [
    # M, N, K, bits
    (64, 1024, 1024, 4),
    (50, 3072, 1024, 4),
    (50, 1024, 4096, 4),
    (1, 256, 2048, 4),
    (16, 8, 32, 4),
    (17, 24, 96, 8),
    (130, 136, 160, 4),
    (300, 264, 2048, 8),
    (816, 512, 2048, 4),
    (816, 256, 2048, 8),
    (257, 384, 16384, 8),
    (520, 128, 8192, 4),
]


@pytest.mark.parametrize("M,N,K,bits", GEMM_CASES)
@pytest.mark.parametrize("kernel", ["tcgen05", "simt"])
def test_int32_accumulators_bit_exact(M, N, K, bits, kernel):
    rng = np.random.default_rng(M * 7 + N * 3 + K + bits)
    a = random_codes(rng, M, K, bits)
    w = random_codes(rng, N, K, bits)
    want = oracle.gemm_i32(a, w, K, bits)
    h = import_codes(w, K, bits)
    if kernel == "tcgen05":
        got = fq.gemm_acc_i32(to_dev(a), h)
    else:
        got = fq.gemm_simt(to_dev(a), None, h, raw_acc=True)
    assert np.array_equal(to_np(got), want)


@pytest.mark.parametrize("bits", [4, 8])
def test_accumulator_extremes_and_one_hot(bits):
    q = 7 if bits == 4 else 127
    K, M, N = 16384, 40, 136
    a = oracle.pack(np.full((M, K), q, np.int32), bits)
    w = oracle.pack(np.full((N, K), -q, np.int32), bits)
    got = fq.gemm_acc_i32(to_dev(a), import_codes(w, K, bits))
    assert (got == -q * q * K).all()
    # one-hot activations pick single weight codes: catches any K permutation or operand swap
    K = 256
    rng = np.random.default_rng(0)
    wi = rng.integers(-q, q + 1, size=(N, K)).astype(np.int32)
    eye = np.eye(K, dtype=np.int32)
    got = fq.gemm_acc_i32(to_dev(oracle.pack(eye, bits)), import_codes(oracle.pack(wi, bits), K, bits))
    assert np.array_equal(to_np(got), wi.T)


@pytest.mark.parametrize("M,N,K,bits", [(100, 256, 16384, 4), (208, 384, 16384, 8), (130, 128, 16384, 4), (64, 256, 16384, 8)])
def test_k_split_equals_unsplit_and_oracle(M, N, K, bits):
    """Few tiles and a long K: the planner splits K over a CTA cluster when the workspace has room
    for the partial sums.  With a workspace that holds only the activation codes and steps the same
    call runs unsplit; both must give the oracle's integer sums exactly."""
    rng = np.random.default_rng(M + N + K + bits)
    a, w = random_codes(rng, M, K, bits), random_codes(rng, N, K, bits)
    want = oracle.gemm_i32(a, w, K, bits)
    h = import_codes(w, K, bits)
    base = (M * K + 255) // 256 * 256 + (4 * M + 255) // 256 * 256
    full = fq.workspace_bytes(M, K, N, bits)
    assert full > base, "the planner was expected to ask for split scratch on this shape"
    split = fq.gemm_acc_i32(to_dev(a), h, workspace=torch.empty(full, dtype=torch.uint8, device="cuda"))
    unsplit = fq.gemm_acc_i32(to_dev(a), h, workspace=torch.empty(base, dtype=torch.uint8, device="cuda"))
    assert np.array_equal(to_np(split), want)
    assert np.array_equal(to_np(unsplit), want)
    # and through the scaled epilogue (bf16 output, ragged token tail)
    delta = torch.rand(M, device="cuda") + 0.5
    y1 = fq.gemm_w4a4(to_dev(a), delta, h, out_dtype=torch.bfloat16) if bits == 4 else \
        fq.gemm_w8a8(to_dev(a), delta, h, out_dtype=torch.bfloat16)
    ws = torch.empty(base, dtype=torch.uint8, device="cuda")
    y2 = fq.gemm_w4a4(to_dev(a), delta, h, out_dtype=torch.bfloat16, workspace=ws) if bits == 4 else \
        fq.gemm_w8a8(to_dev(a), delta, h, out_dtype=torch.bfloat16, workspace=ws)
    assert torch.equal(y1, y2)
    st, word = fq.device_status()
    assert st == fq.OK and word == 0


def test_back_to_back_calls_share_a_workspace_without_syncs():
    """The kernels are launched with programmatic stream serialization (each may start its on-chip
    set-up, and the GEMM its weight loads, before the kernel ahead has finished).  A chain of calls
    on one stream that reuse ONE workspace and feed each other must give exactly what the same
    calls give when the device is synchronised after every call."""
    torch.manual_seed(7)
    dev = "cuda"
    K0, N0, N1 = 2048, 1024, 768
    M = 300
    hs = []
    for (n, k, bits) in [(N0, K0, 4), (N1, N0, 8), (N0, N1, 4)]:
        w = (torch.randn((n, k), device=dev) * 0.02)
        hs.append(fq.fold_weights(w, None, torch.randn(n, device=dev) * 0.02, 128 if k % 128 == 0 else 32, bits))
    x0 = torch.randn((M, K0), device=dev).to(torch.bfloat16)
    ws = torch.empty(max(fq.workspace_bytes(M, h.K, h.N, h.bits) for h in hs), dtype=torch.uint8, device=dev)

    def chain(sync):
        outs, x = [], x0
        for rep in range(3):
            for h in hs:
                y = fq.linear(x, h, 1.0, out_dtype=torch.bfloat16, workspace=ws)
                if sync:
                    torch.cuda.synchronize()
                outs.append(y)
                x = y if h is not hs[-1] else x0      # the next call reads this call's output
        torch.cuda.synchronize()
        return outs

    want = chain(sync=True)
    for _ in range(3):
        got = chain(sync=False)
        for a, b in zip(got, want):
            assert torch.equal(a, b)


def _pack_dev(c: torch.Tensor, bits: int) -> torch.Tensor:
    if bits == 8:
        return c.view(torch.uint8)
    u = c.to(torch.int16) & 15
    return (u[:, 0::2] | (u[:, 1::2] << 4)).to(torch.uint8)


def test_random_shapes_against_the_second_witness():
    """Seeded random (M, N, K, bits): every launch configuration the planner can pick (token tiles of 16..208,
    one-, two- and four-atom stages, K splits, CTA pairs, the streaming kernel) must give the dp4a witness's
    accumulators bit for bit and its outputs, with no bounded wait expiring."""
    rng = np.random.default_rng(2024)
    done = 0
    while done < 48:
        bits = int(rng.choice([4, 4, 4, 8]))
        M = int(rng.choice([1, 3, 8, 16, 17, 33, 50, 64, 65, 100, 128, 129, 200, 256, 300, 520, 816]))
        N = int(rng.choice([8, 72, 128, 136, 1024, 3072, 4096, 8192]))
        K = int(rng.choice([32, 96, 128, 256, 384, 512, 640, 1024, 1536, 2048, 4096, 8192, 16384]))
        if N * K > 1 << 26 or M * N > 1 << 22:
            continue
        done += 1
        q = 7 if bits == 4 else 127
        gen = torch.Generator(device="cuda").manual_seed(done)
        wc = torch.randint(-q, q + 1, (N, K), dtype=torch.int8, device="cuda", generator=gen)
        ac = torch.randint(-q, q + 1, (M, K), dtype=torch.int8, device="cuda", generator=gen)
        h = fq.weights_import(_pack_dev(wc, bits), torch.ones(N, device="cuda"), None, None, K, 32, bits)
        a = _pack_dev(ac, bits)
        assert torch.equal(fq.gemm_acc_i32(a, h), fq.gemm_simt(a, None, h, raw_acc=True)), (M, N, K, bits)
        d = torch.rand(M, device="cuda", generator=gen) + 0.5
        y = (fq.gemm_w4a4 if bits == 4 else fq.gemm_w8a8)(a, d, h, torch.float32)
        assert torch.allclose(y, fq.gemm_simt(a, d, h, torch.float32), rtol=1e-5, atol=1e-5), (M, N, K, bits)
        st, word = fq.device_status()
        assert st == fq.OK, (M, N, K, bits, hex(word))


@pytest.mark.parametrize("M,N,K", [(1, 72, 1152), (9, 136, 640), (16, 1032, 2176), (5, 8, 128), (16, 4096, 16384)])
def test_short_batches_on_8bit_weights_take_the_streaming_kernel_bit_exact(M, N, K):
    """At most 16 tokens on 8-bit weights of at most 32 x SMs rows: rows that end inside a stage (K not a multiple of
    1024), row groups that end inside the matrix (N not a multiple of 32), one and two token groups, and the longest
    rows it is given -- integer sums against the oracle, outputs against its epilogue."""
    rng = np.random.default_rng(M + N + K)
    a, w = random_codes(rng, M, K, 8), random_codes(rng, N, K, 8)
    ws = np.exp2(rng.uniform(-10, -6, size=N)).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    h = fq.weights_import(to_dev(w), to_dev(ws), None, to_dev(bias), K, 32, 8)
    want = oracle.gemm_i32(a, w, K, 8)
    assert np.array_equal(to_np(fq.gemm_acc_i32(to_dev(a), h)), want)
    delta = (rng.random(M) + 0.5).astype(np.float32)
    y = fq.gemm_w8a8(to_dev(a), to_dev(delta), h, out_dtype=torch.float32)
    assert_close(to_np(y), oracle.epilogue(want, delta, ws, bias, "f32"), "f32", f"w8 stream {M}x{N}x{K}")
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


@pytest.mark.parametrize("M,K,N,bits", [(816, 2048, 4096, 4), (50, 4096, 1024, 4), (256, 4096, 4096, 4), (64, 8192, 2048, 8),
                                        (16, 16384, 1024, 4), (100, 16384, 256, 4)])
def test_repeated_launches_return_the_same_bits(M, K, N, bits):
    """Rings that are full all the time (weights prefetched far ahead) hand their stages over thousands of times per
    launch: a stage given back an instant too early shows up as a rare wrong output, not as a failure.  Six hundred
    launches per configuration (one-, two- and four-atom stages, 8-bit operands, the streaming kernel, a K split)
    must return the bits of the first, which match the dp4a witness."""
    q = 7 if bits == 4 else 127
    gen = torch.Generator(device="cuda").manual_seed(M + K + N)
    wc = torch.randint(-q, q + 1, (N, K), dtype=torch.int8, device="cuda", generator=gen)
    ac = torch.randint(-q, q + 1, (M, K), dtype=torch.int8, device="cuda", generator=gen)
    h = fq.weights_import(_pack_dev(wc, bits), torch.rand(N, device="cuda", generator=gen) * 0.01 + 0.001, None,
                          torch.randn(N, device="cuda", generator=gen), K, 32, bits)
    a = _pack_dev(ac, bits)
    d = torch.rand(M, device="cuda", generator=gen) + 0.5
    ws = torch.empty(fq.workspace_bytes(M, K, N, bits), dtype=torch.uint8, device="cuda")
    f = fq.gemm_w4a4 if bits == 4 else fq.gemm_w8a8
    ref = f(a, d, h, torch.float32, workspace=ws).clone()
    assert torch.allclose(ref, fq.gemm_simt(a, d, h, torch.float32), rtol=1e-5, atol=1e-5)
    y = torch.empty_like(ref)
    for it in range(600):
        f(a, d, h, y=y, workspace=ws)
        if it % 50 == 49:
            assert torch.equal(y, ref), f"launch {it} differs from the first"
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


@pytest.mark.parametrize("M,sites", [
    (50, [(1024, 3072, 4), (1024, 1024, 4), (1024, 8192, 4), (4096, 1024, 4)]),          # an action-expert layer
    (100, [(16384, 256, 4), (2048, 2048, 4), (16384, 256, 8), (1024, 1024, 8)]),         # K splits between unsplit calls
    (16, [(4096, 4096, 4), (4096, 4096, 8), (8192, 1024, 4), (1024, 4096, 8)]),          # the streaming kernel, both widths
])
def test_calls_of_a_layer_share_one_workspace_in_a_graph(M, sites):
    """A model runs its layers' projections one after the other on one stream with ONE workspace.  Each call's prologue
    overwrites the codes and steps that the call before it may still be reading when it starts early (programmatic
    dependent launch), and a K split's counters are cleared between unrelated launches: a graph of three such layers,
    replayed a hundred times, must give what the calls give with workspaces of their own."""
    gen = torch.Generator(device="cuda").manual_seed(M)
    hs, xs, ys, need = [], [], [], 0
    for K, N, bits in sites:
        W = torch.randn((N, K), device="cuda", generator=gen) * 0.02
        hs.append(fq.fold_weights(W, None, torch.randn(N, device="cuda", generator=gen), 64, bits))
        xs.append(torch.randn((M, K), device="cuda", generator=gen).to(torch.bfloat16))
        ys.append(torch.empty((M, N), dtype=torch.bfloat16, device="cuda"))
        need = max(need, fq.workspace_bytes(M, K, N, bits))
    want = [fq.linear(x, h, 1.0, torch.bfloat16) for x, h in zip(xs, hs)]
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    for x, h, y in zip(xs, hs, ys):
        fq.linear(x, h, 1.0, y=y, workspace=ws)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(3):
            for x, h, y in zip(xs, hs, ys):
                fq.linear(x, h, 1.0, y=y, workspace=ws)
    for it in range(100):
        if it % 10 == 0:
            for y in ys:
                y.zero_()
        g.replay()
        if it % 10 == 9:
            torch.cuda.synchronize()
            for a, b in zip(ys, want):
                assert torch.equal(a, b), f"replay {it}"
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


@pytest.mark.parametrize("M", [1, 16, 64])
def test_short_batch_on_a_large_matrix(M):
    """Long K loops on many tiles (128 stages of four atoms, or a K split): the regime where a pipeline that
    loses a barrier phase would stall rather than miscompute."""
    N, K = 8192, 16384
    gen = torch.Generator(device="cuda").manual_seed(M)
    wc = torch.randint(-7, 8, (N, K), dtype=torch.int8, device="cuda", generator=gen)
    ac = torch.randint(-7, 8, (M, K), dtype=torch.int8, device="cuda", generator=gen)
    h = fq.weights_import(_pack_dev(wc, 4), torch.ones(N, device="cuda"), None, None, K, 32, 4)
    a = _pack_dev(ac, 4)
    for _ in range(3):                                        # back to back: ring phases carry over nothing
        acc = fq.gemm_acc_i32(a, h)
    assert torch.equal(acc, fq.gemm_simt(a, None, h, raw_acc=True))
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


def test_gemm_is_deterministic_run_to_run():
    rng = np.random.default_rng(5)
    a, w = random_codes(rng, 333, 2048, 4), random_codes(rng, 520, 2048, 4)
    h = import_codes(w, 2048, 4)
    first = fq.gemm_acc_i32(to_dev(a), h)
    for _ in range(3):
        assert torch.equal(fq.gemm_acc_i32(to_dev(a), h), first)


# ------------------------------------------------------- whole runtime path ----
def run_site(data: synth.SiteData, rows=None, clip=1.0):
    """Fold + run one site on the GPU and in the oracle; returns dicts of results."""
    site = data.site
    s = oracle_smooth(data)
    W, b = concat_consumers(data)
    wc, ws, g = oracle.fold_weights(W, "f32", s, site.beta, site.bits)
    y_ref, codes_ref, delta_ref, acc_ref = oracle.linear(data.x, site.x_dtype, g, site.beta, site.bits, clip, wc, ws,
                                                         b, site.y_dtype, rows=rows)
    h = fq.fold_weights(to_dev(W), to_dev(s), to_dev(b), site.beta, site.bits)
    ydt = torch.float32 if site.y_dtype == "f32" else torch.bfloat16
    x_dev = to_dev(data.x, site.x_dtype)
    y = assert_fused_stages(x_dev, h, clip, ydt, codes_ref, delta_ref, site.name)
    codes, delta = fq.quantize_act(x_dev, h, site.beta, site.bits, clip)
    return dict(h=h, y=y, codes=codes, delta=delta, x=x_dev), dict(y=y_ref, codes=codes_ref, delta=delta_ref,
                                                                  acc=acc_ref, wc=wc, ws=ws, g=g)


def test_config1_single_w4a4_linear_full_parity():
    data = synth.make_site(synth.config1_site(), seed=0, calib_tokens=512)
    gpu, ref = run_site(data)
    assert np.array_equal(to_np(gpu["codes"]), ref["codes"])
    assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
    hc, hs, hg, _ = gpu["h"].export()
    assert np.array_equal(to_np(hc), ref["wc"]) and np.array_equal(to_np(hs), ref["ws"])
    acc = fq.gemm_acc_i32(gpu["codes"], gpu["h"])
    assert np.array_equal(to_np(acc), ref["acc"])
    assert_close(to_np(gpu["y"]), ref["y"], "f32", "config 1 fused")
    y2 = fq.gemm_w4a4(gpu["codes"], gpu["delta"], gpu["h"], torch.float32)
    assert_close(to_np(y2), ref["y"], "f32", "config 1 two-call")
    # and the layer does what it is for: close to the unquantised projection
    want = data.x.astype(np.float64) @ data.W["proj"].astype(np.float64).T + data.bias["proj"]
    assert np.linalg.norm(to_np(gpu["y"]) - want) / np.linalg.norm(want) < 0.35


@pytest.mark.parametrize("site_idx", [0, 1, 3])
@pytest.mark.parametrize("selective", [True, False])
def test_backbone_layer_sites_small_n(site_idx, selective):
    """Backbone-layer shapes (M = 816, K = 2048 / 16384) with N cut to 512 so the oracle runs in full."""
    site = synth.backbone_layer_sites(selective)[site_idx]
    site.consumers = [(n, min(k, 256)) for n, k in site.consumers][:2]
    data = synth.make_site(site, seed=2 + site_idx)
    gpu, ref = run_site(data)
    assert np.array_equal(to_np(gpu["codes"]), ref["codes"])
    assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
    assert np.array_equal(to_np(fq.gemm_acc_i32(gpu["codes"], gpu["h"])), ref["acc"])
    assert_close(to_np(gpu["y"]), ref["y"], site.y_dtype, site.name)


def test_shared_site_consumers_see_the_same_codes():
    """q/k/v run as one concatenated GEMM equal three separate consumer calls bit for bit."""
    site = synth.backbone_layer_sites()[0]
    site.M = 200
    data = synth.make_site(site, seed=11)
    s = oracle_smooth(data)
    W, b = concat_consumers(data)
    x = to_dev(data.x, "bf16")
    h_all = fq.fold_weights(to_dev(W), to_dev(s), to_dev(b), site.beta, 4)
    codes, delta = fq.quantize_act(x, h_all, site.beta, 4)
    y_all = fq.gemm_w4a4(codes, delta, h_all, torch.bfloat16)
    col = 0
    for name, n in site.consumers:
        h = fq.fold_weights(to_dev(data.W[name]), to_dev(s), to_dev(data.bias[name]), site.beta, 4)
        y = fq.gemm_w4a4(codes, delta, h, torch.bfloat16)
        assert torch.equal(y, y_all[:, col:col + n]), name
        col += n


@pytest.mark.parametrize("bits", [4, 8])
def test_zero_token_gives_bias_and_rows_beyond_m_are_untouched(bits):
    M, K, N = 70, 1024, 264
    rng = np.random.default_rng(3)
    x = make_x(M, K, "bf16", seed=8).copy()
    x[5] = 0
    W = synth.draw_weights(rng, N, K)
    bias = rng.standard_normal(N).astype(np.float32)
    h = fq.fold_weights(to_dev(W), None, to_dev(bias), 128, bits)
    y = torch.full((M + 2, N + 8), 123.0, dtype=torch.float32, device="cuda")
    fq.linear(to_dev(x, "bf16"), h, 1.0, y=y[:M, :N])
    assert np.array_equal(to_np(y[5, :N]), bias)
    assert (y[M:] == 123.0).all() and (y[:, N:] == 123.0).all()
    wc, ws, g = oracle.fold_weights(W, "f32", None, 128, bits)
    ref = oracle.linear(x, "bf16", g, 128, bits, 1.0, wc, ws, bias, "f32")[0]
    assert_close(to_np(y[:M, :N]), ref, "f32", "strided output")


def test_expert_layer_sites_and_amplitude_drift():
    """Action-expert shapes (M = 50, block 64, W4A4) at two denoising amplitudes."""
    for sigma in (1.0, 0.1):
        for site in synth.expert_layer_sites(sigma=sigma):
            data = synth.make_site(site, seed=3)
            gpu, ref = run_site(data)
            assert np.array_equal(to_np(gpu["codes"]), ref["codes"]), site.name
            assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
            assert np.array_equal(to_np(fq.gemm_acc_i32(gpu["codes"], gpu["h"])), ref["acc"]), site.name
            assert_close(to_np(gpu["y"]), ref["y"], site.y_dtype, f"{site.name} sigma={sigma}")


def test_full_size_backbone_sites_sampled_rows_and_second_witness():
    """Full-size backbone layer (gate/up N = 32768, down K = 16384): prologue checked in full,
    outputs checked on sampled token rows, accumulators checked against the dp4a kernel."""
    rows = [0, 1, 127, 128, 207, 208, 415, 500, 623, 624, 799, 815]
    # selective INT8 layer, then the two sites that differ in the uniform W4A4 layer (o_proj and down_proj at 4 bits:
    # the latter is the K split on a 128-k-block tile with multi-atom stages)
    for site in synth.backbone_layer_sites(True) + synth.backbone_layer_sites(False)[1::2]:
        data = synth.make_site(site, seed=2)
        gpu, ref = run_site(data, rows=rows)
        assert np.array_equal(to_np(gpu["codes"]), ref["codes"]), site.name
        assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
        assert_close(to_np(gpu["y"][rows]), ref["y"], site.y_dtype, site.name)
        acc = fq.gemm_acc_i32(gpu["codes"], gpu["h"])
        assert np.array_equal(to_np(acc[rows]), ref["acc"]), site.name
        assert torch.equal(acc, fq.gemm_simt(gpu["codes"], None, gpu["h"], raw_acc=True)), site.name


SWEEP_SAMPLE = [
    # M, K=N, block, bits  (a sample of the throughput-sweep grid; outputs checked on sampled token rows)
    (1, 1024, 32, 4), (1, 4096, 256, 8), (16, 2048, 64, 4), (64, 1024, 128, 8), (256, 4096, 32, 8),
    (256, 2048, 256, 4), (1024, 1024, 64, 4), (1024, 4096, 128, 8), (4096, 2048, 128, 4),
    (8, 8192, 128, 4), (16, 8192, 64, 4),      # the weight-streaming kernel at its largest square (64 Mi weights)
    (3, 1024, 32, 8), (16, 4096, 64, 8), (9, 2048, 256, 8),   # ... and on 8-bit weights
]


@pytest.mark.parametrize("M,KN,block,bits", SWEEP_SAMPLE)
def test_sweep_points_sampled_rows(M, KN, block, bits):
    """Throughput-sweep shapes: prologue bit-exact on every token, accumulators bit-exact and
    outputs within tolerance on sampled rows (first, last and tile-boundary tokens)."""
    data = synth.make_site(synth.sweep_site(M, KN, KN, block, bits), seed=5)
    rows = sorted({0, M - 1, min(M - 1, 207), min(M - 1, 208), M // 2, min(M - 1, 255), min(M - 1, 256)})
    gpu, ref = run_site(data, rows=rows)
    assert np.array_equal(to_np(gpu["codes"]), ref["codes"])
    assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
    acc = fq.gemm_acc_i32(gpu["codes"], gpu["h"])
    assert np.array_equal(to_np(acc[rows]), ref["acc"])
    assert_close(to_np(gpu["y"][rows]), ref["y"], "bf16", f"sweep M={M} K=N={KN}")


@pytest.mark.parametrize("M,KN,block,bits", [(16384, 4096, 64, 4), (4096, 8192, 128, 8)])
def test_sweep_corners_sampled_rows(M, KN, block, bits):
    """Two large points of the throughput sweep (the streaming prologue on long batches; CTA pairs at 8 bits):
    every token's codes and steps, of the canonical call and of the one-call path, against the oracle; accumulators
    and outputs on sampled rows."""
    data = synth.make_site(synth.sweep_site(M, KN, KN, block, bits), seed=5)
    rows = sorted({0, 1, 207, 208, 255, 256, M // 2 + 3, M - 209, M - 2, M - 1})
    gpu, ref = run_site(data, rows=rows)
    assert np.array_equal(to_np(gpu["codes"]), ref["codes"])
    assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
    acc = fq.gemm_acc_i32(gpu["codes"], gpu["h"])
    assert np.array_equal(to_np(acc[rows]), ref["acc"])
    assert_close(to_np(gpu["y"][rows]), ref["y"], "bf16", f"sweep corner M={M} K=N={KN}")


@pytest.mark.parametrize("clip", [1.0, 0.7])
@pytest.mark.parametrize("M,K,block,bits,dtype", [
    (64, 2048, 128, 4, "bf16"), (816, 2048, 128, 4, "f32"),            # register kernel
    (1184, 2048, 128, 4, "bf16"), (1500, 4096, 64, 4, "f32"),          # streaming kernel, 8 rows per SM and more
    (296, 8192, 256, 4, "bf16"), (400, 16384, 256, 8, "bf16"),         # streaming kernel on long rows
    (2000, 1024, 32, 8, "bf16"),
])
def test_fused_call_integer_stages_both_prologue_kernels(M, K, block, bits, dtype, clip):
    """The codes and steps that fq_linear_* hands from its prologue to its GEMM, read back from the workspace."""
    x = make_x(M, K, dtype, seed=M + K)
    rng = np.random.default_rng(M + K + bits)
    s = np.exp(rng.uniform(-1, 1, K)).astype(np.float32)
    W = synth.draw_weights(rng, 72, K)
    wc, ws, g = oracle.fold_weights(W, "f32", s, block, bits)
    want_codes, want_delta = oracle.quantize_act(x, dtype, g, block, bits, clip)
    h = fq.fold_weights(to_dev(W), to_dev(s), None, block, bits)
    y = assert_fused_stages(to_dev(x, dtype), h, clip, torch.float32, want_codes, want_delta, "fused stages")
    rows = [0, M // 2, M - 1]
    sub = oracle.pack(oracle.unpack(want_codes, K, bits)[rows], bits)
    want_y = oracle.epilogue(oracle.gemm_i32(sub, wc, K, bits), want_delta[rows], ws, np.zeros(72, np.float32), "f32")
    assert_close(to_np(y[rows]), want_y, "f32", "fused stages")
    # and without smoothing: the handle's multiplier is the constant block^-1/2, which the one-call path applies
    # without reading a per-channel vector
    wc0, ws0, g0 = oracle.fold_weights(W, "f32", None, block, bits)
    c0, d0 = oracle.quantize_act(x, dtype, g0, block, bits, clip)
    h0 = fq.fold_weights(to_dev(W), None, None, block, bits)
    assert_fused_stages(to_dev(x, dtype), h0, clip, torch.bfloat16, c0, d0, "fused stages, constant multiplier")


def test_one_handle_three_streams_three_workspaces():
    """A weight handle is read-only at run time: consumers of one handle on three streams, each with its own
    workspace (K split included), give what the same calls give one after the other."""
    rng = np.random.default_rng(12)
    M, K, N = 100, 16384, 256                   # few tiles, long K: the planner splits K when scratch is there
    W = synth.draw_weights(rng, N, K)
    h = fq.fold_weights(to_dev(W), None, None, 128, 4)
    need = fq.workspace_bytes(M, K, N, 4)
    assert need > (M * K + 255) // 256 * 256 + 256, "expected split scratch for this shape"
    xs = [to_dev(make_x(M, K, "bf16", seed=20 + i), "bf16") for i in range(3)]
    want = [fq.linear(x, h, 1.0, torch.bfloat16) for x in xs]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(3)]
    wss = [torch.empty(need, dtype=torch.uint8, device="cuda") for _ in range(3)]
    for rep in range(5):
        got = []
        for x, st, ws in zip(xs, streams, wss):
            with torch.cuda.stream(st):
                for _ in range(4):
                    y = fq.linear(x, h, 1.0, torch.bfloat16, workspace=ws)
                got.append(y)
        torch.cuda.synchronize()
        for a, b in zip(got, want):
            assert torch.equal(a, b)


@pytest.mark.parametrize("M,K,N,bits", [(50, 1024, 3072, 4), (50, 4096, 1024, 4), (16, 8192, 8192, 4), (64, 8192, 8192, 4),
                                        (256, 4096, 4096, 4), (816, 2048, 2560, 4), (64, 8192, 2048, 8), (816, 2048, 2048, 8),
                                        (100, 16384, 256, 4), (64, 16384, 256, 8)])      # the last two split K
def test_linear_replayed_in_a_cuda_graph_equals_the_eager_call(M, K, N, bits):
    """The benchmark and any latency-minded caller replay the one-call path from CUDA graphs, where the prologue, the
    GEMM (programmatic dependent launch) and the K split's counter memset really overlap and follow each other
    without host gaps: two rotating operand sets, one step per graph, replayed back to back, must reproduce the
    eager results bit for bit with no bounded wait expiring."""
    gen = torch.Generator(device="cuda").manual_seed(M + K + N)
    sets = []
    for r in range(2):
        W = torch.randn((N, K), device="cuda", generator=gen) * 0.02
        b = torch.randn(N, device="cuda", generator=gen) * 0.02
        h = fq.fold_weights(W, None, b, 64, bits)
        x = (torch.randn((M, K), device="cuda", generator=gen) * 2).to(torch.bfloat16)
        ws = torch.empty(fq.workspace_bytes(M, K, N, bits), dtype=torch.uint8, device="cuda")
        y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        sets.append((x, h, ws, y))
    want = [fq.linear(x, h, 1.0, torch.bfloat16, workspace=ws).clone() for x, h, ws, _ in sets]
    torch.cuda.synchronize()
    graphs = []
    for x, h, ws, y in sets:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fq.linear(x, h, 1.0, y=y, workspace=ws)
        graphs.append(g)
    for rep in range(6):
        for g in graphs:
            g.replay()
    torch.cuda.synchronize()
    for (_, _, _, y), w in zip(sets, want):
        assert torch.equal(y, w)
    st, word = fq.device_status()
    assert st == fq.OK, hex(word)


def test_gemm_accepts_a_step_vector_at_any_float_offset():
    """a_delta need only be 4-byte aligned: a slice of a longer vector of steps gives what a copy of it gives."""
    rng = np.random.default_rng(8)
    M, K, N = 70, 1024, 136
    h = import_codes(random_codes(rng, N, K, 4), K, 4)
    a = to_dev(random_codes(rng, M, K, 4))
    long = torch.rand(M + 8, device="cuda") + 0.5
    for off in (1, 2, 3, 4):
        d = long[off:off + M]
        assert d.data_ptr() % 16 != 0 or off == 4
        for ydt in (torch.float32, torch.bfloat16):
            assert torch.equal(fq.gemm_w4a4(a, d, h, ydt), fq.gemm_w4a4(a, d.clone(), h, ydt))


def test_bounded_wait_expires_into_the_watchdog_and_the_device_stays_usable():
    """fq_watchdog_selftest: a wait nobody ends must give up after its limit, surface once as FQ_ERR_TIMEOUT
    through fq_device_status, and leave the context usable."""
    assert fq.device_status()[0] == fq.OK
    fq.watchdog_selftest(2_000_000)                         # 2 ms
    st, word = fq.device_status()
    assert st == fq.ERR_TIMEOUT and word == 0x400, (st, hex(word))
    assert fq.device_status() == (fq.OK, 0)                 # the record was cleared by the read
    x = to_dev(make_x(50, 1024, "bf16", seed=1), "bf16")
    h = fq.fold_weights(torch.randn((264, 1024), device="cuda") * 0.02, None, None, 64, 4)
    y = fq.linear(x, h, 1.0, torch.bfloat16)
    c, d = fq.quantize_act(x, h, 64, 4)
    assert torch.equal(y, fq.gemm_w4a4(c, d, h, torch.bfloat16))
    assert fq.device_status() == (fq.OK, 0)


def test_calibration_helpers_match_oracle():
    data = synth.make_site(synth.config1_site(), seed=0, calib_tokens=512)
    a = fq.col_absmax(to_dev(data.calib))
    w = fq.col_absmax(to_dev(data.W["proj"]))
    assert np.array_equal(to_np(a), oracle.col_absmax(data.calib))
    assert np.array_equal(to_np(w), oracle.col_absmax(data.W["proj"]))
    w2 = fq.col_absmax(to_dev(2 * data.W["proj"][:100]), out=w.clone())      # accumulate over consumers
    assert np.array_equal(to_np(w2), np.maximum(oracle.col_absmax(data.W["proj"]),
                                                oracle.col_absmax(2 * data.W["proj"][:100])))
    s = fq.smooth_scale(a, w, 0.5)
    assert np.allclose(to_np(s), oracle.smooth_scale(to_np(a), to_np(w), 0.5), rtol=1e-6)


# ------------------------------- weight-only 4-bit projection, float activations ----
W4A16_CASES = [
    # M, N, K, xdtype, ydtype          (adaptive layer-norm modulation: one conditioning vector per sample)
    (1, 3072, 1536, "bf16", "bf16"),
    (1, 3072, 1536, "f32", "f32"),
    (2, 512, 2048, "bf16", "f32"),
    (4, 3072, 1536, "bf16", "bf16"),
    (7, 264, 96, "f32", "f32"),
    (16, 1024, 1024, "bf16", "bf16"),
    (50, 4096, 1024, "bf16", "f32"),
    (3, 8, 32, "f32", "bf16"),
    (5, 6144, 4096, "f32", "f32"),
    (300, 72, 544, "bf16", "f32"),      # more token groups than the grid's second dimension
]


@pytest.mark.parametrize("M,N,K,xdtype,ydtype", W4A16_CASES)
def test_linear_w4a16_matches_oracle(M, N, K, xdtype, ydtype):
    rng = np.random.default_rng(M + 3 * N + 7 * K)
    W = synth.draw_weights(rng, N, K)
    bias = rng.standard_normal(N).astype(np.float32)
    x = synth.as_dtype(rng.standard_normal((M, K)).astype(np.float32), xdtype)
    wc, ws, _ = oracle.fold_weights(W, "f32", None, 1, 4)           # identity transform: RTN of W itself
    h = fq.fold_weights(to_dev(W), None, to_dev(bias), 1, 4)
    hc, hs, _, _ = h.export()
    assert np.array_equal(to_np(hc), wc) and np.array_equal(to_np(hs).view(np.uint32), ws.view(np.uint32))
    want = oracle.linear_wonly(x, xdtype, wc, ws, bias, 4, ydtype)
    ydt = torch.float32 if ydtype == "f32" else torch.bfloat16
    y = fq.linear_w4a16(to_dev(x, xdtype), h, ydt)
    assert_close(to_np(y), want, ydtype, f"w4a16 {M}x{N}x{K}")
    # it does what it is for: the 4-bit weights reproduce the float projection to RTN accuracy
    ref = synth.to_f32(x, xdtype).astype(np.float64) @ W.astype(np.float64).T + bias
    assert np.linalg.norm(as_f64(to_np(y)) - ref) / np.linalg.norm(ref) < 0.2


@pytest.mark.parametrize("M,N,K,xdtype,mean", [(9, 512, 8192, "f32", 4.0), (1, 8192, 8192, "bf16", 0.0), (8, 1024, 16384, "bf16", -2.0),
                                               (3, 264, 16384, "f32", 50.0)])
def test_linear_w4a16_long_rows_and_activations_with_a_mean(M, N, K, xdtype, mean):
    """The kernel multiplies the codes 136 too large and cancels the offset with a second MMA of -136 against the same
    activations, sixteen channels at a time: activations whose sum is far from zero (mean / sigma up to 50, K up to
    16384) must cost it no accuracy (taking 136 x the whole row's sum off at the end left such rows at the edge of
    the tolerance).  Same tolerance as everywhere; also the largest rows the streaming ring sees here."""
    rng = np.random.default_rng(M + N + K)
    q = rng.integers(-8, 8, size=(N, K)).astype(np.int32)
    wc = oracle.pack(q, 4)
    ws = np.exp2(rng.uniform(-9, -7, size=N)).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    x = synth.as_dtype((mean + rng.standard_normal((M, K))).astype(np.float32), xdtype)
    h = fq.weights_import(to_dev(wc), to_dev(ws), None, to_dev(bias), K, 1, 4)
    want = oracle.linear_wonly(x, xdtype, wc, ws, bias, 4, "f32")
    y = fq.linear_w4a16(to_dev(x, xdtype), h, torch.float32)
    assert_close(to_np(y), want, "f32", f"w4a16 mean {mean} {M}x{N}x{K}")


def test_linear_w4a16_rows_longer_than_the_ring_are_reproducible():
    """K = 16384 is eight stages through a ring of six: with the float path's slow consumers the ring stays full and a
    stage given back is overwritten at once.  Two thousand launches on the same operands must return the same bits
    (a stage released before its loads had been performed showed up as wrong sums in about one launch in a thousand)."""
    rng = np.random.default_rng(5)
    M, N, K = 8, 1024, 16384
    q = rng.integers(-8, 8, size=(N, K)).astype(np.int32)
    ws = np.exp2(rng.uniform(-9, -7, size=N)).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    wc = oracle.pack(q, 4)
    x = synth.as_dtype(rng.standard_normal((M, K)).astype(np.float32), "bf16")
    h = fq.weights_import(to_dev(wc), to_dev(ws), None, to_dev(bias), K, 1, 4)
    xd = to_dev(x, "bf16")
    ref = fq.linear_w4a16(xd, h, torch.float32).clone()
    assert_close(to_np(ref), oracle.linear_wonly(x, "bf16", wc, ws, bias, 4, "f32"), "f32", "w4a16 long rows")
    y = torch.empty_like(ref)
    for it in range(2000):
        fq.linear_w4a16(xd, h, y=y)
        if it % 50 == 49:
            assert torch.equal(y, ref), f"launch {it} differs from the first"
    # the integer path shares the ring
    a = random_codes(rng, 16, K, 4)
    hi = import_codes(wc, K, 4)
    acc = fq.gemm_acc_i32(to_dev(a), hi).clone()
    assert np.array_equal(to_np(acc), oracle.gemm_i32(a, wc, K, 4))
    for it in range(500):
        got = fq.gemm_acc_i32(to_dev(a), hi) if it % 50 == 49 else None
        if got is not None:
            assert torch.equal(got, acc)


def test_linear_w4a16_exact_on_integer_activations_and_edges():
    """Integer activations make every binary32 partial sum exact, whatever the order of the additions:
    the kernel must then equal the oracle bit for bit (any indexing slip shows).  Plus the edges: zero
    tokens give the bias, rows beyond M and columns beyond N of a wider output stay untouched."""
    rng = np.random.default_rng(77)
    M, N, K = 6, 136, 1120
    q = rng.integers(-8, 8, size=(N, K)).astype(np.int32)
    wc = oracle.pack(q, 4)
    ws = np.exp2(rng.integers(-8, -3, size=N)).astype(np.float32)
    bias = (rng.integers(-64, 64, size=N) / 8).astype(np.float32)
    x = rng.integers(-31, 32, size=(M, K)).astype(np.float32)
    x[2] = 0
    h = fq.weights_import(to_dev(wc), to_dev(ws), None, to_dev(bias), K, 1, 4)
    want = oracle.linear_wonly(x, "f32", wc, ws, bias)
    ybuf = torch.full((M + 2, N + 8), -7.0, dtype=torch.float32, device="cuda")
    fq.linear_w4a16(to_dev(x), h, y=ybuf[:M, :N])
    got = to_np(ybuf)
    assert np.array_equal(got[:M, :N], want)
    assert np.array_equal(got[2, :N], bias)
    assert np.all(got[M:] == -7.0) and np.all(got[:, N:] == -7.0)
    xb = synth.as_dtype(x, "bf16")                                   # small integers are exact in bf16 too
    assert np.array_equal(to_np(fq.linear_w4a16(to_dev(xb, "bf16"), h)), want)
    assert fq.linear_w4a16(to_dev(x[:0]), h).shape == (0, N)
    h8 = fq.weights_import(to_dev(oracle.pack(q, 8)), to_dev(ws), None, None, K, 1, 8)
    with pytest.raises(fq.FqError) as e:
        fq.linear_w4a16(to_dev(x), h8)
    assert e.value.status == fq.ERR_UNSUPPORTED


def test_identity_rotation_linear_end_to_end():
    """block 1 through the whole W4A4 / W8A8 path: smoothing only, no rotation."""
    for bits, M, K, N in [(4, 70, 1024, 256), (8, 33, 544, 72)]:
        site = synth.Site("scale_only", M, K, [("p", N)], beta=1, bits=bits, x_dtype="bf16", y_dtype="f32", alpha=0.5)
        data = synth.make_site(site, seed=bits, calib_tokens=128)
        gpu, ref = run_site(data)
        assert np.array_equal(to_np(gpu["codes"]), ref["codes"])
        assert np.array_equal(to_np(gpu["delta"]).view(np.uint32), ref["delta"].view(np.uint32))
        assert np.array_equal(to_np(fq.gemm_acc_i32(gpu["codes"], gpu["h"])), ref["acc"])
        assert_close(to_np(gpu["y"]), ref["y"], "f32", f"identity rotation W{bits}")


# ----------------------------------------------------- stored composite rotation ----
COMPOSITE_CASES = [
    # M, K, beta, bits, dtype, smooth, clip
    (50, 1024, 64, 4, "bf16", True, 1.0),
    (50, 4096, 64, 4, "bf16", False, 1.0),
    (7, 96, 32, 8, "f32", True, 0.9),
    (33, 512, 16, 4, "f32", False, 1.0),
    (131, 2048, 128, 8, "bf16", True, 1.0),
    (20, 1024, 256, 4, "f32", True, 0.8),
    (816, 2048, 64, 4, "bf16", True, 1.0),
]


@pytest.mark.parametrize("M,K,beta,bits,dtype,smooth,clip", COMPOSITE_CASES)
def test_quantize_act_composite_bit_exact(M, K, beta, bits, dtype, smooth, clip):
    x = make_x(M, K, dtype, seed=M + K + beta)
    rng = np.random.default_rng(K + beta)
    calib = rng.standard_normal((256, K)).astype(np.float32) * np.exp(rng.uniform(-1, 2, K)).astype(np.float32)
    perm, blocks = synth.composite_rotation(K, beta, seed=3, calib=calib if beta <= 64 else None)
    g = (1.0 / np.exp(rng.uniform(-2, 2, K))).astype(np.float32) if smooth else None
    want_codes, want_delta = oracle.composite_quantize(x, dtype, g, perm, blocks, bits, clip)
    codes, delta = fq.quantize_act_composite(to_dev(x, dtype), to_dev(g), to_dev(perm), to_dev(blocks), bits, clip)
    assert np.array_equal(to_np(delta).view(np.uint32), want_delta.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)


def test_composite_rotation_fold_and_two_call_linear():
    """Offline fold bit-exact; runtime = fq_quantize_act_composite + fq_gemm_*; the result tracks the float
    projection as well as the butterfly rotation does (the paper's ablation finds them equivalent)."""
    site = synth.Site("expert_qkv", 50, 1024, [("qkv", 3072)], beta=64, bits=4, x_dtype="bf16", y_dtype="f32", alpha=0.5)
    data = synth.make_site(site, seed=11, calib_tokens=256)
    W, b = concat_consumers(data)
    s = oracle_smooth(data)
    perm, blocks = synth.composite_rotation(site.K, site.beta, seed=5, calib=data.calib / s)
    wc, ws, g = oracle.fold_weights_composite(W, "f32", s, perm, blocks, 4)
    ac, ad = oracle.composite_quantize(data.x, "bf16", g, perm, blocks, 4, 1.0)
    want = oracle.epilogue(oracle.gemm_i32(ac, wc, site.K, 4), ad, ws, b, "f32")
    dperm, dblocks = to_dev(perm), to_dev(blocks)
    h = fq.fold_weights_composite(to_dev(W), to_dev(s), to_dev(b), dperm, dblocks, 4)
    hc, hs, hg, _ = h.export()
    assert np.array_equal(to_np(hc), wc) and np.array_equal(to_np(hs).view(np.uint32), ws.view(np.uint32))
    assert np.array_equal(to_np(hg).view(np.uint32), g.view(np.uint32))
    x_dev = to_dev(data.x, "bf16")
    codes, delta = fq.quantize_act_composite(x_dev, h, dperm, dblocks, 4)
    assert np.array_equal(to_np(codes), ac) and np.array_equal(to_np(delta).view(np.uint32), ad.view(np.uint32))
    y = fq.gemm_w4a4(codes, delta, h, torch.float32)
    assert_close(to_np(y), want, "f32", "composite rotation, two calls")
    ref = synth.to_f32(data.x, "bf16").astype(np.float64) @ W.astype(np.float64).T + b
    err_c = np.linalg.norm(to_np(y) - ref) / np.linalg.norm(ref)
    gpu_b, _ = run_site(data)
    err_b = np.linalg.norm(to_np(gpu_b["y"]) - ref) / np.linalg.norm(ref)
    assert err_c < 0.35 and err_c < 1.5 * err_b, (err_c, err_b)
    # the one-call entry points refuse a composite handle, and a bad permutation is refused at fold time
    with pytest.raises(fq.FqError) as e:
        fq.linear_w4a4(x_dev, h)
    assert e.value.status == fq.ERR_UNSUPPORTED
    bad = perm.copy()
    bad[3] = site.K
    with pytest.raises(fq.FqError) as e:
        fq.fold_weights_composite(to_dev(W), None, None, to_dev(bad), dblocks, 4)
    assert e.value.status == fq.ERR_INVALID_ARG


# ------------------------------------------- GPTQ rounding in transformed coordinates ----
def _correlated_calib(rng, Mc, K, rank=16, corr=0.85):
    base = rng.standard_normal((Mc, rank)).astype(np.float32)
    mix = rng.standard_normal((rank, K)).astype(np.float32)
    return (corr * base @ mix + (1 - corr) * rng.standard_normal((Mc, K))).astype(np.float32)


GPTQ_CASES = [
    # N, K, Mc, block, bits, smooth, wdtype, cdtype
    (24, 64, 160, 32, 4, False, "f32", "f32"),
    (72, 256, 300, 64, 4, True, "f32", "bf16"),
    (40, 96, 50, 32, 4, False, "bf16", "f32"),       # fewer tokens than channels: the damping carries the rank deficit
    (136, 512, 700, 128, 4, True, "f32", "f32"),
    (16, 128, 200, 1, 8, False, "f32", "f32"),       # identity rotation, 8-bit codes
]


@pytest.mark.parametrize("N,K,Mc,block,bits,smooth,wdtype,cdtype", GPTQ_CASES)
def test_fold_weights_gptq_bit_exact(N, K, Mc, block, bits, smooth, wdtype, cdtype):
    rng = np.random.default_rng(N + K + Mc)
    W = synth.as_dtype(synth.draw_weights(rng, N, K), wdtype)
    W_f = synth.to_f32(W, wdtype)
    calib = synth.as_dtype(_correlated_calib(rng, Mc, K), cdtype)
    if block == 1:
        calib[:, 5] = 0                                    # a dead channel (no rotation: channel 5 itself never fires)
    bias = rng.standard_normal(N).astype(np.float32)
    s = np.exp(rng.uniform(-1, 1, K)).astype(np.float32) if smooth else None
    wc, ws, g, wt, z, U, dead = oracle.fold_weights_gptq(W, wdtype, s, block, calib, cdtype, 0.01, bits, return_all=True)
    h = fq.fold_weights_gptq(to_dev(W, wdtype), to_dev(s), to_dev(bias), to_dev(calib, cdtype), block, bits, 0.01)
    hc, hs, hg, hb = h.export()
    assert np.array_equal(to_np(hs).view(np.uint32), ws.view(np.uint32))
    assert np.array_equal(to_np(hg).view(np.uint32), g.view(np.uint32))
    got, want = oracle.unpack(to_np(hc), K, bits), oracle.unpack(wc, K, bits)
    assert np.array_equal(got, want), f"{(got != want).sum()} of {got.size} codes differ"
    if block == 1:
        assert dead[5] and not got[:, 5].any()
    # the handle runs like any other, and on the calibration tokens it beats the RTN fold (the objective of Eq. 7)
    h_rtn = fq.fold_weights(to_dev(W, wdtype), to_dev(s), to_dev(bias), block, bits)
    rtn = oracle.unpack(to_np(h_rtn.export()[0]), K, bits)
    z64, w64 = z.astype(np.float64), wt.astype(np.float64)
    obj = lambda q: np.linalg.norm((w64 - q * ws[:, None].astype(np.float64)) @ z64.T) ** 2
    assert obj(got) < obj(rtn)
    x = to_dev(calib[: min(Mc, 64)], cdtype)
    y = fq.linear(x, h, 1.0, torch.float32)
    ac, ad = oracle.quantize_act(calib[: min(Mc, 64)], cdtype, g, block, bits)
    want_y = oracle.epilogue(oracle.gemm_i32(ac, wc, K, bits), ad, ws, bias, "f32")
    assert_close(to_np(y), want_y, "f32", "gptq handle through the runtime path")


def test_fold_weights_gptq_backbone_width_sampled_and_errors():
    """K = 2048 (the backbone's 4-bit sites): the oracle's factorisation takes seconds, so it runs once and
    all codes are compared; then the argument checks."""
    rng = np.random.default_rng(9)
    N, K, Mc, block = 64, 2048, 1024, 128
    W = synth.draw_weights(rng, N, K)
    calib = _correlated_calib(rng, Mc, K, rank=64)
    wc, ws, g = oracle.fold_weights_gptq(W, "f32", None, block, calib, "f32", 0.01, 4)
    h = fq.fold_weights_gptq(to_dev(W), None, None, to_dev(calib), block, 4, 0.01)
    hc, hs, _, _ = h.export()
    assert np.array_equal(to_np(hs).view(np.uint32), ws.view(np.uint32))
    assert np.array_equal(to_np(hc), wc)
    with pytest.raises(fq.FqError) as e:
        fq.fold_weights_gptq(torch.zeros((8, 32768), device="cuda"), None, None, torch.zeros((4, 32768), device="cuda"), 64, 4)
    assert e.value.status == fq.ERR_UNSUPPORTED
    # two channels that always fire together and no damping: the second moment is exactly singular
    twin = 2.0 * np.eye(32, dtype=np.float32)
    twin[:, 1] = twin[:, 0]
    with pytest.raises(fq.FqError) as e:
        fq.fold_weights_gptq(to_dev(W[:, :32].copy()), None, None, to_dev(twin), 1, 4, 0.0)
    assert e.value.status == fq.ERR_INVALID_ARG
    with pytest.raises(RuntimeError):
        oracle.gptq_factor(twin, 0.0)


def test_fold_weights_gptq_long_rows_by_properties():
    """K = 8192: beyond what the oracle's cubic factorisation finishes in test time, so properties instead of codes.
    The handle keeps the round-to-nearest steps; the codes stay in range; and on the calibration tokens the GPTQ
    codes reconstruct the transformed weights' outputs better than round-to-nearest does -- the objective of Eq. 7,
    evaluated in binary64 from the oracle's transformed weights and tokens."""
    rng = np.random.default_rng(21)
    N, K, Mc, block = 16, 8192, 192, 256
    W = synth.draw_weights(rng, N, K)
    calib = _correlated_calib(rng, Mc, K, rank=32)
    wc_rtn, ws, g, wt = oracle.fold_weights(W, "f32", None, block, 4, return_wt=True)
    z = (calib * g[None, :]).astype(np.float32)
    for t in range(Mc):
        for b0 in range(0, K, block):
            z[t, b0:b0 + block] = oracle.fwht_block(z[t, b0:b0 + block])
    h = fq.fold_weights_gptq(to_dev(W), None, None, to_dev(calib), block, 4, 0.01)
    hc, hs, _, _ = h.export()
    assert np.array_equal(to_np(hs).view(np.uint32), ws.view(np.uint32))
    q_gptq = oracle.unpack(to_np(hc), K, 4).astype(np.float64)
    q_rtn = oracle.unpack(wc_rtn, K, 4).astype(np.float64)
    assert np.abs(q_gptq).max() <= 7
    z64 = z.astype(np.float64)

    def objective(q):
        return np.linalg.norm((wt.astype(np.float64) - ws.astype(np.float64)[:, None] * q) @ z64.T)

    assert objective(q_gptq) < 0.8 * objective(q_rtn), (objective(q_gptq), objective(q_rtn))


# ------------------------------------------------- gate product fused into the prologue ----
GATED_CASES = [
    # M, K, block, bits, dtype, act, smooth, clip
    (50, 4096, 64, 4, "bf16", oracle.SILU, False, 1.0),
    (816, 16384, 256, 8, "bf16", oracle.GELU_TANH, False, 1.0),
    (7, 96, 32, 8, "f32", oracle.SILU, True, 0.9),
    (300, 2048, 128, 4, "f32", oracle.GELU_TANH, True, 1.0),
    (33, 512, 1, 4, "bf16", oracle.GELU_TANH, False, 1.0),
    (131, 8192, 128, 4, "bf16", oracle.SILU, True, 0.8),
]


def _gate_up(rng, M, K, dtype):
    gu = rng.standard_normal((M, 2 * K)).astype(np.float32)
    gu[:, :K] *= 3.0                                          # gates reach both saturated ends
    gu[0, :8] = [0.0, -0.0, 100.0, -100.0, 88.5, -87.5, 1e-6, -1e-6]
    if M > 1:
        gu[1] = 0                                             # a zero token
    return synth.as_dtype(gu, dtype)


@pytest.mark.parametrize("M,K,block,bits,dtype,act,smooth,clip", GATED_CASES)
def test_quantize_act_gated_bit_exact(M, K, block, bits, dtype, act, smooth, clip):
    rng = np.random.default_rng(M + K + act)
    gu = _gate_up(rng, M, K, dtype)
    g = None
    if smooth:
        g = ((1.0 / np.exp(rng.uniform(-2, 2, K))) * (1.0 / np.sqrt(block))).astype(np.float32)
    want_codes, want_delta = oracle.quantize_act_gated(gu, dtype, act, g, block, bits, clip)
    codes, delta = fq.quantize_act_gated(to_dev(gu, dtype), act, to_dev(g), block, bits, clip)
    assert np.array_equal(to_np(delta).view(np.uint32), want_delta.view(np.uint32))
    assert np.array_equal(to_np(codes), want_codes)
    if M > 1:
        assert to_np(delta)[1] == 0 and not to_np(codes)[1].any()


@pytest.mark.parametrize("bits,act", [(8, oracle.GELU_TANH), (4, oracle.SILU)])
def test_linear_gated_is_down_proj_on_the_gate_product(bits, act):
    rng = np.random.default_rng(40 + bits)
    M, K, N, block = 70, 4096, 1024, 128
    gu = _gate_up(rng, M, K, "bf16")
    W = synth.draw_weights(rng, N, K)
    b = rng.standard_normal(N).astype(np.float32)
    wc, ws, g = oracle.fold_weights(W, "f32", None, block, bits)
    ac, ad = oracle.quantize_act_gated(gu, "bf16", act, g, block, bits)
    want = oracle.epilogue(oracle.gemm_i32(ac, wc, K, bits), ad, ws, b, "bf16")
    h = fq.fold_weights(to_dev(W), None, to_dev(b), block, bits)
    y = fq.linear_gated(to_dev(gu, "bf16"), act, h, 1.0, torch.bfloat16)
    assert_close(to_np(y), want, "bf16", "gated down_proj")
    # and it is the projection of the float gate product, to quantization accuracy
    hf = oracle.gated_product(gu, "bf16", act).astype(np.float64)
    ref = hf @ W.astype(np.float64).T + b
    assert np.linalg.norm(as_f64(to_np(y)) - ref) / np.linalg.norm(ref) < (0.05 if bits == 8 else 0.35)
    with pytest.raises(fq.FqError) as e:
        fq.linear_gated(to_dev(gu, "bf16")[:, :K].contiguous(), act, h)  # only K columns: no up branch
    assert e.value.status == fq.ERR_INVALID_ARG


def test_error_codes_on_device_arguments():
    x = torch.zeros((8, 1024), dtype=torch.float32, device="cuda")
    W = torch.zeros((16, 1024), dtype=torch.float32, device="cuda")
    h8 = fq.fold_weights(W, None, None, 128, 8)
    with pytest.raises(fq.FqError) as e:
        fq.linear_w4a4(x, h8)                                   # handle is 8-bit
    assert e.value.status == fq.ERR_UNSUPPORTED
    with pytest.raises(fq.FqError) as e:
        fq.linear_w8a8(x, h8, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == fq.ERR_NOMEM
    with pytest.raises(fq.FqError) as e:
        fq.quantize_act(x[:, 1:1 + 992], None, 32, 4)           # misaligned base pointer
    assert e.value.status == fq.ERR_ALIGNMENT
    with pytest.raises(fq.FqError) as e:
        fq.linear_w8a8(x, h8, clip_ratio=0.0)
    assert e.value.status == fq.ERR_INVALID_ARG
