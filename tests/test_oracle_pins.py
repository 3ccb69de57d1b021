"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself -- an explicit Sylvester matrix product, hand-worked quantizer
and packing cases, brute-force loops, closed forms and the identities the paper
states (fold identity, H H^T = beta I, norm preservation, amplitude invariance,
zero token -> bias)."""
import os

import numpy as np
import pytest

import oracle
from paper_2609_24433_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def sylvester(n: int) -> np.ndarray:
    """H_1 = [1], H_2n = [[H, H], [H, -H]] (entries +-1), built independently of the oracle."""
    H = np.array([[1]], dtype=np.int64)
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def inv_transform(z: np.ndarray, beta: int) -> np.ndarray:
    """x with R x = z for the normalised block Hadamard R (R is an involution): exact
    float64 matrix product, used only to craft oracle inputs."""
    H = sylvester(beta).astype(np.float64)
    zb = z.reshape(-1, beta).astype(np.float64)
    return (zb @ H.T / np.sqrt(beta)).reshape(z.shape)


# ------------------------------------------------------------------ FWHT ----
@pytest.mark.parametrize("beta", [2, 4, 8, 16, 32, 64, 128, 256])
def test_fwht_basis_vectors_give_sylvester_columns(beta):
    H = sylvester(beta)
    # entry rule H[i][j] = (-1)^popcount(i & j)
    i, j = np.meshgrid(np.arange(beta), np.arange(beta), indexing="ij")
    pop = np.array([[bin(a & b).count("1") for b in range(beta)] for a in range(beta)])
    assert np.array_equal(H, (-1) ** pop)
    for col in range(beta):
        e = np.zeros(beta, dtype=np.float32)
        e[col] = 1.0
        assert np.array_equal(oracle.fwht_block(e).astype(np.int64), H[:, col])


@pytest.mark.parametrize("beta", [2, 4, 8, 16, 32, 64, 128, 256])
def test_fwht_integer_inputs_equal_exact_matrix_product(beta):
    rng = np.random.default_rng(beta)
    H = sylvester(beta)
    for _ in range(8):
        x = rng.integers(-1024, 1025, size=beta)
        got = oracle.fwht_block(x.astype(np.float32))
        assert np.array_equal(got.astype(np.int64), H @ x)          # exact in binary32
        # H H^T = beta I  (applying the butterfly network twice)
        if beta <= 64:
            twice = oracle.fwht_block(got)
            assert np.array_equal(twice.astype(np.int64), beta * x)


def test_fwht_is_not_symmetric_mistake_detector():
    # A non-symmetric probe: a wrong pairing (i, i+h swapped, or descending order with
    # wrong sign) changes the image of this vector.
    x = np.array([1, 2, 3, 4, 5, 6, 7, 8], dtype=np.float32)
    assert np.array_equal(oracle.fwht_block(x), np.array([36, -4, -8, 0, -16, 0, 0, 0], np.float32))


@pytest.mark.parametrize("beta", [32, 64, 128, 256])
def test_normalised_rotation_preserves_norm_and_is_involution(beta):
    rng = np.random.default_rng(7)
    K = 4 * beta
    x = rng.standard_normal((3, K)).astype(np.float32)
    _, _, z = oracle.quantize_act(x, "f32", None, beta, 8, return_z=True)
    assert np.allclose((z.astype(np.float64) ** 2).sum(1), (x.astype(np.float64) ** 2).sum(1), rtol=1e-5)
    _, _, back = oracle.quantize_act(z, "f32", None, beta, 8, return_z=True)
    assert np.allclose(back, x, rtol=0, atol=2e-5)
    # against the explicit normalised matrix in float64
    H = sylvester(beta) / np.sqrt(beta)
    ref = (x.reshape(3, -1, beta).astype(np.float64) @ H.T).reshape(3, K)
    assert np.allclose(z, ref, rtol=0, atol=1e-5)


@pytest.mark.parametrize("beta", [4, 16, 64, 256])
def test_power_of_two_normalisation_commutes_exactly(beta):
    # beta^(-1/2) is a power of two: scaling before or after the butterflies is bit-identical.
    rng = np.random.default_rng(11)
    x = rng.standard_normal((2, 2 * beta)).astype(np.float32)
    _, _, z = oracle.quantize_act(x, "f32", None, beta, 8, return_z=True)
    post = np.stack([np.concatenate([oracle.fwht_block(r[b:b + beta]) for b in range(0, r.size, beta)])
                     for r in x]) * np.float32(1.0 / np.sqrt(beta))
    assert np.array_equal(z, post.astype(np.float32))


def test_blocks_are_independent():
    beta, K = 32, 96
    x = np.zeros((1, K), dtype=np.float32)
    x[0, 40] = 3.0                                     # lives in block 1 only
    _, _, z = oracle.quantize_act(x, "f32", np.ones(K, np.float32), beta, 8, return_z=True)
    assert np.all(z[0, :32] == 0) and np.all(z[0, 64:] == 0)
    assert np.array_equal(np.abs(z[0, 32:64]), np.full(32, 3.0, np.float32))


# ------------------------------------------------------------- quantizer ----
def _read_quant_cases():
    cases = []
    with open(os.path.join(GOLDEN, "quantizer_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, r, z, delta, codes = [p.strip() for p in line.split("|")]
            cases.append((int(bits), float(r), np.array(z.split(), dtype=np.float64), float(delta),
                          np.array(codes.split(), dtype=np.int32)))
    return cases


@pytest.mark.parametrize("case", _read_quant_cases())
def test_quantizer_hand_cases(case):
    bits, r, z, delta, codes = case
    x = inv_transform(z, 4).astype(np.float32)[None, :]   # exact: dyadic values
    got_codes, got_delta, got_z = oracle.quantize_act(x, "f32", None, 4, bits, r, return_z=True)
    assert np.array_equal(got_z[0].astype(np.float64), z)
    assert got_delta[0] == np.float32(delta)
    assert np.array_equal(oracle.unpack(got_codes, z.size, bits)[0], codes)


@pytest.mark.parametrize("bits", [4, 8])
def test_codes_range_and_extreme_code_is_q(bits):
    q = 7 if bits == 4 else 127
    d = synth.make_site(synth.Site("t", 37, 512, [("p", 8)], beta=64, bits=bits, x_dtype="f32"), seed=3)
    codes, delta = oracle.quantize_act(d.x, "f32", None, 64, bits)
    c = oracle.unpack(codes, 512, bits)
    assert c.min() >= -q and c.max() <= q
    assert np.array_equal(np.abs(c).max(1), np.full(37, q))
    assert np.all(delta > 0)


@pytest.mark.parametrize("bits", [4, 8])
def test_step_is_absmax_over_whole_token(bits):
    # two Hadamard blocks with very different ranges share one step
    q = 7.0 if bits == 4 else 127.0
    z = np.concatenate([np.full(4, 0.5), np.array([64.0, 0, 0, 0])])
    x = inv_transform(z, 4).astype(np.float32)[None, :]
    codes, delta = oracle.quantize_act(x, "f32", None, 4, bits)
    assert delta[0] == np.float32(np.float32(64.0) / np.float32(q))
    c = oracle.unpack(codes, 8, bits)[0]
    assert c[4] == q and np.all(c[:4] == int(np.rint(0.5 / (64.0 / q))))


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("k", [-20, -3, 1, 9])
def test_amplitude_invariance(bits, k):
    # Proposition 2: scaling a token by 2^k leaves the codes and scales the step exactly.
    d = synth.make_site(synth.Site("t", 16, 256, [("p", 8)], beta=64, bits=bits, x_dtype="f32"), seed=5)
    c0, d0 = oracle.quantize_act(d.x, "f32", None, 64, bits)
    c1, d1 = oracle.quantize_act(d.x * np.float32(2.0 ** k), "f32", None, 64, bits)
    assert np.array_equal(c0, c1)
    assert np.array_equal(d1, d0 * np.float32(2.0 ** k))


@pytest.mark.parametrize("bits", [4, 8])
def test_zero_and_tiny_tokens_give_zero_codes_and_bias_output(bits):
    K, N = 128, 16
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, K)).astype(np.float32)
    x[1] = 0.0
    x[2] = np.float32(1e-42)                            # denormal token: step below FLT_MIN
    W = synth.draw_weights(rng, N, K)
    bias = rng.standard_normal(N).astype(np.float32)
    wc, ws, g = oracle.fold_weights(W, "f32", None, 32, bits)
    y, codes, delta, acc = oracle.linear(x, "f32", g, 32, bits, 1.0, wc, ws, bias)
    for t in (1, 2):
        assert delta[t] == 0.0 and not codes[t].any() and not acc[t].any()
        assert np.array_equal(y[t], bias)
    assert delta[0] > 0 and delta[3] > 0


# ------------------------------------------------------------------ pack ----
def test_pack_hand_cases_and_roundtrip():
    with open(os.path.join(GOLDEN, "pack_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            codes, hexes = [p.strip() for p in line.split("|")]
            c = np.array(codes.split(), dtype=np.int32)[None, :]
            want = np.array([int(h, 16) for h in hexes.split()], dtype=np.uint8)
            assert np.array_equal(oracle.pack(c, 4)[0], want)
    rng = np.random.default_rng(0)
    for bits, q in ((4, 7), (8, 127)):
        c = rng.integers(-q, q + 1, size=(5, 64)).astype(np.int32)
        assert np.array_equal(oracle.unpack(oracle.pack(c, bits), 64, bits), c)
    assert np.array_equal(oracle.pack(np.array([[-128, 127, -1]], np.int32)[:, :2], 8).view(np.int8)[0],
                          np.array([-128, 127], np.int8))


# ------------------------------------------------------------------ GEMM ----
@pytest.mark.parametrize("bits", [4, 8])
def test_integer_gemm_equals_brute_force(bits):
    q = 7 if bits == 4 else 127
    rng = np.random.default_rng(bits)
    M, N, K = 5, 7, 64
    a = rng.integers(-q, q + 1, size=(M, K)).astype(np.int32)
    w = rng.integers(-q, q + 1, size=(N, K)).astype(np.int32)
    got = oracle.gemm_i32(oracle.pack(a, bits), oracle.pack(w, bits), K, bits)
    want = np.zeros((M, N), dtype=np.int64)
    for t in range(M):
        for j in range(N):
            s = 0
            for c in range(K):
                s += int(a[t, c]) * int(w[j, c])
            want[t, j] = s
    assert np.array_equal(got.astype(np.int64), want)
    # a transposed-operand mistake would change this non-square case
    assert got.shape == (M, N)


@pytest.mark.parametrize("bits", [4, 8])
def test_integer_gemm_extremes_and_one_hot(bits):
    q = 7 if bits == 4 else 127
    K = 4096
    a = np.full((2, K), q, np.int32)
    w = np.full((3, K), -q, np.int32)
    assert np.all(oracle.gemm_i32(oracle.pack(a, bits), oracle.pack(w, bits), K, bits) == -q * q * K)
    rng = np.random.default_rng(2)
    w = rng.integers(-q, q + 1, size=(6, 32)).astype(np.int32)
    a = np.zeros((32, 32), np.int32)
    a[np.arange(32), np.arange(32)] = 1                   # one-hot rows pick single weights
    assert np.array_equal(oracle.gemm_i32(oracle.pack(a, bits), oracle.pack(w, bits), 32, bits), w.T)
    assert 127 * 127 * 131072 < 2 ** 31                   # accumulator bound at the largest K accepted


# ------------------------------------------------------------------ fold ----
@pytest.mark.parametrize("beta", [32, 64, 128, 256])
@pytest.mark.parametrize("smoothed", [False, True])
def test_fold_identity_before_rounding(beta, smoothed):
    # (W S R^T)(R S^-1 x) = W x
    rng = np.random.default_rng(beta)
    K, N, M = 512, 24, 9
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = synth.draw_weights(rng, N, K)
    s = np.exp(rng.uniform(-2, 2, K)).astype(np.float32) if smoothed else None
    _, _, g, wt = oracle.fold_weights(W, "f32", s, beta, 8, return_wt=True)
    _, _, z = oracle.quantize_act(x, "f32", g, beta, 8, return_z=True)
    want = x.astype(np.float64) @ W.astype(np.float64).T
    got = z.astype(np.float64) @ wt.astype(np.float64).T
    assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max()
    if not smoothed:
        assert np.allclose(np.linalg.norm(wt, axis=1), np.linalg.norm(W, axis=1), rtol=1e-5)
        assert np.array_equal(g, np.full(K, np.float32(1.0 / np.sqrt(beta))))
    else:
        c = np.float32(1.0 / np.sqrt(beta))
        assert np.array_equal(g, (np.float32(1.0) / s) * c)


def test_fold_mismatch_is_detected():
    # A consumer folded with another block size than the runtime uses is badly wrong.
    rng = np.random.default_rng(0)
    K, N, M = 512, 32, 16
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = synth.draw_weights(rng, N, K)
    want = x.astype(np.float64) @ W.astype(np.float64).T
    wc, ws, g = oracle.fold_weights(W, "f32", None, 64, 8)
    good = oracle.linear(x, "f32", g, 64, 8, 1.0, wc, ws, None)[0]
    bad = oracle.linear(x, "f32", oracle.multiplier(None, K, 128, False), 128, 8, 1.0, wc, ws, None)[0]
    rel = lambda y: np.linalg.norm(y - want) / np.linalg.norm(want)
    assert rel(good) < 0.02 and rel(bad) > 0.5


@pytest.mark.parametrize("bits", [4, 8])
def test_weight_rounding_is_rtn_per_output_channel(bits):
    q = 7 if bits == 4 else 127
    rng = np.random.default_rng(4)
    W = synth.draw_weights(rng, 10, 256)
    W[3] = 0.0
    codes, ws, _, wt = oracle.fold_weights(W, "f32", None, 64, bits, return_wt=True)
    c = oracle.unpack(codes, 256, bits)
    assert ws[3] == 0 and not c[3].any()
    rows = [j for j in range(10) if j != 3]
    assert np.array_equal(np.abs(c[rows]).max(1), np.full(9, q))
    assert np.array_equal(ws[rows], (np.abs(wt[rows]).max(1) / np.float32(q)).astype(np.float32))
    # nearest code: |W~ - s*code| <= s/2 (+ rounding slack)
    err = np.abs(wt[rows] - ws[rows, None] * c[rows])
    assert np.all(err <= 0.5 * ws[rows, None] * (1 + 1e-5))


# -------------------------------------------------------------- epilogue ----
@pytest.mark.parametrize("bits", [4, 8])
def test_eq8_equals_product_of_dequantised_operands(bits):
    d = synth.make_site(synth.Site("t", 12, 256, [("p", 40)], beta=64, bits=bits, x_dtype="f32",
                                   y_dtype="f32"), seed=9)
    W, b = d.W["p"], d.bias["p"]
    wc, ws, g = oracle.fold_weights(W, "f32", None, 64, bits)
    y, codes, delta, acc = oracle.linear(d.x, "f32", g, 64, bits, 1.0, wc, ws, b)
    zhat = delta[:, None].astype(np.float64) * oracle.unpack(codes, 256, bits)
    what = ws[:, None].astype(np.float64) * oracle.unpack(wc, 256, bits)
    want = zhat @ what.T + b
    assert np.abs(y - want).max() <= 1e-6 * np.abs(want).max()
    # bf16 output is the float result rounded to nearest even
    yb = oracle.epilogue(acc, delta, ws, b, "bf16")
    assert np.array_equal(yb, synth.f32_to_bf16_bits(y))


def test_int8_sites_are_more_accurate_than_int4():
    d = synth.make_site(synth.Site("t", 64, 1024, [("p", 128)], beta=128, bits=4, x_dtype="f32"), seed=21)
    W = d.W["p"]
    want = d.x.astype(np.float64) @ W.astype(np.float64).T
    rel = {}
    for bits in (4, 8):
        wc, ws, g = oracle.fold_weights(W, "f32", None, 128, bits)
        y = oracle.linear(d.x, "f32", g, 128, bits, 1.0, wc, ws, None)[0]
        rel[bits] = np.linalg.norm(y - want) / np.linalg.norm(want)
    assert rel[8] < 0.03 and rel[8] < rel[4] < 0.5


def test_rows_subset_matches_full():
    d = synth.make_site(synth.Site("t", 20, 256, [("p", 24)], beta=32, bits=4, x_dtype="bf16"), seed=2)
    wc, ws, g = oracle.fold_weights(d.W["p"], "f32", None, 32, 4)
    full = oracle.linear(d.x, "bf16", g, 32, 4, 1.0, wc, ws, d.bias["p"], "bf16")
    sub = oracle.linear(d.x, "bf16", g, 32, 4, 1.0, wc, ws, d.bias["p"], "bf16", rows=[19, 0, 7])
    assert np.array_equal(sub[0], full[0][[19, 0, 7]])
    assert np.array_equal(sub[3], full[3][[19, 0, 7]])


# --------------------------------------------------------- smoothing scale ----
def test_smoothing_scale_closed_forms():
    rng = np.random.default_rng(3)
    a = np.exp(rng.uniform(-3, 3, 64)).astype(np.float32)
    w = np.exp(rng.uniform(-3, 1, 64)).astype(np.float32)
    s1 = oracle.smooth_scale(a, w, 1.0)
    assert np.allclose(a / s1, 1.0, rtol=1e-6)             # alpha = 1 equalises calibrated ranges
    s0 = oracle.smooth_scale(a, w, 0.0)
    assert np.allclose(s0 * w, 1.0, rtol=1e-6)
    sh = oracle.smooth_scale(a, w, 0.5)
    assert np.allclose(a / sh, w * sh, rtol=1e-5)           # alpha = 1/2 balances both sides
    assert np.allclose(sh, np.sqrt(a.astype(np.float64) / w.astype(np.float64)), rtol=1e-6)
    # floors and bounds
    s = oracle.smooth_scale(np.array([0.0, 1e9], np.float32), np.array([1e9, 0.0], np.float32), 0.5)
    assert s[0] == np.float32(1e-5) and s[1] == np.float32(1e5)


def test_col_absmax_against_numpy():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((33, 48)).astype(np.float32)
    assert np.array_equal(oracle.col_absmax(x), np.abs(x).max(0))
    xb = synth.f32_to_bf16_bits(x)
    assert np.array_equal(oracle.col_absmax(xb, "bf16"), np.abs(synth.bf16_bits_to_f32(xb)).max(0))


def test_smoothing_moves_outliers_into_weights():
    site = synth.config1_site()
    d = synth.make_site(site, seed=0, calib_tokens=512)
    a = oracle.col_absmax(d.calib)
    w = oracle.col_absmax(d.W["proj"])
    s = oracle.smooth_scale(a, w, site.alpha)
    ch = d.outlier_channels
    assert s[ch].min() > 3 * np.median(s)
    want = d.x.astype(np.float64) @ d.W["proj"].astype(np.float64).T
    wc, ws, g = oracle.fold_weights(d.W["proj"], "f32", s, site.beta, 4)
    y = oracle.linear(d.x, "f32", g, site.beta, 4, 1.0, wc, ws, None)[0]
    assert np.linalg.norm(y - want) / np.linalg.norm(want) < 0.35


# ------------------------------------------------------------ bf16 helpers ----
def test_bf16_helpers_match_torch():
    import torch
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(4096) * np.exp(rng.uniform(-20, 20, 4096))).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(synth.f32_to_bf16_bits(x), want)
    assert np.array_equal(synth.bf16_bits_to_f32(want),
                          torch.from_numpy(x).to(torch.bfloat16).float().numpy())


# ------------------------------------- transform family T = D^o R D^i, fold-after ----
def dense_rotation(K: int, beta: int) -> np.ndarray:
    """R = I (x) beta^(-1/2) H_beta as a dense float64 matrix, built independently of the oracle."""
    H = sylvester(beta).astype(np.float64) / np.sqrt(beta)
    return np.kron(np.eye(K // beta), H)


def test_transform_family_reduces_to_fold_before():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((9, 256)).astype(np.float32)
    g = (rng.random(256).astype(np.float32) + 0.5) / np.float32(8.0)
    for bits in (4, 8):
        a = oracle.quantize_act(x, "f32", g, 64, bits, 0.9)
        b = oracle.transform_quantize(x, "f32", g, None, 64, bits, 0.9)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
        # D^o = I written out as a vector of ones changes nothing (x * 1.0 is exact)
        c = oracle.transform_quantize(x, "f32", g, np.ones(256, np.float32), 64, bits, 0.9)
        assert np.array_equal(a[0], c[0]) and np.array_equal(a[1].view(np.uint32), c[1].view(np.uint32))


def test_fold_after_hand_case():
    """beta = K = 4: x = (1,1,1,1) -> R x = (2,0,0,0); p = (4,1,1,1) -> z = (0.5,0,0,0), delta = 0.5/7.
    w = (2,2,2,2) -> R w = (4,0,0,0), times p = (16,0,0,0), s^W = 16/7.  codes (7,0,0,0) on both
    sides, acc = 49, y = (0.5/7)(16/7) 49 = 8 = w . x."""
    x = np.ones((1, 4), np.float32)
    w = np.full((1, 4), 2.0, np.float32)
    p = np.array([4, 1, 1, 1], np.float32)
    wc, ws, gpost, wt = oracle.fold_weights_after(w, "f32", p, 4, 4, return_wt=True)
    assert np.array_equal(wt, [[16, 0, 0, 0]]) and np.array_equal(gpost, [0.25, 1, 1, 1])
    assert ws[0] == np.float32(16.0) / np.float32(7.0)
    assert np.array_equal(oracle.unpack(wc, 4, 4), [[7, 0, 0, 0]])
    ac, ad, z = oracle.quantize_act_after(x, "f32", gpost, 4, 4, return_z=True)
    assert np.array_equal(z, [[0.5, 0, 0, 0]]) and ad[0] == np.float32(0.5) / np.float32(7.0)
    assert np.array_equal(oracle.unpack(ac, 4, 4), [[7, 0, 0, 0]])
    acc = oracle.gemm_i32(ac, wc, 4, 4)
    assert acc[0, 0] == 49
    y = oracle.epilogue(acc, ad, ws, np.zeros(1, np.float32))
    assert abs(float(y[0, 0]) - 8.0) < 1e-5


@pytest.mark.parametrize("beta", [4, 64, 256])
def test_fold_after_matches_dense_matrices_and_preserves_the_projection(beta):
    """z = P^-1 R x and W~ = W R^T P against dense float64 matrices (the diagonal sits AFTER the rotation on
    the activation side and multiplies the rotated weight columns), and W~ z = W x before rounding."""
    rng = np.random.default_rng(beta)
    K, N, M = 2 * beta, 6, 5
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.1).astype(np.float32)
    p = (rng.random(K) * 3 + 0.25).astype(np.float32)
    R = dense_rotation(K, beta)
    _, _, gpost, wt = oracle.fold_weights_after(W, "f32", p, beta, 8, return_wt=True)
    _, _, z = oracle.quantize_act_after(x, "f32", gpost, beta, 8, return_z=True)
    z_ref = (x.astype(np.float64) @ R.T) / p.astype(np.float64)
    wt_ref = (W.astype(np.float64) @ R.T) * p.astype(np.float64)
    assert np.allclose(z, z_ref, rtol=1e-5, atol=1e-6)
    assert np.allclose(wt, wt_ref, rtol=1e-5, atol=1e-6)
    assert np.allclose(wt.astype(np.float64) @ z.astype(np.float64).T, W.astype(np.float64) @ x.astype(np.float64).T,
                       rtol=1e-4, atol=1e-5)
    # fold-before with the same vector is a DIFFERENT transform (R S R^T is dense): the two must not coincide
    _, _, g_before = oracle.fold_weights(W, "f32", p, beta, 8)
    _, _, z_before = oracle.quantize_act(x, "f32", g_before, beta, 8, return_z=True)
    assert not np.allclose(z_before, z, rtol=1e-3, atol=1e-4)


def test_fold_after_end_to_end_accuracy_is_that_of_the_quantizer():
    """Eq. 8 on a fold-after site: the output error stays at the level the code width allows."""
    rng = np.random.default_rng(3)
    M, K, N, beta = 32, 512, 48, 128
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, :4] *= 30.0                                    # outlier channels
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    b = (rng.standard_normal(N) * 0.02).astype(np.float32)
    R = dense_rotation(K, beta)
    # P calibrated after rotation, in the coordinates where it is applied (SmoothQuant rule, alpha = 0.5)
    a_rot = np.abs(x.astype(np.float64) @ R.T).max(0).astype(np.float32)
    w_rot = np.abs(W.astype(np.float64) @ R.T).max(0).astype(np.float32)
    p = oracle.smooth_scale(a_rot, w_rot, 0.5)
    y_ref = x.astype(np.float64) @ W.astype(np.float64).T + b
    errs = {}
    for bits in (4, 8):
        wc, ws, gpost = oracle.fold_weights_after(W, "f32", p, beta, bits)
        ac, ad = oracle.quantize_act_after(x, "f32", gpost, beta, bits)
        y = oracle.epilogue(oracle.gemm_i32(ac, wc, K, bits), ad, ws, b)
        errs[bits] = np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref)
    assert errs[8] < 0.02 and errs[4] < 0.25 and errs[8] < errs[4] / 5


# ------------------------------------------ exact folds into neighbouring operators (Eq. 4) ----
def test_rms_gain_is_absorbed_by_the_runtime_multiplier():
    """x = Gamma h: R S^-1 (Gamma h) with the multiplier (gamma/s) beta^-1/2 on the gain-free input equals
    the same transform of x with (1/s) beta^-1/2, up to the single rounding of gamma * h."""
    rng = np.random.default_rng(21)
    K, beta = 512, 64
    h = rng.standard_normal((7, K)).astype(np.float32)
    gamma = (rng.random(K) + 0.5).astype(np.float32)
    s = np.exp(rng.uniform(-1, 1, K)).astype(np.float32)
    g = oracle.multiplier(s, K, beta, False)
    _, _, z_plain = oracle.quantize_act(gamma * h, "f32", g, beta, 8, return_z=True)
    _, _, z_fold = oracle.quantize_act(h, "f32", gamma * g, beta, 8, return_z=True)
    assert np.allclose(z_plain, z_fold, rtol=1e-5, atol=1e-6)


def test_input_diagonal_is_absorbed_by_the_linear_up_branch():
    """x_down = act(gate) * up.  Scaling the up branch's output channel c by 1/s_c (its s^W and bias) makes the
    producer emit x/s, so down_proj's runtime multiplier becomes the constant beta^-1/2; Eq. 8 of down_proj on
    the absorbed pair equals Eq. 8 on the plain pair up to rounding of the intermediate activation."""
    rng = np.random.default_rng(22)
    M, D, I, beta = 24, 128, 256, 64
    x = rng.standard_normal((M, D)).astype(np.float32)
    Wg, Wu = (rng.standard_normal((2, I, D)) * 0.1).astype(np.float32)
    bu = (rng.standard_normal(I) * 0.1).astype(np.float32)
    Wd = (rng.standard_normal((16, I)) * 0.1).astype(np.float32)
    s = np.exp(rng.uniform(-1, 1, I)).astype(np.float32)
    # up branch through the quantized path (8 bits), gate kept in floating point for the test
    uc, us, ug = oracle.fold_weights(Wu, "f32", None, beta, 8)
    ac, ad = oracle.quantize_act(x, "f32", ug, beta, 8)
    acc = oracle.gemm_i32(ac, uc, D, 8)
    up = oracle.epilogue(acc, ad, us, bu)
    up_abs = oracle.epilogue(acc, ad, us * (np.float32(1) / s), bu * (np.float32(1) / s))   # absorbed: same codes
    gate = np.tanh(x.astype(np.float64) @ Wg.astype(np.float64).T).astype(np.float32)
    dc, ds, dg = oracle.fold_weights(Wd, "f32", s, beta, 8)
    y_plain = oracle.linear(gate * up, "f32", dg, beta, 8, 1.0, dc, ds, None)[0]
    y_abs = oracle.linear(gate * up_abs, "f32", None, beta, 8, 1.0, dc, ds, None)[0]
    assert np.allclose(up_abs, up / s, rtol=1e-5, atol=1e-6)
    assert np.linalg.norm(y_abs - y_plain) < 2e-2 * np.linalg.norm(y_plain)


# ---------------------------------------------- identity rotation (beta = 1) ----
def test_identity_rotation_hand_case():
    """beta = 1 is R = I: the fold rounds the scaled weights themselves and the prologue quantizes
    x (.) g.  Hand-worked: W row (7, -3.5, 1.75, 0) has s^W = 1, codes (7, -4, 2, 0) (ties to even);
    the token (0.5, -1.5, 3.5, 0.25) at 4 bits has delta = 0.5, codes (1, -3, 7, 0) (0.5 is a tie -> 0)."""
    W = np.zeros((8, 32), np.float32)
    W[0, :4] = [7.0, -3.5, 1.75, 0.0]
    wc, ws, g = oracle.fold_weights(W, "f32", None, 1, 4)
    assert ws[0] == np.float32(1.0) and np.all(g == np.float32(1.0))
    assert np.array_equal(oracle.unpack(wc, 32, 4)[0, :4], [7, -4, 2, 0])
    x = np.zeros((1, 32), np.float32)
    x[0, :4] = [0.5, -1.5, 3.5, 0.25]
    codes, delta, z = oracle.quantize_act(x, "f32", None, 1, 4, 1.0, return_z=True)
    assert np.array_equal(z, x)                            # no rotation, unit multiplier
    assert delta[0] == np.float32(0.5)
    assert np.array_equal(oracle.unpack(codes, 32, 4)[0, :4], [1, -3, 7, 0])


def test_identity_rotation_with_smoothing_keeps_the_projection():
    """W~ z = (W S)(S^-1 x) = W x before rounding, with no rotation in between."""
    rng = np.random.default_rng(5)
    W = rng.standard_normal((8, 64)).astype(np.float32)
    x = rng.standard_normal((3, 64)).astype(np.float32)
    s = np.exp2(rng.integers(-2, 3, size=64)).astype(np.float32)      # powers of two: exact scaling
    _, _, g, wt = oracle.fold_weights(W, "f32", s, 1, 8, return_wt=True)
    _, _, z = oracle.quantize_act(x, "f32", g, 1, 8, 1.0, return_z=True)
    assert np.array_equal(wt, W * s) and np.array_equal(z, x / s)
    assert np.allclose(z.astype(np.float64) @ wt.astype(np.float64).T, x.astype(np.float64) @ W.astype(np.float64).T,
                       rtol=1e-12, atol=1e-12)


# ------------------------------------- weight-only projection, float activations ----
def test_weight_only_linear_hand_case():
    """y = s^W (q . x) + b: q = (3, -8, 7, 1), x = (0.5, 0.25, -1, 2), s^W = 0.5, b = 1
    -> q.x = 1.5 - 2 - 7 + 2 = -5.5, y = -1.75."""
    K = 32
    q = np.zeros((8, K), np.int32)
    q[0, :4] = [3, -8, 7, 1]
    x = np.zeros((2, K), np.float32)
    x[0, :4] = [0.5, 0.25, -1.0, 2.0]
    ws = np.full(8, 0.5, np.float32)
    b = np.full(8, 1.0, np.float32)
    y = oracle.linear_wonly(x, "f32", oracle.pack(q, 4), ws, b)
    assert y[0, 0] == np.float32(-1.75)
    assert np.all(y[1] == 1.0) and np.all(y[0, 1:] == 1.0)     # zero token / zero rows give the bias


@pytest.mark.parametrize("bits", [4, 8])
def test_weight_only_linear_on_integer_activations_equals_eq8(bits):
    """With activations that are themselves integer codes, the weight-only product is Eq. 8 with
    delta = 1: the brute-force-pinned integer product and epilogue give the same numbers."""
    qm = 7 if bits == 4 else 127
    rng = np.random.default_rng(10 + bits)
    M, N, K = 5, 16, 96
    a = rng.integers(-qm, qm + 1, size=(M, K)).astype(np.int32)
    w = rng.integers(-qm, qm + 1, size=(N, K)).astype(np.int32)
    ws = rng.uniform(0.01, 0.1, N).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    wc = oracle.pack(w, bits)
    want = oracle.epilogue(oracle.gemm_i32(oracle.pack(a, bits), wc, K, bits), np.ones(M, np.float32), ws, b)
    got = oracle.linear_wonly(a.astype(np.float32), "f32", wc, ws, b, bits)
    assert np.array_equal(got, want)
    assert got.shape == (M, N)


def test_weight_only_linear_one_hot_bf16_and_linearity():
    rng = np.random.default_rng(12)
    N, K = 16, 64
    w = rng.integers(-8, 8, size=(N, K)).astype(np.int32)          # the full two's-complement nibble range
    ws = np.exp2(rng.integers(-6, -2, size=N)).astype(np.float32)
    wc = oracle.pack(w, 4)
    eye = np.eye(K, dtype=np.float32)
    y = oracle.linear_wonly(synth.f32_to_bf16_bits(eye), "bf16", wc, ws, None)
    assert np.array_equal(y, (w.T * ws).astype(np.float32))          # one-hot tokens read the dequantised columns
    x1 = rng.integers(-64, 64, size=(4, K)).astype(np.float32) / 16  # dyadic: sums are exact
    x2 = rng.integers(-64, 64, size=(4, K)).astype(np.float32) / 16
    y12 = oracle.linear_wonly(x1 + x2, "f32", wc, ws, None)
    assert np.array_equal(y12, oracle.linear_wonly(x1, "f32", wc, ws, None) + oracle.linear_wonly(x2, "f32", wc, ws, None))
    # bf16 output: one rounding of the binary64 result
    yb = oracle.linear_wonly(x1, "f32", wc, ws, None, out_dtype="bf16")
    assert np.array_equal(yb, synth.f32_to_bf16_bits(oracle.linear_wonly(x1, "f32", wc, ws, None)))


# ----------------------------------------------- stored composite rotation ----
def _random_rotation(rng, K, beta):
    """Random permutation and per-block orthogonal matrices (QR of Gaussians), float32."""
    perm = rng.permutation(K).astype(np.int32)
    blocks = np.stack([np.linalg.qr(rng.standard_normal((beta, beta)))[0] for _ in range(K // beta)]).astype(np.float32)
    return perm, blocks


def test_composite_rotation_hand_case():
    """beta = 2, K = 4 (padded to 32 with identity blocks): perm = (1, 0, 3, 2), B_0 = [[1, 2], [3, 4]],
    B_1 = [[0.5, -0.5], [0.25, 1]], pre = (2, 1, 1, 0.5), x = (1, 2, 3, 4):
    v = (2, 2, 3, 2); p = (2, 2, 2, 3); u = (1*2 + 2*2, 3*2 + 4*2, 0.5*2 - 0.5*3, 0.25*2 + 3) = (6, 14, -0.5, 3.5)."""
    K, beta = 32, 2
    perm = np.arange(K, dtype=np.int32)
    perm[:4] = [1, 0, 3, 2]
    blocks = np.tile(np.eye(2, dtype=np.float32), (K // beta, 1, 1))
    blocks[0] = [[1, 2], [3, 4]]
    blocks[1] = [[0.5, -0.5], [0.25, 1]]
    pre = np.ones(K, np.float32)
    pre[:4] = [2, 1, 1, 0.5]
    x = np.zeros((1, K), np.float32)
    x[0, :4] = [1, 2, 3, 4]
    codes, delta, z = oracle.composite_quantize(x, "f32", pre, perm, blocks, 8, 1.0, return_z=True)
    assert np.array_equal(z[0, :4], [6, 14, -0.5, 3.5]) and not z[0, 4:].any()
    assert delta[0] == np.float32(14.0) / np.float32(127.0)
    assert np.array_equal(oracle.unpack(codes, K, 8)[0, :4], [54, 127, -5, 32])     # rint(u * 127 / 14), -4.54 -> -5


@pytest.mark.parametrize("beta", [16, 64])
def test_composite_rotation_with_hadamard_blocks_is_the_fwht_path(beta):
    """Identity permutation and B_b = beta^-1/2 H_beta (entries +-2^-k, exact) on integer inputs: every
    operation of both routes is exact, so the stored-matrix route must reproduce the butterflies."""
    rng = np.random.default_rng(beta)
    K = 4 * beta
    x = rng.integers(-50, 51, size=(6, K)).astype(np.float32)
    H = (sylvester(beta) / np.sqrt(beta)).astype(np.float32)
    blocks = np.tile(H, (K // beta, 1, 1))
    c1, d1, z1 = oracle.composite_quantize(x, "f32", None, np.arange(K), blocks, 4, 1.0, return_z=True)
    c2, d2, z2 = oracle.quantize_act(x, "f32", None, beta, 4, 1.0, return_z=True)
    assert np.array_equal(z1, z2) and np.array_equal(d1, d2) and np.array_equal(c1, c2)


def test_composite_rotation_matches_dense_matrices_and_keeps_the_projection():
    rng = np.random.default_rng(21)
    K, beta, N = 128, 32, 24
    perm, blocks = _random_rotation(rng, K, beta)
    x = rng.standard_normal((5, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    s = np.exp(rng.uniform(-1, 1, K)).astype(np.float32)
    # dense R = blockdiag(B) Pi, built independently in float64
    Pi = np.zeros((K, K))
    Pi[np.arange(K), perm] = 1.0
    Bd = np.zeros((K, K))
    for b in range(K // beta):
        Bd[b * beta:(b + 1) * beta, b * beta:(b + 1) * beta] = blocks[b]
    R = Bd @ Pi
    _, _, g, wt = oracle.fold_weights_composite(W, "f32", s, perm, blocks, 8, return_wt=True)
    _, _, z = oracle.composite_quantize(x, "f32", g, perm, blocks, 8, 1.0, return_z=True)
    assert np.allclose(z, (R @ (x / s).T.astype(np.float64)).T, rtol=1e-5, atol=1e-5)
    assert np.allclose(wt, (R @ (W * s).T.astype(np.float64)).T, rtol=1e-5, atol=1e-5)
    # R is orthogonal (to float32 accuracy of the stored blocks): the unquantized projection is preserved
    want = x.astype(np.float64) @ W.astype(np.float64).T
    assert np.allclose(z.astype(np.float64) @ wt.astype(np.float64).T, want, rtol=1e-4, atol=1e-4)
    # a transposed block or an inverted permutation would not preserve it
    wrong = np.transpose(blocks, (0, 2, 1)).copy()
    _, _, zbad = oracle.composite_quantize(x, "f32", g, perm, wrong, 8, 1.0, return_z=True)
    assert not np.allclose(zbad.astype(np.float64) @ wt.astype(np.float64).T, want, rtol=1e-2, atol=1e-2)
    inv = np.argsort(perm).astype(np.int32)
    _, _, zbad = oracle.composite_quantize(x, "f32", g, inv, blocks, 8, 1.0, return_z=True)
    assert not np.allclose(zbad.astype(np.float64) @ wt.astype(np.float64).T, want, rtol=1e-2, atol=1e-2)


# ------------------------------------- GPTQ rounding in transformed coordinates ----
def _gptq_inputs(seed, N=24, K=64, Mc=160, beta=32, corr=0.9):
    """Weights and strongly correlated calibration tokens (GPTQ only differs from RTN when G is not diagonal)."""
    rng = np.random.default_rng(seed)
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    base = rng.standard_normal((Mc, 8)).astype(np.float32)
    mix = rng.standard_normal((8, K)).astype(np.float32)
    calib = (corr * base @ mix + (1 - corr) * rng.standard_normal((Mc, K))).astype(np.float32)
    return W, calib, beta


def test_gptq_factor_is_the_upper_cholesky_factor_of_the_inverse():
    W, calib, beta = _gptq_inputs(1)
    _, _, z = oracle.quantize_act(calib, "f32", None, beta, 4, 1.0, return_z=True)
    U, dead = oracle.gptq_factor(z, damp=0.01)
    assert not dead.any() and np.allclose(np.tril(U, -1), 0)
    z64 = z.astype(np.float64)
    G = z64.T @ z64
    H = G + 0.01 * np.mean(np.diag(G)) * np.eye(G.shape[0])
    want = np.linalg.cholesky(np.linalg.inv(H)).T           # unique upper factor with positive diagonal
    assert np.allclose(U, want, rtol=2e-3, atol=2e-3 * np.abs(want).max())
    assert np.allclose(U.T.astype(np.float64) @ U.astype(np.float64) @ H, np.eye(H.shape[0]), atol=5e-3)


def test_gptq_with_uncorrelated_channels_is_rtn():
    """A diagonal second moment leaves nothing to compensate: U is diagonal and the sweep is RTN."""
    rng = np.random.default_rng(2)
    N, K = 16, 32
    wt = rng.standard_normal((N, K)).astype(np.float32)
    z = np.zeros((K, K), np.float32)
    z[np.arange(K), np.arange(K)] = np.exp2(rng.integers(-2, 3, size=K)).astype(np.float32)   # one token per channel
    U, dead = oracle.gptq_factor(z, damp=0.0)
    assert np.count_nonzero(U - np.diag(np.diag(U))) == 0
    s = (np.abs(wt).max(axis=1) / np.float32(7)).astype(np.float32)
    codes = oracle.gptq_round(wt, U, dead, s, 4)
    rtn = np.clip(np.rint(wt * (np.float32(1) / s)[:, None]), -7, 7).astype(np.int32)
    assert np.array_equal(codes, rtn)


def test_gptq_hand_case_two_channels():
    """K = 2 worked by hand.  z rows (1, 1) and (1, -0.5): G = [[2, 0.5], [0.5, 1.25]], no damping.
    H = M M^T with M = [[m00, m01], [0, m11]]: m11 = sqrt(1.25), m01 = 0.5 / m11, m00 = sqrt(2 - m01^2);
    U = M^-1 = [[1/m00, -m01 / (m00 m11)], [0, 1/m11]].  Row w = (0.9, 0.2), step 0.25 (q irrelevant):
    code0 = rint(3.6) = 4, e = (0.9 - 1.0) / U00 = -0.1 m00; w1 <- 0.2 - e U01 = 0.2 - 0.1 m01 / m11 = 0.2 - 0.04 = 0.16;
    code1 = rint(0.64) = 1.  RTN would give rint(0.8) = 1 too; with w = (0.9, 0.14): RTN (4, 1), GPTQ (4, 0) since 0.10 / 0.25 = 0.4."""
    z = np.zeros((2, 32), np.float32)        # pad to 32 channels with dead ones
    z[0, :2] = [1.0, 1.0]
    z[1, :2] = [1.0, -0.5]
    U, dead = oracle.gptq_factor(z, damp=0.0)
    assert dead[2:].all() and not dead[:2].any()
    m11 = np.sqrt(1.25); m01 = 0.5 / m11; m00 = np.sqrt(2 - m01 ** 2)
    assert np.allclose(U[:2, :2], [[1 / m00, -m01 / (m00 * m11)], [0, 1 / m11]], rtol=1e-6)
    wt = np.zeros((8, 32), np.float32)
    wt[0, :2] = [0.9, 0.2]
    wt[1, :2] = [0.9, 0.14]
    wt[:, 31] = 1.75                             # fixes the row step at 1.75 / 7 = 0.25 (a dead channel: code 0)
    s = np.full(8, 0.25, np.float32)
    codes = oracle.gptq_round(wt, U, dead, s, 4)
    assert list(codes[0, :2]) == [4, 1] and list(codes[1, :2]) == [4, 0]
    assert not codes[:, 2:].any()               # dead channels get zero codes


def test_gptq_lowers_the_objective_of_eq7_against_rtn():
    W, calib, beta = _gptq_inputs(3)
    wc, ws, g, wt, z, U, dead = oracle.fold_weights_gptq(W, "f32", None, beta, calib, return_all=True)
    rtn_codes, ws2, _ = oracle.fold_weights(W, "f32", None, beta, 4)
    assert np.array_equal(ws, ws2)               # same per-output-channel steps as the RTN fold
    q_g = oracle.unpack(wc, W.shape[1], 4).astype(np.float64) * ws[:, None]
    q_r = oracle.unpack(rtn_codes, W.shape[1], 4).astype(np.float64) * ws[:, None]
    z64, w64 = z.astype(np.float64), wt.astype(np.float64)
    obj = lambda q: np.linalg.norm((w64 - q) @ z64.T) ** 2
    assert obj(q_g) < 0.7 * obj(q_r)
    assert np.abs(oracle.unpack(wc, W.shape[1], 4)).max() <= 7


# ---------------------------------------------- gated-MLP product (SiLU / GELU-tanh) ----
def test_gate_activations_against_float64_and_special_values():
    x = np.concatenate([np.linspace(-30, 30, 2001), [-100.0, -88.5, 100.0, 0.0, 1e-6, -1e-6]]).astype(np.float32)
    x64 = x.astype(np.float64)
    silu = x64 / (1.0 + np.exp(-x64))
    gelu = 0.5 * x64 * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x64 + 0.044715 * x64 ** 3)))
    got_s, got_g = oracle.gate_act(x, oracle.SILU), oracle.gate_act(x, oracle.GELU_TANH)
    # relative to the magnitude of the result, with an absolute floor in the far negative tail
    assert np.all(np.abs(got_s - silu) <= 2e-6 * np.abs(silu) + 1e-30 + 1e-6 * np.exp(-np.abs(x64)))
    assert np.all(np.abs(got_g - gelu) <= 3e-6 * np.abs(gelu) + 1e-30 + 1e-6 * np.exp(-np.abs(x64)))
    assert oracle.gate_act(0.0, oracle.SILU) == 0.0 and oracle.gate_act(0.0, oracle.GELU_TANH) == 0.0
    assert oracle.gate_act(50.0, oracle.SILU) == np.float32(50.0)          # sigmoid saturates to 1
    assert oracle.gate_act(10.0, oracle.GELU_TANH) == np.float32(10.0)
    assert abs(float(oracle.gate_act(-50.0, oracle.SILU))) < 1e-19       # and to 0
    assert oracle.gate_act(1.0, oracle.SILU) == pytest.approx(0.7310585786300049, rel=2e-7)
    assert oracle.gate_act(1.0, oracle.GELU_TANH) == pytest.approx(0.8411919906082768, rel=3e-7)


def test_gated_product_layout_and_composition():
    rng = np.random.default_rng(30)
    M, K = 3, 64
    gu = rng.standard_normal((M, 2 * K)).astype(np.float32)
    h = oracle.gated_product(gu, "f32", oracle.SILU)
    assert h.shape == (M, K)
    # gate is the first half, up the second: swapping them changes the result; a unit up branch returns act(gate)
    assert np.array_equal(h, oracle.gate_act(gu[:, :K], oracle.SILU) * gu[:, K:])
    ones = gu.copy()
    ones[:, K:] = 1.0
    assert np.array_equal(oracle.gated_product(ones, "f32", oracle.GELU_TANH), oracle.gate_act(gu[:, :K], oracle.GELU_TANH))
    # bf16 inputs are widened exactly; the quantizer then sees the product
    gb = synth.f32_to_bf16_bits(gu)
    hb = oracle.gated_product(gb, "bf16", oracle.SILU)
    assert np.array_equal(hb, oracle.gated_product(synth.bf16_bits_to_f32(gb), "f32", oracle.SILU))
    c1, d1 = oracle.quantize_act_gated(gb, "bf16", oracle.SILU, None, 32, 4)
    c2, d2 = oracle.quantize_act(hb, "f32", None, 32, 4)
    assert np.array_equal(c1, c2) and np.array_equal(d1, d2)
