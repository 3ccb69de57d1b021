"""Property tests of the CPU oracle on randomly drawn small cases (hypothesis): invariants that hold
for every input, checked against plain numpy integer / float64 arithmetic rather than against the
oracle itself."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle

SET = settings(max_examples=40, deadline=None)


def _codes(rng, rows, K, bits, full_range=False):
    q = 7 if bits == 4 else 127
    lo = -q - 1 if full_range else -q
    return rng.integers(lo, q + 1, size=(rows, K)).astype(np.int32)


@SET
@given(st.integers(1, 6), st.integers(1, 8), st.sampled_from([4, 8]), st.integers(0, 2 ** 31 - 1))
def test_pack_unpack_roundtrip_and_layout(rows, k16, bits, seed):
    K = 16 * k16
    c = _codes(np.random.default_rng(seed), rows, K, bits, full_range=True)
    p = oracle.pack(c, bits)
    assert p.shape == (rows, K * bits // 8)
    assert np.array_equal(oracle.unpack(p, K, bits), c)
    if bits == 4:      # even channel in the low nibble, odd channel in the high nibble, two's complement
        assert np.array_equal(p & 15, c[:, 0::2] & 15) and np.array_equal(p >> 4, c[:, 1::2] & 15)
    else:
        assert np.array_equal(p.view(np.int8), c.astype(np.int8))


@SET
@given(st.integers(1, 5), st.integers(1, 6), st.integers(1, 8), st.sampled_from([4, 8]), st.integers(0, 2 ** 31 - 1))
def test_integer_product_equals_numpy_int64(M, N, k16, bits, seed):
    rng = np.random.default_rng(seed)
    K = 16 * k16
    a, w = _codes(rng, M, K, bits), _codes(rng, N, K, bits)
    got = oracle.gemm_i32(oracle.pack(a, bits), oracle.pack(w, bits), K, bits)
    assert np.array_equal(got.astype(np.int64), a.astype(np.int64) @ w.astype(np.int64).T)


@SET
@given(st.integers(1, 4), st.sampled_from([1, 2, 8, 32]), st.integers(1, 4), st.sampled_from([4, 8]),
       st.floats(0.5, 1.0), st.integers(-6, 6), st.integers(0, 2 ** 31 - 1))
def test_quantizer_invariants(M, beta, nblk, bits, clip, shift, seed):
    rng = np.random.default_rng(seed)
    K = max(32, beta * nblk * (32 // min(32, beta)))
    K = (K + 31) // 32 * 32
    if K % beta:
        K = beta * ((K + beta - 1) // beta)
    x = rng.standard_normal((M, K)).astype(np.float32)
    q = 7 if bits == 4 else 127
    codes, delta, z = oracle.quantize_act(x, "f32", None, beta, bits, np.float32(clip), return_z=True)
    c = oracle.unpack(codes, K, bits)
    assert np.abs(c).max() <= q
    # the step is (clip * max|z|) / q in binary32, and every code is the rounded, clipped quotient
    m = np.abs(z).max(axis=1)
    assert np.array_equal(delta, (np.float32(clip) * m) / np.float32(q))
    want = np.clip(np.rint(z * (np.float32(1.0) / delta)[:, None]), -q, q).astype(np.int32)
    assert np.array_equal(c, want)
    # scaling the input by a power of two scales the step and leaves the codes alone
    codes2, delta2 = oracle.quantize_act(x * np.float32(2.0 ** shift), "f32", None, beta, bits, np.float32(clip))
    assert np.array_equal(codes2, codes) and np.array_equal(delta2, delta * np.float32(2.0 ** shift))


@SET
@given(st.integers(1, 4), st.integers(1, 3), st.integers(1, 6), st.sampled_from(["f32", "bf16"]), st.integers(0, 2 ** 31 - 1))
def test_weight_only_projection_equals_float64_matmul(M, n8, k32, dtype, seed):
    from paper_2609_24433_b200 import synth
    rng = np.random.default_rng(seed)
    N, K = 8 * n8, 32 * k32
    q = _codes(rng, N, K, 4, full_range=True)
    ws = rng.uniform(0.01, 1.0, N).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    x = synth.as_dtype(rng.standard_normal((M, K)).astype(np.float32), dtype)
    got = oracle.linear_wonly(x, dtype, oracle.pack(q, 4), ws, b)
    want = (synth.to_f32(x, dtype).astype(np.float64) @ q.astype(np.float64).T) * ws.astype(np.float64) + b
    assert np.allclose(got, want.astype(np.float32), rtol=1e-6, atol=1e-6)


@SET
@given(st.integers(1, 3), st.sampled_from([16, 32]), st.integers(1, 3), st.sampled_from([4, 8]), st.integers(0, 2 ** 31 - 1))
def test_composite_rotation_with_identity_pieces_is_the_identity_transform(M, beta, nblk, bits, seed):
    rng = np.random.default_rng(seed)
    K = beta * nblk * (32 // min(32, beta))
    x = rng.standard_normal((M, K)).astype(np.float32)
    g = np.exp2(rng.integers(-3, 4, size=K)).astype(np.float32)
    eye = np.tile(np.eye(beta, dtype=np.float32), (K // beta, 1, 1))
    c1, d1 = oracle.composite_quantize(x, "f32", g, np.arange(K), eye, bits)
    c2, d2 = oracle.quantize_act(x, "f32", g, 1, bits)
    assert np.array_equal(c1, c2) and np.array_equal(d1, d2)
    # a permutation alone only reorders the codes
    perm = rng.permutation(K).astype(np.int32)
    c3, d3 = oracle.composite_quantize(x, "f32", g, perm, eye, bits)
    assert np.array_equal(d3, d2)
    assert np.array_equal(oracle.unpack(c3, K, bits), oracle.unpack(c2, K, bits)[:, perm])
