"""CPU oracle of the folded quantized linear layer (test infrastructure only).

Thin numpy/ctypes front end over ``fq_oracle.c``; every numerical step lives in
that C file, which restates Eq. 3, Eq. 5, Eq. 8 and Algorithm 1 of the paper.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA product path never does.

bfloat16 tensors are numpy ``uint16`` arrays holding the raw bit patterns and
are tagged with ``dtype="bf16"``; everything else is ``float32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fq_oracle.c")
_LIB = os.path.join(_HERE, "libfq_oracle.so")

F32, BF16 = 0, 1
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.fqo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().fqo_num_threads())


def _dt(dtype: str) -> int:
    if dtype in ("f32", "fp32", "float32"):
        return F32
    if dtype in ("bf16", "bfloat16"):
        return BF16
    raise ValueError(dtype)


def _mat(x: np.ndarray, dtype: str) -> np.ndarray:
    want = np.float32 if _dt(dtype) == F32 else np.uint16
    x = np.ascontiguousarray(x)
    if x.dtype != want:
        raise TypeError(f"expected {want} for dtype={dtype}, got {x.dtype}")
    return x


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def fwht_block(v: np.ndarray) -> np.ndarray:
    """Unnormalised Sylvester-Hadamard product of one block (length = beta)."""
    out = np.array(v, dtype=np.float32, copy=True).reshape(-1)
    _load().fqo_fwht_block(_p(out), ctypes.c_int(out.size))
    return out


def multiplier(smooth, K: int, beta: int, for_weights: bool) -> np.ndarray:
    g = np.empty(K, dtype=np.float32)
    s = _f32(smooth)
    _check(_load().fqo_multiplier(_p(s), ctypes.c_int64(K), ctypes.c_int(beta),
                                  ctypes.c_int(1 if for_weights else 0), _p(g)), "multiplier")
    return g


def smooth_scale(a, w, alpha: float) -> np.ndarray:
    a = _f32(a)
    w = _f32(w)
    s = np.empty_like(a)
    _check(_load().fqo_smooth_scale(_p(a), _p(w), ctypes.c_int64(a.size), ctypes.c_double(alpha),
                                    _p(s)), "smooth_scale")
    return s


def col_absmax(x: np.ndarray, dtype: str = "f32") -> np.ndarray:
    x = _mat(x, dtype)
    M, K = x.shape
    out = np.empty(K, dtype=np.float32)
    _check(_load().fqo_col_absmax(_p(x), ctypes.c_int(_dt(dtype)), ctypes.c_int64(M),
                                  ctypes.c_int64(K), ctypes.c_int64(K), _p(out)), "col_absmax")
    return out


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    rows, K = codes.shape
    out = np.empty((rows, K * bits // 8), dtype=np.uint8)
    _check(_load().fqo_pack(_p(codes), ctypes.c_int64(rows), ctypes.c_int64(K), ctypes.c_int(bits),
                            _p(out)), "pack")
    return out


def unpack(packed: np.ndarray, K: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed).view(np.uint8)
    rows = packed.shape[0]
    out = np.empty((rows, K), dtype=np.int32)
    _check(_load().fqo_unpack(_p(packed), ctypes.c_int64(rows), ctypes.c_int64(K),
                              ctypes.c_int(bits), _p(out)), "unpack")
    return out


def quantize_act(x: np.ndarray, dtype: str, g, beta: int, bits: int, clip_ratio: float = 1.0,
                 return_z: bool = False):
    """Runtime prologue: returns (codes[M, K*bits/8] u8, delta[M] f32[, z[M, K] f32])."""
    x = _mat(x, dtype)
    M, K = x.shape
    g = _f32(g)
    codes = np.zeros((M, K * bits // 8), dtype=np.uint8)
    delta = np.zeros(M, dtype=np.float32)
    z = np.zeros((M, K), dtype=np.float32) if return_z else None
    _check(_load().fqo_quantize_act(_p(x), ctypes.c_int(_dt(dtype)), ctypes.c_int64(M),
                                    ctypes.c_int64(K), ctypes.c_int64(K), _p(g), ctypes.c_int(beta),
                                    ctypes.c_int(bits), ctypes.c_float(clip_ratio), _p(codes),
                                    _p(delta), _p(z)), "quantize_act")
    return (codes, delta, z) if return_z else (codes, delta)


def fold_weights(W: np.ndarray, dtype: str, smooth, beta: int, bits: int, return_wt: bool = False):
    """Offline fold + RTN + pack: returns (codes, w_scale[N], mult_g[K][, W~[N, K]])."""
    W = _mat(W, dtype)
    N, K = W.shape
    s = _f32(smooth)
    codes = np.zeros((N, K * bits // 8), dtype=np.uint8)
    w_scale = np.zeros(N, dtype=np.float32)
    g = np.zeros(K, dtype=np.float32)
    wt = np.zeros((N, K), dtype=np.float32) if return_wt else None
    _check(_load().fqo_fold_weights(_p(W), ctypes.c_int(_dt(dtype)), ctypes.c_int64(N),
                                    ctypes.c_int64(K), ctypes.c_int64(K), _p(s), ctypes.c_int(beta),
                                    ctypes.c_int(bits), _p(codes), _p(w_scale), _p(g), _p(wt)),
           "fold_weights")
    return (codes, w_scale, g, wt) if return_wt else (codes, w_scale, g)


def transform_quantize(x: np.ndarray, dtype: str, pre, post, beta: int, bits: int, clip_ratio: float = 1.0,
                       return_z: bool = False):
    """z = D^o (R (D^i x)) then Eq. 5, for the whole family T = D^o R D^i: ``pre`` = d^i * beta^-1/2 per
    channel (None: the constant beta^-1/2), ``post`` = d^o per channel (None: 1).
    Returns (codes, delta[, z])."""
    x = _mat(x, dtype)
    M, K = x.shape
    codes = np.zeros((M, K * bits // 8), dtype=np.uint8)
    delta = np.zeros(M, dtype=np.float32)
    z = np.zeros((M, K), dtype=np.float32) if return_z else None
    _check(_load().fqo_transform_quantize(_p(x), ctypes.c_int(_dt(dtype)), ctypes.c_int64(M), ctypes.c_int64(K),
                                          ctypes.c_int64(K), _p(_f32(pre)), _p(_f32(post)), ctypes.c_int(beta),
                                          ctypes.c_int(bits), ctypes.c_float(clip_ratio), _p(codes), _p(delta),
                                          _p(z)), "transform_quantize")
    return (codes, delta, z) if return_z else (codes, delta)


def quantize_act_after(x: np.ndarray, dtype: str, g_post, beta: int, bits: int, clip_ratio: float = 1.0,
                       return_z: bool = False):
    """Runtime prologue of a fold-after site: z = P^-1 R x with g_post = 1/p."""
    return transform_quantize(x, dtype, None, g_post, beta, bits, clip_ratio, return_z)


def fold_weights_after(W: np.ndarray, dtype: str, p, beta: int, bits: int, return_wt: bool = False):
    """Fold-after, offline: W~ = W R^T P, RTN, pack.  Returns (codes, w_scale[N], g_post[K] = 1/p[, W~])."""
    W = _mat(W, dtype)
    N, K = W.shape
    codes = np.zeros((N, K * bits // 8), dtype=np.uint8)
    w_scale = np.zeros(N, dtype=np.float32)
    g = np.zeros(K, dtype=np.float32)
    wt = np.zeros((N, K), dtype=np.float32) if return_wt else None
    _check(_load().fqo_fold_weights_after(_p(W), ctypes.c_int(_dt(dtype)), ctypes.c_int64(N), ctypes.c_int64(K),
                                          ctypes.c_int64(K), _p(_f32(p)), ctypes.c_int(beta), ctypes.c_int(bits),
                                          _p(codes), _p(w_scale), _p(g), _p(wt)), "fold_weights_after")
    return (codes, w_scale, g, wt) if return_wt else (codes, w_scale, g)


def gemm_i32(a_codes: np.ndarray, w_codes: np.ndarray, K: int, bits: int) -> np.ndarray:
    a = np.ascontiguousarray(a_codes).view(np.uint8)
    w = np.ascontiguousarray(w_codes).view(np.uint8)
    M, N = a.shape[0], w.shape[0]
    acc = np.zeros((M, N), dtype=np.int32)
    _check(_load().fqo_gemm_i32(_p(a), _p(w), ctypes.c_int64(M), ctypes.c_int64(N),
                                ctypes.c_int64(K), ctypes.c_int(bits), _p(acc)), "gemm_i32")
    return acc


def epilogue(acc: np.ndarray, delta, w_scale, bias, out_dtype: str = "f32") -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M, N = acc.shape
    y = np.zeros((M, N), dtype=np.float32 if _dt(out_dtype) == F32 else np.uint16)
    _check(_load().fqo_epilogue(_p(acc), _p(_f32(delta)), _p(_f32(w_scale)), _p(_f32(bias)),
                                ctypes.c_int64(M), ctypes.c_int64(N), _p(y),
                                ctypes.c_int(_dt(out_dtype)), ctypes.c_int64(N)), "epilogue")
    return y


def linear(x: np.ndarray, xdtype: str, g, beta: int, bits: int, clip_ratio: float,
           w_codes: np.ndarray, w_scale, bias, out_dtype: str = "f32",
           rows: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Whole runtime path. Returns (y, a_codes, delta, acc); with ``rows`` the
    integer product and epilogue run on those token rows only."""
    x = _mat(x, xdtype)
    M, K = x.shape
    w = np.ascontiguousarray(w_codes).view(np.uint8)
    N = w.shape[0]
    sel = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    Ms = M if sel is None else sel.size
    y = np.zeros((Ms, N), dtype=np.float32 if _dt(out_dtype) == F32 else np.uint16)
    codes = np.zeros((M, K * bits // 8), dtype=np.uint8)
    delta = np.zeros(M, dtype=np.float32)
    acc = np.zeros((Ms, N), dtype=np.int32)
    _check(_load().fqo_linear(_p(x), ctypes.c_int(_dt(xdtype)), ctypes.c_int64(M), ctypes.c_int64(K),
                              ctypes.c_int64(K), _p(_f32(g)), ctypes.c_int(beta), ctypes.c_int(bits),
                              ctypes.c_float(clip_ratio), _p(w), _p(_f32(w_scale)), _p(_f32(bias)),
                              ctypes.c_int64(N), _p(sel), ctypes.c_int64(0 if sel is None else sel.size),
                              _p(y), ctypes.c_int(_dt(out_dtype)), ctypes.c_int64(N), _p(codes),
                              _p(delta), _p(acc)), "linear")
    return y, codes, delta, acc


def linear_wonly(x: np.ndarray, xdtype: str, w_codes: np.ndarray, w_scale, bias, bits: int = 4,
                 out_dtype: str = "f32") -> np.ndarray:
    """Weight-only projection with floating-point activations: y = s^W (qW x) + b in binary64."""
    x = _mat(x, xdtype)
    M, K = x.shape
    w = np.ascontiguousarray(w_codes).view(np.uint8)
    N = w.shape[0]
    y = np.zeros((M, N), dtype=np.float32 if _dt(out_dtype) == F32 else np.uint16)
    _check(_load().fqo_linear_wonly(_p(x), ctypes.c_int(_dt(xdtype)), ctypes.c_int64(M), ctypes.c_int64(K),
                                    ctypes.c_int64(K), _p(w), _p(_f32(w_scale)), _p(_f32(bias)),
                                    ctypes.c_int64(N), ctypes.c_int(bits), _p(y), ctypes.c_int(_dt(out_dtype)),
                                    ctypes.c_int64(N)), "linear_wonly")
    return y


def composite_quantize(x: np.ndarray, dtype: str, pre, perm, blocks, bits: int, clip_ratio: float = 1.0,
                       return_z: bool = False):
    """Stored composite rotation R = blockdiag(B_b) Pi: z = R (pre (.) x), then Eq. 5.  ``blocks`` is
    [K/beta, beta, beta]; ``perm[c]`` the source channel of position c.  Returns (codes, delta[, z])."""
    x = _mat(x, dtype)
    M, K = x.shape
    blocks = np.ascontiguousarray(blocks, dtype=np.float32)
    beta = blocks.shape[1]
    assert blocks.shape == (K // beta, beta, beta)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    codes = np.zeros((M, K * bits // 8), dtype=np.uint8)
    delta = np.zeros(M, dtype=np.float32)
    z = np.zeros((M, K), dtype=np.float32) if return_z else None
    _check(_load().fqo_composite_quantize(_p(x), ctypes.c_int(_dt(dtype)), ctypes.c_int64(M), ctypes.c_int64(K),
                                          ctypes.c_int64(K), _p(_f32(pre)), _p(perm), _p(blocks), ctypes.c_int(beta),
                                          ctypes.c_int(bits), ctypes.c_float(clip_ratio), _p(codes), _p(delta), _p(z)),
           "composite_quantize")
    return (codes, delta, z) if return_z else (codes, delta)


def fold_weights_composite(W: np.ndarray, dtype: str, smooth, perm, blocks, bits: int, return_wt: bool = False):
    """Offline fold for a composite rotation: row j of W~ = R (s (.) w_j), RTN, pack.  Returns
    (codes, w_scale[N], mult_g[K] = 1/s (ones without smoothing)[, W~])."""
    K = W.shape[1]
    s = None if smooth is None else _f32(smooth)
    out = composite_quantize(W, dtype, s, perm, blocks, bits, 1.0, return_z=return_wt)
    g = np.ones(K, np.float32) if s is None else (np.float32(1.0) / s).astype(np.float32)
    return (out[0], out[1], g, out[2]) if return_wt else (out[0], out[1], g)


def gptq_factor(z: np.ndarray, damp: float = 0.01):
    """Upper Cholesky factor U of (Z^T Z + lambda I)^-1 (rows of z are transformed calibration tokens) and the
    dead-channel mask, in binary32 as the device computes them.  Returns (U[K, K], dead[K] bool)."""
    z = np.ascontiguousarray(z, dtype=np.float32)
    Mc, K = z.shape
    U = np.zeros((K, K), dtype=np.float32)
    dead = np.zeros(K, dtype=np.uint8)
    _check(_load().fqo_gptq_factor(_p(z), ctypes.c_int64(Mc), ctypes.c_int64(K), ctypes.c_float(damp), _p(U), _p(dead)),
           "gptq_factor")
    return U, dead.astype(bool)


def gptq_round(wt: np.ndarray, U: np.ndarray, dead: np.ndarray, w_scale: np.ndarray, bits: int = 4) -> np.ndarray:
    """The GPTQ sweep over the transformed weights W~ [N, K]; returns int codes [N, K]."""
    w = np.array(wt, dtype=np.float32, order="C", copy=True)
    N, K = w.shape
    codes = np.zeros((N, K), dtype=np.int32)
    _check(_load().fqo_gptq_round(_p(w), ctypes.c_int64(N), ctypes.c_int64(K), _p(np.ascontiguousarray(U, dtype=np.float32)),
                                  _p(np.ascontiguousarray(dead, dtype=np.uint8)), _p(_f32(w_scale)),
                                  ctypes.c_int(7 if bits == 4 else 127), _p(codes)), "gptq_round")
    return codes


def fold_weights_gptq(W: np.ndarray, dtype: str, smooth, beta: int, calib: np.ndarray, calib_dtype: str = "f32",
                      damp: float = 0.01, bits: int = 4, return_all: bool = False):
    """Offline fold with GPTQ rounding (Eq. 7): W~ = W S R^T, Z = T(calibration tokens), sweep, pack.
    Per-output-channel steps are those of the RTN fold (max|W~_j| / q).  Returns (codes, w_scale, mult_g)."""
    _, w_scale, g, wt = fold_weights(W, dtype, smooth, beta, bits, return_wt=True)
    _, _, z = quantize_act(calib, calib_dtype, g, beta, bits, 1.0, return_z=True)
    U, dead = gptq_factor(z, damp)
    q = gptq_round(wt, U, dead, w_scale, bits)
    out = (pack(q, bits), w_scale, g)
    return out + (wt, z, U, dead) if return_all else out


SILU, GELU_TANH = 0, 1


def gate_act(x, act: int) -> np.ndarray:
    """act(x) = x * sigmoid(k(x)) in the fixed binary32 arithmetic of the gated product (elementwise)."""
    lib = _load()
    lib.fqo_gate_act.restype = ctypes.c_float
    xs = np.asarray(x, dtype=np.float32).ravel()
    return np.array([lib.fqo_gate_act(ctypes.c_float(float(v)), ctypes.c_int(act)) for v in xs], dtype=np.float32).reshape(np.shape(x))


def gated_product(gate_up: np.ndarray, dtype: str, act: int) -> np.ndarray:
    """h = act(gate) * up for gate_up [M, 2K] (gate first); binary32 [M, K]."""
    gu = _mat(gate_up, dtype)
    M, K2 = gu.shape
    h = np.zeros((M, K2 // 2), dtype=np.float32)
    _check(_load().fqo_gated_product(_p(gu), ctypes.c_int(_dt(dtype)), ctypes.c_int64(M), ctypes.c_int64(K2 // 2),
                                     ctypes.c_int64(K2), ctypes.c_int(act), _p(h)), "gated_product")
    return h


def quantize_act_gated(gate_up: np.ndarray, dtype: str, act: int, g, beta: int, bits: int, clip_ratio: float = 1.0):
    """Runtime prologue of the site behind a gated MLP: Eq. 5 on T (act(gate) * up)."""
    return quantize_act(gated_product(gate_up, dtype, act), "f32", g, beta, bits, clip_ratio)
