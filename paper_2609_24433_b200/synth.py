"""Seeded synthetic inputs shaped like the paper's GR00T / pi0.5 projection sites.

This module only draws random tensors and converts storage types.  It holds
none of the method's arithmetic (no transform, no quantizer, no scale rule) and
imports nothing from the CUDA binding or from the CPU oracle, so both sides can
be fed from it.

bfloat16 tensors are carried as numpy ``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np


# ----------------------------------------------------------------------------
# storage-type helpers
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even) and return the raw uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_dtype(x_f32: np.ndarray, dtype: str) -> np.ndarray:
    """float32 -> the storage array for ``dtype`` ('f32' | 'bf16')."""
    if dtype == "f32":
        return np.ascontiguousarray(x_f32, dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(x_f32)
    raise ValueError(dtype)


def to_f32(x: np.ndarray, dtype: str) -> np.ndarray:
    return x.astype(np.float32) if dtype == "f32" else bf16_bits_to_f32(x)


# ----------------------------------------------------------------------------
# site description
# ----------------------------------------------------------------------------
@dataclass
class Site:
    """One shared activation site with its consumer projections."""
    name: str
    M: int
    K: int
    consumers: List[Tuple[str, int]]          # (projection name, N)
    beta: int
    bits: int
    x_dtype: str = "bf16"
    y_dtype: str = "bf16"
    alpha: Optional[float] = None             # smoothing exponent, None = no smoothing
    outlier_frac: float = 0.01
    outlier_kind: str = "student_t"           # 'student_t' | 'scale'
    outlier_gain: float = 30.0
    sigma: float = 1.0
    fold_after: bool = False                  # the site's diagonal sits behind the rotation (T = P^-1 R)
    composite: bool = False                   # stored composite rotation instead of the butterflies

    @property
    def N_total(self) -> int:
        return sum(n for _, n in self.consumers)


@dataclass
class SiteData:
    site: Site
    x: np.ndarray                 # [M, K] storage dtype of site.x_dtype
    calib: Optional[np.ndarray]   # [Mc, K] float32 calibration batch (disjoint seed) or None
    W: Dict[str, np.ndarray] = field(default_factory=dict)      # name -> [N, K] float32
    bias: Dict[str, np.ndarray] = field(default_factory=dict)   # name -> [N] float32
    outlier_channels: Optional[np.ndarray] = None


def outlier_channels(rng: np.random.Generator, K: int, frac: float, minimum: int = 8) -> np.ndarray:
    n = max(minimum, int(round(frac * K)))
    n = min(n, K)
    return np.sort(rng.choice(K, n, replace=False))


def draw_acts(rng: np.random.Generator, M: int, K: int, channels: np.ndarray, kind: str,
              gain: float, sigma: float = 1.0) -> np.ndarray:
    """Gaussian base with outlier channels: either scaled Gaussians ('scale') or
    heavy-tailed Student-t(df=3) entries times ``gain`` ('student_t')."""
    x = rng.standard_normal((M, K), dtype=np.float32)
    if channels.size:
        if kind == "scale":
            x[:, channels] *= np.float32(gain)
        elif kind == "student_t":
            x[:, channels] = (gain * rng.standard_t(3.0, size=(M, channels.size))).astype(np.float32)
        else:
            raise ValueError(kind)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return x


def draw_weights(rng: np.random.Generator, N: int, K: int, std: float = 0.02) -> np.ndarray:
    return (std * rng.standard_normal((N, K), dtype=np.float32)).astype(np.float32)


def make_site(site: Site, seed: int, calib_tokens: int = 256, with_weights: bool = True) -> SiteData:
    rng = np.random.default_rng(seed)
    ch = outlier_channels(rng, site.K, site.outlier_frac)
    x = draw_acts(rng, site.M, site.K, ch, site.outlier_kind, site.outlier_gain, site.sigma)
    data = SiteData(site=site, x=as_dtype(x, site.x_dtype), calib=None, outlier_channels=ch)
    if with_weights:
        for name, n in site.consumers:
            data.W[name] = draw_weights(rng, n, site.K)
            data.bias[name] = (0.02 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
    if site.alpha is not None:
        crng = np.random.default_rng(seed + 100003)     # disjoint calibration stream
        data.calib = draw_acts(crng, calib_tokens, site.K, ch, site.outlier_kind, site.outlier_gain,
                               site.sigma)
    return data


# ----------------------------------------------------------------------------
# the five workload families
# ----------------------------------------------------------------------------
def config1_site() -> Site:
    """Single W4A4 linear, fp32 in/out, 8 outlier channels scaled x50, alpha = 0.5."""
    return Site("single", M=64, K=1024, consumers=[("proj", 1024)], beta=128, bits=4,
                x_dtype="f32", y_dtype="f32", alpha=0.5, outlier_frac=8 / 1024,
                outlier_kind="scale", outlier_gain=50.0)


def backbone_layer_sites(selective_int8: bool = True, M: int = 816, hidden: int = 2048,
                         mlp: int = 16384, kv: int = 256) -> List[Site]:
    """pi0.5-like language-backbone layer: four activation sites, seven projections."""
    od_bits = 8 if selective_int8 else 4
    return [
        Site("qkv", M, hidden, [("q_proj", hidden), ("k_proj", kv), ("v_proj", kv)], beta=128, bits=4,
             alpha=0.5, outlier_frac=0.01),
        Site("o", M, hidden, [("o_proj", hidden)], beta=128, bits=od_bits, alpha=None,
             outlier_frac=0.01),
        Site("gate_up", M, hidden, [("gate_proj", mlp), ("up_proj", mlp)], beta=128, bits=4,
             alpha=0.5, outlier_frac=0.01),
        Site("down", M, mlp, [("down_proj", hidden)], beta=256, bits=od_bits, alpha=None,
             outlier_frac=0.005),
    ]


def expert_layer_sites(M: int = 50, width: int = 1024, mlp: int = 4096, sigma: float = 1.0) -> List[Site]:
    """Action-expert layer: W4A4 everywhere, Hadamard block 64, 0.5 % outlier channels x20."""
    kw = dict(beta=64, bits=4, alpha=None, outlier_frac=0.005, outlier_kind="scale",
              outlier_gain=20.0, sigma=sigma)
    return [
        Site("qkv", M, width, [("q_proj", width), ("k_proj", width), ("v_proj", width)], **kw),
        Site("o", M, width, [("o_proj", width)], **kw),
        Site("gate_up", M, width, [("gate_proj", mlp), ("up_proj", mlp)], **kw),
        Site("down", M, mlp, [("down_proj", width)], **kw),
    ]


def sweep_site(M: int, K: int, N: int, beta: int, bits: int, fold_after: bool = False, composite: bool = False) -> Site:
    tag = "_after" if fold_after else ("_composite" if composite else "")
    return Site(f"sweep_m{M}_k{K}_n{N}_b{beta}_w{bits}" + tag, M, K, [("proj", N)],
                beta=beta, bits=bits, alpha=None, outlier_frac=0.005, outlier_kind="scale", outlier_gain=30.0,
                fold_after=fold_after, composite=composite)


def post_scale(site: Site, seed: int) -> np.ndarray:
    """Positive post-rotation diagonal P of a fold-after site: log-uniform in [1/e, e] (stands in for a
    calibrated one; the kernels do not care where it came from)."""
    rng = np.random.default_rng(seed + 424243)
    return np.exp(rng.uniform(-1.0, 1.0, site.K)).astype(np.float32)


def expert_step_sigma(step: int, steps: int = 10) -> float:
    """Activation scale drifting from 1.0 to 0.1 over the denoising steps."""
    if steps <= 1:
        return 1.0
    return 1.0 - 0.9 * step / (steps - 1)


# ----------------------------------------------------------------------------
# stored composite rotation: a stand-in for the calibration that produces it
# ----------------------------------------------------------------------------
def composite_rotation(K: int, beta: int, seed: int, calib: Optional[np.ndarray] = None):
    """A permutation and per-block orthogonal matrices shaped like the paper's stored composite
    rotation: channels ranked by calibrated magnitude are dealt to the blocks in zigzag order
    (0, 1, .., B-1, B-1, .., 1, 0, 0, 1, ..) so that every block receives a mix of large and small
    channels, and each block's matrix is a normalised Hadamard matrix applied after the block's
    principal axes (beta^-1/2 H U^T, U from an SVD of the block's calibration columns).  Without a
    calibration batch the ranking is random and U is a random orthogonal matrix.
    Returns (perm int32[K], blocks float32[K/beta, beta, beta])."""
    rng = np.random.default_rng(seed)
    nb = K // beta
    order = np.argsort(-np.abs(calib).max(axis=0), kind="stable") if calib is not None else rng.permutation(K)
    perm = np.empty(K, dtype=np.int32)
    fill = np.zeros(nb, dtype=np.int64)
    for rank, c in enumerate(order):
        r, pos = divmod(rank, nb)
        b = pos if r % 2 == 0 else nb - 1 - pos
        perm[b * beta + fill[b]] = c
        fill[b] += 1
    H = np.array([[1.0]])
    while H.shape[0] < beta:
        H = np.block([[H, H], [H, -H]])
    H = H / np.sqrt(beta)
    blocks = np.empty((nb, beta, beta), dtype=np.float32)
    for b in range(nb):
        if calib is not None and calib.shape[0] >= beta:
            cols = calib[:, perm[b * beta:(b + 1) * beta]].astype(np.float64)
            U = np.linalg.svd(cols.T @ cols)[0]
        else:
            U = np.linalg.qr(rng.standard_normal((beta, beta)))[0]
        blocks[b] = (H @ U.T).astype(np.float32)
    return perm, blocks
