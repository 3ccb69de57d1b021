"""Shared helpers of the GPU parity tests: numpy <-> device tensors, the oracle
side of a site, and the floating-point comparison rule."""
import numpy as np
import torch

import oracle
from paper_2609_24433_b200 import synth

TOL = {"f32": 1e-3, "bf16": 1e-2}   # relative tolerance on outputs: 1e-3 for binary32, 1e-2 for bfloat16


def to_dev(a: np.ndarray, dtype: str = "f32") -> torch.Tensor:
    if a is None:
        return None
    if dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.contiguous().cpu().numpy()


def as_f64(y: np.ndarray) -> np.ndarray:
    return synth.bf16_bits_to_f32(y).astype(np.float64) if y.dtype == np.uint16 else y.astype(np.float64)


def assert_close(y_gpu: np.ndarray, y_ref: np.ndarray, dtype: str, what: str = ""):
    """|y_gpu - y| <= tol * max(|y|, rms(y_row)): relative, with a per-row floor so that entries
    where the bias cancels the product do not raise false alarms."""
    g, r = as_f64(y_gpu), as_f64(y_ref)
    assert g.shape == r.shape, (what, g.shape, r.shape)
    floor = np.sqrt((r ** 2).mean(axis=1, keepdims=True))
    bound = TOL[dtype] * np.maximum(np.abs(r), floor)
    bad = np.abs(g - r) > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outputs outside tolerance, worst " \
                          f"{(np.abs(g - r) / np.maximum(bound, 1e-300)).max():.3g}x"


def oracle_smooth(data: synth.SiteData):
    """SmoothQuant scale of a site from its calibration batch and ALL its consumers' weights."""
    site = data.site
    if site.alpha is None:
        return None
    a = oracle.col_absmax(data.calib)
    w = None
    for name, _ in site.consumers:
        wc = oracle.col_absmax(data.W[name])
        w = wc if w is None else np.maximum(w, wc)
    return oracle.smooth_scale(a, w, site.alpha)


def concat_consumers(data: synth.SiteData):
    W = np.concatenate([data.W[n] for n, _ in data.site.consumers], axis=0)
    b = np.concatenate([data.bias[n] for n, _ in data.site.consumers], axis=0)
    return W, b
