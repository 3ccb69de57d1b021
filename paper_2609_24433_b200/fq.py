"""ctypes binding of the C-ABI library (include/fq.h), same names without the ``fq_`` prefix.

Argument marshalling only: every function below turns torch CUDA tensors into
device pointers, calls the library on torch's current stream and wraps the
outputs.  There is no Python, torch or CPU implementation of any step here; if
the shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfq_b200.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ARCH, ERR_CUDA, ERR_NOMEM, ERR_TIMEOUT = range(8)
F32, BF16 = 0, 1

EXPORTS = [
    "fq_status_string", "fq_fold_weights", "fq_weights_destroy", "fq_weights_info", "fq_weights_multiplier",
    "fq_weights_export", "fq_weights_import", "fq_col_absmax", "fq_smooth_scale", "fq_quantize_act",
    "fq_gemm_w4a4", "fq_gemm_w8a8", "fq_linear_w4a4", "fq_linear_w8a8", "fq_workspace_bytes",
    "fq_gemm_acc_i32", "fq_gemm_simt", "fq_device_status", "fq_profile_mark", "fq_linear_w4a4_static",
    "fq_fold_weights_after", "fq_weights_fold_after", "fq_weights_import_after", "fq_quantize_act_after",
    "fq_weights_set_multiplier", "fq_weights_scale_outputs", "fq_linear_w4a16",
    "fq_fold_weights_composite", "fq_quantize_act_composite", "fq_weights_composite", "fq_fold_weights_gptq",
    "fq_quantize_act_gated", "fq_linear_gated", "fq_watchdog_selftest",
]

_lib = None


class FqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (fq_status {status})")


def lib() -> ctypes.CDLL:
    """Load the CUDA library; fail loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_24433_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.fq_status_string.restype = ctypes.c_char_p
        L.fq_status_string.argtypes = [ctypes.c_int]
        L.fq_weights_multiplier.restype = ctypes.c_void_p
        L.fq_weights_multiplier.argtypes = [ctypes.c_void_p]
        L.fq_weights_fold_after.restype = ctypes.c_int
        L.fq_weights_fold_after.argtypes = [ctypes.c_void_p]
        L.fq_weights_composite.restype = ctypes.c_int
        L.fq_weights_composite.argtypes = [ctypes.c_void_p]
        L.fq_workspace_bytes.restype = ctypes.c_size_t
        L.fq_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().fq_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        raise FqError(status, what)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _out_dt(dtype: torch.dtype) -> int:
    return {torch.float32: F32, torch.bfloat16: BF16}[dtype]


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _rowmajor(t: torch.Tensor) -> torch.Tensor:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit inner stride")
    return t


class Weights:
    """Owner of an ``fq_weights`` handle."""

    def __init__(self, handle: int):
        self._h = ctypes.c_void_p(handle)
        n, k = ctypes.c_int64(), ctypes.c_int64()
        blk, bits = ctypes.c_int(), ctypes.c_int()
        _check(lib().fq_weights_info(self._h, ctypes.byref(n), ctypes.byref(k), ctypes.byref(blk),
                                     ctypes.byref(bits)), "fq_weights_info")
        self.N, self.K, self.block, self.bits = n.value, k.value, blk.value, bits.value
        self.fold_after = bool(lib().fq_weights_fold_after(self._h))

    @property
    def handle(self) -> ctypes.c_void_p:
        if self._h is None:
            raise RuntimeError("weights handle already destroyed")
        return self._h

    def multiplier_ptr(self) -> int:
        return int(lib().fq_weights_multiplier(self.handle) or 0)

    def export(self) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
        """(codes u8 [N, K*bits/8], w_scale [N], mult_g [K], bias [N]) as new device tensors."""
        dev = torch.device("cuda", torch.cuda.current_device())
        codes = torch.empty((self.N, self.K * self.bits // 8), dtype=torch.uint8, device=dev)
        ws = torch.empty(self.N, dtype=torch.float32, device=dev)
        g = torch.empty(self.K, dtype=torch.float32, device=dev)
        b = torch.empty(self.N, dtype=torch.float32, device=dev)
        _check(lib().fq_weights_export(self.handle, _ptr(codes), _ptr(ws), _ptr(g), _ptr(b), _stream()),
               "fq_weights_export")
        return codes, ws, g, b

    def set_multiplier(self, mult: Optional[torch.Tensor]):
        """Replace the runtime multiplier (None: the constant block^-1/2); offline."""
        _check(lib().fq_weights_set_multiplier(self.handle, _ptr(mult), _stream()), "fq_weights_set_multiplier")

    def scale_outputs(self, first: int, d: torch.Tensor):
        """s^W_j *= d_j, b_j *= d_j for output channels first .. first + len(d); offline."""
        _check(lib().fq_weights_scale_outputs(self.handle, ctypes.c_int64(first), ctypes.c_int64(d.numel()),
                                              _ptr(d), _stream()), "fq_weights_scale_outputs")

    def destroy(self):
        if self._h is not None:
            lib().fq_weights_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def fold_weights(W: torch.Tensor, smooth: Optional[torch.Tensor], bias: Optional[torch.Tensor],
                 hadamard_block: int, bits: int) -> Weights:
    W = _rowmajor(W)
    out = ctypes.c_void_p()
    _check(lib().fq_fold_weights(_ptr(W), _dt(W), ctypes.c_int64(W.shape[0]), ctypes.c_int64(W.shape[1]),
                                 ctypes.c_int64(W.stride(0)), _ptr(smooth), _ptr(bias),
                                 ctypes.c_int(hadamard_block), ctypes.c_int(bits), _stream(), ctypes.byref(out)),
           "fq_fold_weights")
    return Weights(out.value)


def fold_weights_after(W: torch.Tensor, post_scale: torch.Tensor, bias: Optional[torch.Tensor],
                       hadamard_block: int, bits: int) -> Weights:
    """Fold-after variant: W~ = W R^T P; the handle's multiplier 1/p is applied behind the rotation."""
    W = _rowmajor(W)
    out = ctypes.c_void_p()
    _check(lib().fq_fold_weights_after(_ptr(W), _dt(W), ctypes.c_int64(W.shape[0]), ctypes.c_int64(W.shape[1]),
                                       ctypes.c_int64(W.stride(0)), _ptr(post_scale), _ptr(bias),
                                       ctypes.c_int(hadamard_block), ctypes.c_int(bits), _stream(),
                                       ctypes.byref(out)), "fq_fold_weights_after")
    return Weights(out.value)


def fold_weights_gptq(W: torch.Tensor, smooth: Optional[torch.Tensor], bias: Optional[torch.Tensor], calib: torch.Tensor,
                      hadamard_block: int, bits: int = 4, damp: float = 0.01) -> Weights:
    """Fold-before with GPTQ rounding in transformed coordinates (Eq. 7); ``calib``: [Mc, K] calibration tokens of
    the site in original coordinates."""
    W, calib = _rowmajor(W), _rowmajor(calib)
    out = ctypes.c_void_p()
    _check(lib().fq_fold_weights_gptq(_ptr(W), _dt(W), ctypes.c_int64(W.shape[0]), ctypes.c_int64(W.shape[1]),
                                      ctypes.c_int64(W.stride(0)), _ptr(smooth), _ptr(bias), _ptr(calib), _dt(calib),
                                      ctypes.c_int64(calib.shape[0]), ctypes.c_int64(calib.stride(0)),
                                      ctypes.c_int(hadamard_block), ctypes.c_int(bits), ctypes.c_float(damp), _stream(),
                                      ctypes.byref(out)), "fq_fold_weights_gptq")
    return Weights(out.value)


def fold_weights_composite(W: torch.Tensor, smooth: Optional[torch.Tensor], bias: Optional[torch.Tensor],
                           perm: torch.Tensor, blocks: torch.Tensor, bits: int) -> Weights:
    """Fold with a stored composite rotation R = blockdiag(B_b) Pi: rows R (s (.) w_j), RTN, pack.
    ``perm``: int32[K] source channels; ``blocks``: float32[K/beta, beta, beta]."""
    W = _rowmajor(W)
    assert perm.dtype == torch.int32 and blocks.dtype == torch.float32 and blocks.is_contiguous()
    out = ctypes.c_void_p()
    _check(lib().fq_fold_weights_composite(_ptr(W), _dt(W), ctypes.c_int64(W.shape[0]), ctypes.c_int64(W.shape[1]),
                                           ctypes.c_int64(W.stride(0)), _ptr(smooth), _ptr(bias), _ptr(perm), _ptr(blocks),
                                           ctypes.c_int(blocks.shape[1]), ctypes.c_int(bits), _stream(),
                                           ctypes.byref(out)), "fq_fold_weights_composite")
    return Weights(out.value)


def quantize_act_composite(x: torch.Tensor, mult_g, perm: torch.Tensor, blocks: torch.Tensor, bits: int,
                           clip_ratio: float = 1.0, codes: Optional[torch.Tensor] = None,
                           delta: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """Runtime prologue of a composite-rotation site: z = R ((1/s) (.) x), then Eq. 5.  ``mult_g``: device
    float tensor, a Weights (its multiplier) or None.  ``workspace``: uint8 tensor of at least 4*M*K bytes."""
    x = _rowmajor(x)
    M, K = x.shape
    assert perm.dtype == torch.int32 and blocks.dtype == torch.float32 and blocks.is_contiguous()
    if codes is None:
        codes = torch.empty((M, K * bits // 8), dtype=torch.uint8, device=x.device)
    if delta is None:
        delta = torch.empty(M, dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(16, 4 * M * K), dtype=torch.uint8, device=x.device)
    g = ctypes.c_void_p(mult_g.multiplier_ptr()) if isinstance(mult_g, Weights) else _ptr(mult_g)
    _check(lib().fq_quantize_act_composite(_ptr(x), _dt(x), ctypes.c_int64(M), ctypes.c_int64(K), ctypes.c_int64(x.stride(0)),
                                           g, _ptr(perm), _ptr(blocks), ctypes.c_int(blocks.shape[1]), ctypes.c_int(bits),
                                           ctypes.c_float(clip_ratio), _ptr(codes), _ptr(delta), _ptr(workspace),
                                           ctypes.c_size_t(workspace.numel()), _stream()), "fq_quantize_act_composite")
    return codes, delta


def weights_import(codes: torch.Tensor, w_scale: torch.Tensor, mult_g: Optional[torch.Tensor],
                   bias: Optional[torch.Tensor], K: int, hadamard_block: int, bits: int,
                   fold_after: bool = False) -> Weights:
    out = ctypes.c_void_p()
    fn_name = "fq_weights_import_after" if fold_after else "fq_weights_import"
    _check(getattr(lib(), fn_name)(_ptr(codes), _ptr(w_scale), _ptr(mult_g), _ptr(bias),
                                   ctypes.c_int64(codes.shape[0]), ctypes.c_int64(K),
                                   ctypes.c_int(hadamard_block), ctypes.c_int(bits), _stream(), ctypes.byref(out)),
           fn_name)
    return Weights(out.value)


def col_absmax(x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Per-channel max |x| over rows; pass ``out`` to accumulate over several matrices."""
    x = _rowmajor(x)
    acc = out is not None
    if out is None:
        out = torch.empty(x.shape[1], dtype=torch.float32, device=x.device)
    _check(lib().fq_col_absmax(_ptr(x), _dt(x), ctypes.c_int64(x.shape[0]), ctypes.c_int64(x.shape[1]),
                               ctypes.c_int64(x.stride(0)), ctypes.c_int(1 if acc else 0), _ptr(out), _stream()),
           "fq_col_absmax")
    return out


def smooth_scale(a: torch.Tensor, w: torch.Tensor, alpha: float) -> torch.Tensor:
    s = torch.empty_like(a)
    _check(lib().fq_smooth_scale(_ptr(a), _ptr(w), ctypes.c_int64(a.numel()), ctypes.c_double(alpha), _ptr(s),
                                 _stream()), "fq_smooth_scale")
    return s


def quantize_act(x: torch.Tensor, mult_g, hadamard_block: int, bits: int, clip_ratio: float = 1.0,
                 codes: Optional[torch.Tensor] = None, delta: Optional[torch.Tensor] = None,
                 fold_after: Optional[bool] = None):
    """Runtime prologue. ``mult_g``: device float tensor, a Weights (its multiplier) or None.
    ``fold_after``: the multiplier is the post-rotation 1/p (default: what the Weights says, else False)."""
    x = _rowmajor(x)
    M, K = x.shape
    if codes is None:
        codes = torch.empty((M, K * bits // 8), dtype=torch.uint8, device=x.device)
    if delta is None:
        delta = torch.empty(M, dtype=torch.float32, device=x.device)
    if isinstance(mult_g, Weights):
        g = ctypes.c_void_p(mult_g.multiplier_ptr())
        if fold_after is None:
            fold_after = mult_g.fold_after
    else:
        g = _ptr(mult_g)
    fn_name = "fq_quantize_act_after" if fold_after else "fq_quantize_act"
    _check(getattr(lib(), fn_name)(_ptr(x), _dt(x), ctypes.c_int64(M), ctypes.c_int64(K), ctypes.c_int64(x.stride(0)),
                                   g, ctypes.c_int(hadamard_block), ctypes.c_int(bits), ctypes.c_float(clip_ratio),
                                   _ptr(codes), _ptr(delta), _stream()), fn_name)
    return codes, delta


def workspace_bytes(M: int, K: int, N: int, bits: int) -> int:
    return int(lib().fq_workspace_bytes(M, K, N, bits))


def _workspace(M: int, W: Weights, workspace: Optional[torch.Tensor], device) -> torch.Tensor:
    need = workspace_bytes(M, W.K, W.N, W.bits)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace


def _gemm(fn_name: str, a_codes, a_delta, W: Weights, out_dtype, y, workspace):
    M = a_codes.shape[0]
    if y is None:
        y = torch.empty((M, W.N), dtype=out_dtype, device=a_codes.device)
    ws = _workspace(M, W, workspace, a_codes.device)
    fn = getattr(lib(), fn_name)
    _check(fn(_ptr(a_codes), _ptr(a_delta), ctypes.c_int64(M), W.handle, _ptr(y), _out_dt(y.dtype),
              ctypes.c_int64(y.stride(0)), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), fn_name)
    return y


def gemm_w4a4(a_codes, a_delta, W: Weights, out_dtype=torch.float32, y=None, workspace=None):
    return _gemm("fq_gemm_w4a4", a_codes, a_delta, W, out_dtype, y, workspace)


def gemm_w8a8(a_codes, a_delta, W: Weights, out_dtype=torch.float32, y=None, workspace=None):
    return _gemm("fq_gemm_w8a8", a_codes, a_delta, W, out_dtype, y, workspace)


def _linear(fn_name: str, x, W: Weights, clip_ratio, out_dtype, y, workspace):
    x = _rowmajor(x)
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, W.N), dtype=out_dtype, device=x.device)
    ws = _workspace(M, W, workspace, x.device)
    fn = getattr(lib(), fn_name)
    _check(fn(_ptr(x), _dt(x), ctypes.c_int64(M), ctypes.c_int64(x.stride(0)), W.handle, ctypes.c_float(clip_ratio),
              _ptr(y), _out_dt(y.dtype), ctypes.c_int64(y.stride(0)), _ptr(ws), ctypes.c_size_t(ws.numel()),
              _stream()), fn_name)
    return y


def linear_w4a4(x, W: Weights, clip_ratio: float = 1.0, out_dtype=torch.float32, y=None, workspace=None):
    return _linear("fq_linear_w4a4", x, W, clip_ratio, out_dtype, y, workspace)


def linear_w8a8(x, W: Weights, clip_ratio: float = 1.0, out_dtype=torch.float32, y=None, workspace=None):
    return _linear("fq_linear_w8a8", x, W, clip_ratio, out_dtype, y, workspace)


STATIC_MAX_CODE_BYTES = 4 << 20
STATIC_MAX_TOKENS = 16384


def linear_w4a4_static(x, W: Weights, clip_ratio: float = 1.0, out_dtype=torch.float32, y=None):
    """fq_linear_w4a4 on the library's built-in scratch: for callers that cannot allocate device
    memory at call time.  Only the output tensor is created here when ``y`` is not passed in, and
    the entry point itself allocates nothing; M*K must fit STATIC_MAX_CODE_BYTES."""
    x = _rowmajor(x)
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, W.N), dtype=out_dtype, device=x.device)
    _check(lib().fq_linear_w4a4_static(_ptr(x), _dt(x), ctypes.c_int64(M), ctypes.c_int64(x.stride(0)), W.handle,
                                       ctypes.c_float(clip_ratio), _ptr(y), _out_dt(y.dtype),
                                       ctypes.c_int64(y.stride(0)), _stream()), "fq_linear_w4a4_static")
    return y


GATE_SILU, GATE_GELU_TANH = 0, 1


def quantize_act_gated(gate_up: torch.Tensor, act: int, mult_g, hadamard_block: int, bits: int, clip_ratio: float = 1.0):
    """Prologue of the site behind a gated MLP: Eq. 5 on T (act(gate) * up); gate_up is [M, 2K], gate first."""
    gate_up = _rowmajor(gate_up)
    M, K = gate_up.shape[0], gate_up.shape[1] // 2
    codes = torch.empty((M, K * bits // 8), dtype=torch.uint8, device=gate_up.device)
    delta = torch.empty(M, dtype=torch.float32, device=gate_up.device)
    g = ctypes.c_void_p(mult_g.multiplier_ptr()) if isinstance(mult_g, Weights) else _ptr(mult_g)
    _check(lib().fq_quantize_act_gated(_ptr(gate_up), _dt(gate_up), ctypes.c_int64(M), ctypes.c_int64(K),
                                       ctypes.c_int64(gate_up.stride(0)), ctypes.c_int(act), g, ctypes.c_int(hadamard_block),
                                       ctypes.c_int(bits), ctypes.c_float(clip_ratio), _ptr(codes), _ptr(delta), _stream()),
           "fq_quantize_act_gated")
    return codes, delta


def linear_gated(gate_up: torch.Tensor, act: int, W: Weights, clip_ratio: float = 1.0, out_dtype=torch.float32, y=None,
                 workspace=None):
    """down_proj with the gate product fused into its prologue: y = linear(act(gate) * up)."""
    gate_up = _rowmajor(gate_up)
    M = gate_up.shape[0]
    if y is None:
        y = torch.empty((M, W.N), dtype=out_dtype, device=gate_up.device)
    ws = _workspace(M, W, workspace, gate_up.device)
    _check(lib().fq_linear_gated(_ptr(gate_up), _dt(gate_up), ctypes.c_int64(M), ctypes.c_int64(gate_up.stride(0)),
                                 ctypes.c_int(act), W.handle, ctypes.c_float(clip_ratio), _ptr(y), _out_dt(y.dtype),
                                 ctypes.c_int64(y.stride(0)), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "fq_linear_gated")
    return y


def linear_w4a16(x, W: Weights, out_dtype=torch.float32, y=None):
    """Weight-only 4-bit projection of float activations: y = s^W (qW x) + b (no quantization of x)."""
    x = _rowmajor(x)
    M = x.shape[0]
    if y is None:
        y = torch.empty((M, W.N), dtype=out_dtype, device=x.device)
    _check(lib().fq_linear_w4a16(_ptr(x), _dt(x), ctypes.c_int64(M), ctypes.c_int64(x.stride(0)), W.handle,
                                 _ptr(y), _out_dt(y.dtype), ctypes.c_int64(y.stride(0)), _stream()), "fq_linear_w4a16")
    return y


def linear(x, W: Weights, clip_ratio: float = 1.0, out_dtype=torch.float32, y=None, workspace=None):
    """Dispatch on the handle's bit width (the two entry points differ in nothing else)."""
    return (linear_w4a4 if W.bits == 4 else linear_w8a8)(x, W, clip_ratio, out_dtype, y, workspace)


def gemm_acc_i32(a_codes, W: Weights, workspace=None) -> torch.Tensor:
    M = a_codes.shape[0]
    acc = torch.empty((M, W.N), dtype=torch.int32, device=a_codes.device)
    ws = _workspace(M, W, workspace, a_codes.device)
    _check(lib().fq_gemm_acc_i32(_ptr(a_codes), ctypes.c_int64(M), W.handle, _ptr(acc), _ptr(ws),
                                 ctypes.c_size_t(ws.numel()), _stream()), "fq_gemm_acc_i32")
    return acc


def gemm_simt(a_codes, a_delta, W: Weights, out_dtype=torch.float32, raw_acc: bool = False, workspace=None):
    M = a_codes.shape[0]
    ws = _workspace(M, W, workspace, a_codes.device)
    if raw_acc:
        acc = torch.empty((M, W.N), dtype=torch.int32, device=a_codes.device)
        y = None
    else:
        acc = None
        y = torch.empty((M, W.N), dtype=out_dtype, device=a_codes.device)
    _check(lib().fq_gemm_simt(_ptr(a_codes), _ptr(a_delta), ctypes.c_int64(M), W.handle, _ptr(y),
                              _out_dt(out_dtype), ctypes.c_int64(W.N if y is None else y.stride(0)), _ptr(acc),
                              _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "fq_gemm_simt")
    return acc if raw_acc else y


def profile_mark(event: Optional[torch.cuda.Event]):
    """Record ``event`` between the prologue and the GEMM of every linear_* call (None = off)."""
    if event is not None and not event.cuda_event:
        event.record()      # torch creates the underlying cudaEvent_t lazily, on its first record
    _check(lib().fq_profile_mark(ctypes.c_void_p(0 if event is None else event.cuda_event)), "fq_profile_mark")


def watchdog_selftest(limit_ns: int = 2_000_000):
    """Enqueue the one-warp kernel whose bounded wait is certain to expire after ``limit_ns``; the next
    device_status() then reports ERR_TIMEOUT once."""
    _check(lib().fq_watchdog_selftest(ctypes.c_uint64(limit_ns), _stream()), "fq_watchdog_selftest")


def device_status() -> Tuple[int, int]:
    """Synchronise and return (status, raw watchdog word)."""
    word = ctypes.c_uint32(0)
    st = lib().fq_device_status(ctypes.byref(word))
    return int(st), int(word.value)
