"""Thin ctypes binding of libstamp.so: same names as the C ABI (include/stamp.h), argument
marshalling only.  Tensors are torch CUDA tensors used as plain device buffers; every step of the
layer runs inside the CUDA library.  There is no CPU fallback: if the library is missing or a
call fails, an exception is raised."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .build import LIB_PATH

STAMP_OK = 0
F32, BF16 = 0, 1
T_IDENTITY, T_HAAR, T_DCT2, T_HAAR2D, T_WHT, T_HAAR_SKIP1 = 0, 1, 2, 3, 4, 5
G_PER_TOKEN, G_PER_CHANNEL, G_GROUP = 0, 1, 2
W_PACKED4, W_INT8, W_INT8_AND_PACKED4 = 0, 1, 2

EXPORTS = (
    "stamp_workspace_bytes", "stamp_quantize_weights", "stamp_prepare_weights", "stamp_quantize",
    "stamp_linear", "stamp_inverse", "stamp_linear_fused", "stamp_workspace_bytes_host",
    "stamp_linear_fused_host", "stamp_profile_gemm_events", "stamp_debug_transform",
    "stamp_debug_unpack_codes", "stamp_debug_gemm_i32", "stamp_last_device_status",
    "stamp_last_launch_count", "stamp_status_string", "stamp_inverse_noalloc", "stamp_debug_fused_operand",
    "stamp_measure_i8_mma_issue", "stamp_debug_expire_wait",
    "stamp_dequantize", "stamp_prepare_weights_both",
)


class StampConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("transform", "block", "levels", "k_hi", "bits_hi", "bits_lo",
                                              "bits_w", "act_gran", "w_gran", "grid_w", "act_zero_point", "group")]


def make_config(transform: int, block: int = 0, levels: int = 0, k_hi: int = 64, bits_hi: int = 8,
                bits_lo: int = 4, bits_w: int = 4, grid_w: int = 0, zero_point: bool = False,
                group: int = 0) -> StampConfig:
    """grid_w: width of the patch grid for T_HAAR2D (0 for the other transforms); zero_point: activation
    codes with a per-token zero point and min-max range instead of the symmetric ones; group: features per
    scale for activations and weights (0: one scale per token / per output channel)."""
    gran = (G_GROUP, G_GROUP) if group else (G_PER_TOKEN, G_PER_CHANNEL)
    return StampConfig(transform, block, levels, k_hi, bits_hi, bits_lo, bits_w, gran[0], gran[1],
                       grid_w if transform == T_HAAR2D else 0, 1 if zero_point else 0, group)


class StampError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by paper_2510_26771_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"CUDA library not built: {LIB_PATH} is missing "
                               "(run `python -m paper_2510_26771_b200.build`); there is no fallback path")
        _lib = ctypes.CDLL(LIB_PATH)
        _lib.stamp_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            getattr(_lib, name)
    return _lib


def status_string(status: int) -> str:
    return lib().stamp_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise ValueError(f"unsupported dtype {t.dtype}")


def _check(rc: int, what: str) -> None:
    if rc != STAMP_OK:
        raise StampError(rc, what)


def _ws_args(ws: torch.Tensor):
    return _ptr(ws), ctypes.c_size_t(ws.numel() * ws.element_size())


def stamp_workspace_bytes(cfg: StampConfig, B: int, L: int, K: int, N: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stamp_workspace_bytes(ctypes.byref(cfg), B, L, K, N, ctypes.byref(out)), "stamp_workspace_bytes")
    return int(out.value)


def alloc_workspace(cfg: StampConfig, B: int, L: int, K: int, N: int, device="cuda") -> torch.Tensor:
    return torch.empty(stamp_workspace_bytes(cfg, B, L, K, N), dtype=torch.uint8, device=device)


def stamp_quantize_weights(cfg: StampConfig, W: torch.Tensor):
    N, K = W.shape
    wq = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    w_scale = torch.empty((N, K // cfg.group) if cfg.group else (N,), dtype=torch.float32, device=W.device)
    _check(lib().stamp_quantize_weights(ctypes.byref(cfg), _ptr(W), _dtype_code(W), N, K, _ptr(wq), _ptr(w_scale),
                                        _stream()), "stamp_quantize_weights")
    return wq, w_scale


def stamp_prepare_weights(cfg: StampConfig, wq: torch.Tensor) -> torch.Tensor:
    N, K2 = wq.shape
    w8 = torch.empty((N, 2 * K2), dtype=torch.int8, device=wq.device)
    _check(lib().stamp_prepare_weights(ctypes.byref(cfg), _ptr(wq), N, 2 * K2, _ptr(w8), _stream()),
           "stamp_prepare_weights")
    return w8


def stamp_prepare_weights_both(cfg: StampConfig, wq: torch.Tensor) -> torch.Tensor:
    """Expanded int8 codes [N, K] followed by the packed ones [N, K/2] in one buffer of N * K * 3 / 2 bytes
    (weight format W_INT8_AND_PACKED4); pass N to the calls that take it through `n_out`."""
    N, K2 = wq.shape
    both = torch.empty((N * 3 * K2,), dtype=torch.int8, device=wq.device)
    _check(lib().stamp_prepare_weights_both(ctypes.byref(cfg), _ptr(wq), N, 2 * K2, _ptr(both), _stream()),
           "stamp_prepare_weights_both")
    return both


def n_hi_rows(cfg: StampConfig, B: int, L: int) -> int:
    n = cfg.block if cfg.block else L
    return B * (L // n) * cfg.k_hi


def stamp_quantize(cfg: StampConfig, X: torch.Tensor, ws: torch.Tensor):
    B, L, K = X.shape
    nh = n_hi_rows(cfg, B, L)
    q_hi = torch.empty((max(nh, 1), K), dtype=torch.int8, device=X.device)
    q_lo = torch.empty((max(B * L - nh, 1), K // 2), dtype=torch.uint8, device=X.device)
    # zero-point codes: the scales, then the zero points of the stored codes as int32 words (split_zero_points)
    x_scale = torch.empty((2, B, L) if cfg.act_zero_point else (B, L, K // cfg.group) if cfg.group else (B, L),
                          dtype=torch.float32, device=X.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_quantize(ctypes.byref(cfg), _ptr(X), _dtype_code(X), B, L, K, _ptr(q_hi), _ptr(q_lo),
                                _ptr(x_scale), wp, wb, _stream()), "stamp_quantize")
    return q_hi, q_lo, x_scale


def split_zero_points(x_scale: torch.Tensor):
    """The two halves of stamp_quantize's scale buffer in zero-point mode: scales [B, L] float32 and the zero
    points of the stored codes [B, L] int32."""
    return x_scale[0], x_scale[1].view(torch.int32)


def stamp_linear(cfg: StampConfig, q_hi, q_lo, x_scale, w, w_format: int, w_scale, B: int, L: int, K: int, N: int,
                 ws: torch.Tensor) -> torch.Tensor:
    Yt = torch.empty((B, L, N), dtype=torch.float32, device=x_scale.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_linear(ctypes.byref(cfg), _ptr(q_hi), _ptr(q_lo), _ptr(x_scale), _ptr(w), int(w_format),
                              _ptr(w_scale), B, L, K, N, _ptr(Yt), wp, wb, _stream()), "stamp_linear")
    return Yt


def stamp_dequantize(cfg: StampConfig, q_hi, q_lo, x_scale, B: int, L: int, K: int) -> torch.Tensor:
    """Stored codes back to transformed values, s (x_int - z): the read side of a STaMP-quantized cache."""
    T = torch.empty((B, L, K), dtype=torch.float32, device=x_scale.device)
    _check(lib().stamp_dequantize(ctypes.byref(cfg), _ptr(q_hi), _ptr(q_lo), _ptr(x_scale), B, L, K, _ptr(T), _stream()),
           "stamp_dequantize")
    return T


def stamp_inverse(cfg: StampConfig, Yt: torch.Tensor, bias: Optional[torch.Tensor], ws: torch.Tensor,
                  out_dtype=torch.float32, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    B, L, N = Yt.shape
    Y = out if out is not None else torch.empty((B, L, N), dtype=out_dtype, device=Yt.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_inverse(ctypes.byref(cfg), _ptr(Yt), _ptr(bias), B, L, N, _ptr(Y), _dtype_code(Y), wp, wb,
                               _stream()), "stamp_inverse")
    return Y


def stamp_inverse_noalloc(cfg: StampConfig, Yt: torch.Tensor, bias: Optional[torch.Tensor],
                          out_dtype=torch.float32, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """stamp_inverse without a workspace argument, for callers that may not allocate device memory:
    the scratch between the passes is an array built into the library (a few MB per GPU), so sizes
    beyond it raise StampError (status 6).  Calls on one device share that array: keep them ordered."""
    B, L, N = Yt.shape
    Y = out if out is not None else torch.empty((B, L, N), dtype=out_dtype, device=Yt.device)
    _check(lib().stamp_inverse_noalloc(ctypes.byref(cfg), _ptr(Yt), _ptr(bias), B, L, N, _ptr(Y), _dtype_code(Y),
                                       _stream()), "stamp_inverse_noalloc")
    return Y


def stamp_linear_fused(cfg: StampConfig, X: torch.Tensor, w: torch.Tensor, w_format: int, w_scale: torch.Tensor,
                       bias: Optional[torch.Tensor], ws: torch.Tensor, out_dtype=torch.float32,
                       out: Optional[torch.Tensor] = None, n_out: Optional[int] = None) -> torch.Tensor:
    B, L, K = X.shape
    N = n_out if n_out is not None else w.shape[0]
    Y = out if out is not None else torch.empty((B, L, N), dtype=out_dtype, device=X.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_linear_fused(ctypes.byref(cfg), _ptr(X), _dtype_code(X), _ptr(w), int(w_format),
                                    _ptr(w_scale), _ptr(bias), B, L, K, N, _ptr(Y), _dtype_code(Y), wp, wb,
                                    _stream()), "stamp_linear_fused")
    return Y


def stamp_workspace_bytes_host(cfg: StampConfig, B: int, L: int, K: int, N: int, x_dtype: int, y_dtype: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stamp_workspace_bytes_host(ctypes.byref(cfg), B, L, K, N, x_dtype, y_dtype, ctypes.byref(out)),
           "stamp_workspace_bytes_host")
    return int(out.value)


def stamp_linear_fused_host(cfg: StampConfig, X_host: torch.Tensor, w: torch.Tensor, w_format: int,
                            w_scale: torch.Tensor, bias: Optional[torch.Tensor], Y_host: torch.Tensor,
                            ws: torch.Tensor, n_out: Optional[int] = None) -> torch.Tensor:
    """X_host / Y_host are CPU tensors (pinned for asynchronous copies); everything else is on the device."""
    B, L, K = X_host.shape
    N = n_out if n_out is not None else w.shape[0]
    if X_host.is_cuda or Y_host.is_cuda or not X_host.is_contiguous() or not Y_host.is_contiguous():
        raise ValueError("expected contiguous host tensors")
    wp, wb = _ws_args(ws)
    _check(lib().stamp_linear_fused_host(ctypes.byref(cfg), ctypes.c_void_p(X_host.data_ptr()), _dtype_code(X_host),
                                         _ptr(w), int(w_format), _ptr(w_scale), _ptr(bias), B, L, K, N,
                                         ctypes.c_void_p(Y_host.data_ptr()), _dtype_code(Y_host), wp, wb, _stream()),
           "stamp_linear_fused_host")
    return Y_host


def stamp_profile_gemm_events(start: Optional["torch.cuda.Event"], stop: Optional["torch.cuda.Event"]) -> None:
    """Bracket every GEMM launch of this thread with the two (already created) CUDA events."""
    s = ctypes.c_void_p(start.cuda_event) if start is not None else None
    e = ctypes.c_void_p(stop.cuda_event) if stop is not None else None
    _check(lib().stamp_profile_gemm_events(s, e), "stamp_profile_gemm_events")


def stamp_debug_transform(cfg: StampConfig, X: torch.Tensor, ws: torch.Tensor) -> torch.Tensor:
    B, L, K = X.shape
    T = torch.empty((B, L, K), dtype=torch.float32, device=X.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_debug_transform(ctypes.byref(cfg), _ptr(X), _dtype_code(X), B, L, K, _ptr(T), wp, wb,
                                       _stream()), "stamp_debug_transform")
    return T


def stamp_debug_unpack_codes(cfg: StampConfig, q_hi, q_lo, B: int, L: int, K: int) -> torch.Tensor:
    codes = torch.empty((B, L, K), dtype=torch.int8, device=q_lo.device)
    _check(lib().stamp_debug_unpack_codes(ctypes.byref(cfg), _ptr(q_hi), _ptr(q_lo), B, L, K, _ptr(codes), _stream()),
           "stamp_debug_unpack_codes")
    return codes


def stamp_debug_gemm_i32(cfg: StampConfig, q_hi, q_lo, w, w_format: int, B: int, L: int, K: int, N: int,
                         ws: torch.Tensor) -> torch.Tensor:
    acc = torch.empty((B * L, N), dtype=torch.int32, device=w.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_debug_gemm_i32(ctypes.byref(cfg), _ptr(q_hi), _ptr(q_lo), _ptr(w), int(w_format), B, L, K, N,
                                      _ptr(acc), wp, wb, _stream()), "stamp_debug_gemm_i32")
    return acc


def stamp_debug_fused_operand(cfg: StampConfig, X: torch.Tensor, N: int, ws: torch.Tensor):
    """Codes, per-row factors, levels and zero points of the one-call layer's GEMM operand, in logical order."""
    B, L, K = X.shape
    codes = torch.empty((B, L, K), dtype=torch.int8, device=X.device)
    factor = torch.empty((B, L), dtype=torch.float32, device=X.device)
    level = torch.empty((B, L), dtype=torch.int32, device=X.device)
    zero = torch.empty((B, L), dtype=torch.int32, device=X.device)
    wp, wb = _ws_args(ws)
    _check(lib().stamp_debug_fused_operand(ctypes.byref(cfg), _ptr(X), _dtype_code(X), B, L, K, N, _ptr(codes),
                                           _ptr(factor), _ptr(level), _ptr(zero), wp, wb, _stream()),
           "stamp_debug_fused_operand")
    return codes, factor, level, zero


def stamp_last_device_status() -> int:
    st = ctypes.c_int(0)
    _check(lib().stamp_last_device_status(_stream(), ctypes.byref(st)), "stamp_last_device_status")
    return int(st.value)


def stamp_measure_i8_mma_issue(nbatch: int) -> int:
    """Enqueue the issue-only int8 tensor-core loop on the current stream; returns the integer operations it performs."""
    ops = ctypes.c_longlong(0)
    _check(lib().stamp_measure_i8_mma_issue(int(nbatch), ctypes.byref(ops), _stream()), "stamp_measure_i8_mma_issue")
    return int(ops.value)


def stamp_debug_expire_wait(limit_cycles: int) -> None:
    """Launch the test kernel whose bounded wait runs out after limit_cycles SM clocks (device status: time-out)."""
    _check(lib().stamp_debug_expire_wait(ctypes.c_longlong(int(limit_cycles)), _stream()), "stamp_debug_expire_wait")


def stamp_last_launch_count() -> int:
    return int(lib().stamp_last_launch_count())
