"""ctypes wrapper of the CPU oracle (oracle/stamp_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg.  The CUDA product path never imports this module.  The wrapper does
argument marshalling and nothing else; all of the method's arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stamp_oracle.c")
_LIB = os.path.join(_HERE, "libstamp_oracle.so")
_lib = None

T_IDENTITY, T_HAAR, T_DCT2, T_HAAR2D, T_WHT, T_HAAR_SKIP1 = 0, 1, 2, 3, 4, 5


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def transform_matrix(transform: int, n: int, levels: int = 0, grid_w: int = 0) -> np.ndarray:
    """Dense n x n fp64 matrix of the sequence transform (grid_w: patch-grid width of the 2-D Haar)."""
    out = np.empty((n, n), dtype=np.float64)
    if transform == T_HAAR2D:
        _check(lib().oracle_transform_matrix2d(int(n), int(grid_w), int(levels), _p(out)), "transform_matrix2d")
        return out
    _check(lib().oracle_transform_matrix(int(transform), int(n), int(levels), _p(out)), "transform_matrix")
    return out


def haar_matrix_csr(n: int, levels: int = 0):
    lv = levels if levels else int(np.log2(n))
    row_ptr = np.empty(n + 1, dtype=np.int64)
    col = np.empty(n * (lv + 1), dtype=np.int32)
    val = np.empty(n * (lv + 1), dtype=np.float64)
    _check(lib().oracle_haar_matrix_csr(int(n), int(levels), _p(row_ptr), _p(col), _p(val)), "haar_matrix_csr")
    return row_ptr, col, val


def apply_dense(Lmat: np.ndarray, X: np.ndarray, transpose: bool = False) -> np.ndarray:
    """blockdiag(Lmat) (or its transpose) applied along axis 1 of X [B, L, K] (fp64)."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    B, L, K = X.shape
    n = Lmat.shape[0]
    Lmat = np.ascontiguousarray(Lmat, dtype=np.float64)
    out = np.empty_like(X)
    _check(lib().oracle_apply_dense_f64(_p(Lmat), n, int(transpose), _p(X), B, L, K, _p(out)), "apply_dense")
    return out


def apply_csr(csr, n: int, X: np.ndarray) -> np.ndarray:
    row_ptr, col, val = csr
    X = np.ascontiguousarray(X, dtype=np.float32)
    B, L, K = X.shape
    out = np.empty((B, L, K), dtype=np.float64)
    _check(lib().oracle_apply_csr_f32in(_p(row_ptr), _p(col), _p(val), n, _p(X), B, L, K, _p(out)), "apply_csr")
    return out


def apply_csr_transpose(csr, n: int, Yt: np.ndarray) -> np.ndarray:
    row_ptr, col, val = csr
    Yt = np.ascontiguousarray(Yt, dtype=np.float64)
    B, L, K = Yt.shape
    out = np.empty((B, L, K), dtype=np.float64)
    _check(lib().oracle_apply_csr_transpose_f64(_p(row_ptr), _p(col), _p(val), n, _p(Yt), B, L, K, _p(out)),
           "apply_csr_transpose")
    return out


def bit_map(L: int, n: int, k_hi: int, bits_hi: int = 8, bits_lo: int = 4) -> np.ndarray:
    bits = np.empty(L, dtype=np.int32)
    _check(lib().oracle_bit_map(L, n, k_hi, bits_hi, bits_lo, _p(bits)), "bit_map")
    return bits


def set_rounding_decision(fp64: bool) -> bool:
    """Precision in which the symmetric quantizer takes its rounding decision: the fp32 quotient
    (default) or the fp64 quotient.  Returns the previous setting."""
    return bool(lib().oracle_set_rounding_decision(int(bool(fp64))))


def quantize_rows(T: np.ndarray, bits_per_row: np.ndarray):
    """Per-row symmetric RTN quantizer.  T [rows, K] fp64; row r uses bits_per_row[r % len]."""
    T = np.ascontiguousarray(T, dtype=np.float64)
    rows, K = T.shape
    bits_per_row = np.ascontiguousarray(bits_per_row, dtype=np.int32)
    scale = np.empty(rows, dtype=np.float32)
    codes = np.empty((rows, K), dtype=np.int8)
    _check(lib().oracle_quantize_rows(_p(T), ctypes.c_long(rows), K, _p(bits_per_row), len(bits_per_row),
                                      _p(scale), _p(codes)), "quantize_rows")
    return codes, scale


def quantize_rows_asym(T: np.ndarray, bits_per_row: np.ndarray):
    """Per-row zero-point RTN quantizer (Sec. 2.1, first equation, min-max range).  Returns unsigned
    codes [rows, K] uint8, scales [rows] float32 and integer zero points [rows] int32."""
    T = np.ascontiguousarray(T, dtype=np.float64)
    rows, K = T.shape
    bits_per_row = np.ascontiguousarray(bits_per_row, dtype=np.int32)
    scale = np.empty(rows, dtype=np.float32)
    zero = np.empty(rows, dtype=np.int32)
    codes = np.empty((rows, K), dtype=np.uint8)
    _check(lib().oracle_quantize_rows_asym(_p(T), ctypes.c_long(rows), K, _p(bits_per_row), len(bits_per_row),
                                           _p(scale), _p(zero), _p(codes)), "quantize_rows_asym")
    return codes, scale, zero


def gemm_zp_i32(q: np.ndarray, zero: np.ndarray, wq: np.ndarray) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    zero = np.ascontiguousarray(zero, dtype=np.int32)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = q.shape
    N = wq.shape[0]
    acc = np.empty((M, N), dtype=np.int32)
    _check(lib().oracle_gemm_zp_i32(_p(q), _p(zero), _p(wq), ctypes.c_long(M), N, K, _p(acc)), "gemm_zp_i32")
    return acc


def quantize_weights(W: np.ndarray, bits: int = 4):
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    scale = np.empty(N, dtype=np.float32)
    codes = np.empty((N, K), dtype=np.int8)
    _check(lib().oracle_quantize_rows_f32in(_p(W), ctypes.c_long(N), K, bits, _p(scale), _p(codes)),
           "quantize_weights")
    return codes, scale


def quantize_rows_grouped(T: np.ndarray, bits_per_row: np.ndarray, group: int):
    """Symmetric RTN quantizer with one scale per `group` consecutive features.  Returns codes [rows, K] int8 and
    scales [rows, K / group] float32."""
    T = np.ascontiguousarray(T, dtype=np.float64)
    rows, K = T.shape
    bits_per_row = np.ascontiguousarray(bits_per_row, dtype=np.int32)
    scale = np.empty((rows, K // group), dtype=np.float32)
    codes = np.empty((rows, K), dtype=np.int8)
    _check(lib().oracle_quantize_rows_grouped(_p(T), ctypes.c_long(rows), K, _p(bits_per_row), len(bits_per_row),
                                              int(group), _p(scale), _p(codes)), "quantize_rows_grouped")
    return codes, scale


def quantize_weights_grouped(W: np.ndarray, group: int, bits: int = 4):
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    scale = np.empty((N, K // group), dtype=np.float32)
    codes = np.empty((N, K), dtype=np.int8)
    _check(lib().oracle_quantize_rows_grouped_f32in(_p(W), ctypes.c_long(N), K, bits, int(group), _p(scale), _p(codes)),
           "quantize_weights_grouped")
    return codes, scale


def gemm_grouped(q: np.ndarray, sx: np.ndarray, wq: np.ndarray, sw: np.ndarray, group: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    sx = np.ascontiguousarray(sx, dtype=np.float32)
    sw = np.ascontiguousarray(sw, dtype=np.float32)
    M, K = q.shape
    N = wq.shape[0]
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().oracle_gemm_grouped(_p(q), _p(sx), _p(wq), _p(sw), ctypes.c_long(M), N, K, int(group), _p(out)),
           "gemm_grouped")
    return out


def gemm_i32(q: np.ndarray, wq: np.ndarray) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = q.shape
    N = wq.shape[0]
    acc = np.empty((M, N), dtype=np.int32)
    _check(lib().oracle_gemm_i32(_p(q), _p(wq), ctypes.c_long(M), N, K, _p(acc)), "gemm_i32")
    return acc


def dequant(acc: np.ndarray, sx: np.ndarray, sw: np.ndarray) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M, N = acc.shape
    sx = np.ascontiguousarray(sx, dtype=np.float32)
    sw = np.ascontiguousarray(sw, dtype=np.float32)
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().oracle_dequant(_p(acc), _p(sx), _p(sw), ctypes.c_long(M), N, _p(out)), "dequant")
    return out


def matmul_f64(X: np.ndarray, W: np.ndarray) -> np.ndarray:
    X = np.ascontiguousarray(X, dtype=np.float32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    M, K = X.shape
    N = W.shape[0]
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().oracle_matmul_f64(_p(X), _p(W), ctypes.c_long(M), N, K, _p(out)), "matmul_f64")
    return out


def stamp_linear(X: np.ndarray, W: np.ndarray, bias: Optional[np.ndarray] = None, *, transform: int,
                 block: int = 0, levels: int = 0, k_hi: int = 64, bits_hi: int = 8, bits_lo: int = 4,
                 bits_w: int = 4, grid_w: int = 0, asym: bool = False, group: int = 0,
                 want=("T", "x_scale", "q", "w_scale", "wq", "acc", "Yt", "Y")) -> Dict[str, np.ndarray]:
    """Run the whole layer; returns the stages named in `want`.

    asym=True selects the zero-point activation quantizer: "q" is then uint8 and "x_zero" (int32 per
    transformed token) is returned as well.

    group > 0 selects per-block scales of `group` features for activations and weights: "x_scale" is then
    [B*L, K/group], "w_scale" [N, K/group], and "acc" is not available.

    X [B, L, K] float32 (values already rounded to the storage dtype), W [N, K] float32."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    B, L, K = X.shape
    N = W.shape[0]
    M = B * L
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
    if asym and "x_scale" in want:
        want = tuple(want) + ("x_zero",)
    ng = K // group if group else 1
    if group:
        want = tuple(w for w in want if w != "acc")
    shapes = {"T": ((M, K), np.float64), "x_scale": ((M, ng) if group else (M,), np.float32),
              "q": ((M, K), np.uint8 if asym else np.int8), "x_zero": ((M,), np.int32),
              "w_scale": ((N, ng) if group else (N,), np.float32), "wq": ((N, K), np.int8), "acc": ((M, N), np.int32),
              "Yt": ((M, N), np.float64), "Y": ((M, N), np.float64)}
    out = {k: np.empty(s, dtype=d) for k, (s, d) in shapes.items() if k in want}
    g = out.get
    rc = lib().oracle_stamp_linear(_p(X), _p(W), _p(bias), B, L, K, N, int(transform), int(block), int(levels),
                                   int(k_hi), int(bits_hi), int(bits_lo), int(bits_w), _p(g("T")),
                                   _p(g("x_scale")), _p(g("q")), _p(g("w_scale")), _p(g("wq")), _p(g("acc")),
                                   _p(g("Yt")), _p(g("Y")), int(grid_w), int(bool(asym)), _p(g("x_zero")), int(group))
    _check(rc, "stamp_linear")
    return out
