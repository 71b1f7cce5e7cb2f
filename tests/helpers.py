"""Test-side marshalling helpers (format conversion and error norms only)."""
import numpy as np


def to_device(x: np.ndarray, dtype_code: int):
    """float32 numpy (values exactly representable in the target dtype) -> CUDA tensor."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype_code == 1 else t


def pack_nibbles(q: np.ndarray) -> np.ndarray:
    """int8 codes in [-8, 7], shape [..., K] -> uint8 [..., K/2], low nibble = even k."""
    u = (q.astype(np.int16) & 0xF).astype(np.uint8)
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def pack_codes(q: np.ndarray, n: int, k_hi: int):
    """Logical codes [M, K] -> the public (q_hi [n_hi, K] int8, q_lo [M - n_hi, K/2] uint8) pair."""
    M, K = q.shape
    idx = np.arange(M) % n
    hi = idx < k_hi
    q_hi = np.ascontiguousarray(q[hi])
    q_lo = pack_nibbles(np.ascontiguousarray(q[~hi]))
    if q_hi.shape[0] == 0:
        q_hi = np.zeros((1, K), np.int8)
    if q_lo.shape[0] == 0:
        q_lo = np.zeros((1, K // 2), np.uint8)
    return q_hi, q_lo


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300))


def code_mismatch(q_gpu: np.ndarray, q_ref: np.ndarray):
    """(#codes that differ, max |difference|)."""
    d = q_gpu.astype(np.int16) - q_ref.astype(np.int16)
    nz = np.count_nonzero(d)
    return nz, (int(np.abs(d).max()) if nz else 0)
