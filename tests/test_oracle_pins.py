"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix,
never against itself.  Every test names the passage it pins.  CPU only."""
import importlib.util
import math
import os
import subprocess
import tempfile
from fractions import Fraction

import numpy as np
import pytest
import scipy.fft

from paper_2510_26771_b200 import inputs as gen

T_ID, T_HAAR, T_DCT = 0, 1, 2


# --------------------------------------------------------------------------------------
# Transform matrices (Theorem 1 premise: L orthogonal; Sec. "Efficient Energy Concentration")
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("transform,n,levels", [
    (T_HAAR, 2, 0), (T_HAAR, 8, 0), (T_HAAR, 8, 1), (T_HAAR, 64, 3), (T_HAAR, 256, 0), (T_HAAR, 1024, 6),
    (T_DCT, 2, 0), (T_DCT, 8, 0), (T_DCT, 256, 0), (T_DCT, 96, 0),
])
def test_orthonormal(oracle, transform, n, levels):
    Lm = oracle.transform_matrix(transform, n, levels)
    assert np.max(np.abs(Lm @ Lm.T - np.eye(n))) <= 1e-12
    assert np.max(np.abs(Lm.T @ Lm - np.eye(n))) <= 1e-12


def test_haar_n2_hand_case(oracle):
    r = 1.0 / math.sqrt(2.0)
    Lm = oracle.transform_matrix(T_HAAR, 2, 0)
    assert np.allclose(Lm, [[r, r], [r, -r]], rtol=0, atol=1e-15)


def _haar_closed_form(n, levels):
    """Rows written from the closed form: a_l[i] = 2^(-l/2) on [i 2^l, (i+1) 2^l);
    d_j[i] = 2^(-j/2) (+ on the first half, - on the second half of [i 2^j, (i+1) 2^j));
    row order [a_l | d_l | d_(l-1) | ... | d_1]."""
    M = np.zeros((n, n))
    na = n >> levels
    for i in range(na):
        M[i, i << levels:(i + 1) << levels] = 2.0 ** (-levels / 2)
    for j in range(levels, 0, -1):
        base = n >> j
        for i in range(n >> j):
            lo, mid, hi = i << j, (i << j) + (1 << (j - 1)), (i + 1) << j
            M[base + i, lo:mid] = 2.0 ** (-j / 2)
            M[base + i, mid:hi] = -(2.0 ** (-j / 2))
    return M


@pytest.mark.parametrize("n,levels", [(4, 1), (4, 2), (16, 3), (64, 3), (64, 6), (512, 9), (2048, 11)])
def test_haar_closed_form_rows(oracle, n, levels):
    Lm = oracle.transform_matrix(T_HAAR, n, levels)
    assert np.max(np.abs(Lm - _haar_closed_form(n, levels))) <= 1e-14


def test_haar_full_depth_is_levels_zero(oracle):
    assert np.array_equal(oracle.transform_matrix(T_HAAR, 64, 0), oracle.transform_matrix(T_HAAR, 64, 6))


def test_haar_each_level_halves_the_lowpass_band(oracle):
    """Each DWT step concentrates a constant (fully correlated) signal into the first half:
    constant input c => every detail row is 0 and the l-level approximation is c 2^(l/2)."""
    n, K = 64, 3
    X = np.full((1, n, K), 1.75)
    for levels in (1, 2, 3, 6):
        T = oracle.apply_dense(oracle.transform_matrix(T_HAAR, n, levels), X)[0]
        na = n >> levels
        assert np.allclose(T[:na], 1.75 * 2 ** (levels / 2), rtol=1e-14)
        assert np.max(np.abs(T[na:])) <= 1e-14


def test_impulse_gives_matrix_column(oracle):
    n = 32
    for transform, levels in ((T_HAAR, 0), (T_HAAR, 2), (T_DCT, 0)):
        Lm = oracle.transform_matrix(transform, n, levels)
        for t in (0, 5, 31):
            X = np.zeros((1, n, 1))
            X[0, t, 0] = 1.0
            assert np.array_equal(oracle.apply_dense(Lm, X)[0, :, 0], Lm[:, t])


@pytest.mark.parametrize("n", [2, 16, 256])
def test_dct_matches_scipy_ortho_dct2(oracle, n):
    """Special case that reduces to a library routine: the DCT matrix applied to data equals
    SciPy's orthonormal DCT-II along the token axis."""
    rng = np.random.default_rng(11)
    X = rng.standard_normal((1, n, 5))
    T = oracle.apply_dense(oracle.transform_matrix(T_DCT, n), X)
    ref = scipy.fft.dct(X, type=2, norm="ortho", axis=1)
    assert np.max(np.abs(T - ref)) <= 1e-12 * np.max(np.abs(ref))
    # row 0 is the DC row: low frequencies come first
    assert np.allclose(oracle.transform_matrix(T_DCT, n)[0], 1 / math.sqrt(n))


def test_block_diagonal_application(oracle):
    """A blockwise transform acts on each block of n tokens and each batch item separately."""
    rng = np.random.default_rng(5)
    n, B, L, K = 8, 2, 32, 3
    X = rng.standard_normal((B, L, K))
    Lm = oracle.transform_matrix(T_DCT, n)
    T = oracle.apply_dense(Lm, X)
    for b in range(B):
        for blk in range(L // n):
            assert np.allclose(T[b, blk * n:(blk + 1) * n], Lm @ X[b, blk * n:(blk + 1) * n], atol=1e-13)


@pytest.mark.parametrize("transform,n,levels", [(T_HAAR, 128, 0), (T_HAAR, 128, 3), (T_DCT, 64, 0)])
def test_energy_and_reconstruction(oracle, transform, n, levels):
    """Sequence transforms do not alter the total energy (remark after Theorem 1) and
    L^T (L X) = X."""
    rng = np.random.default_rng(3)
    X = rng.standard_normal((2, 2 * n, 7)) * np.array([1, 10, 0.1, 3, 1, 1, 50])
    Lm = oracle.transform_matrix(transform, n, levels)
    T = oracle.apply_dense(Lm, X)
    assert abs(np.sum(T * T) - np.sum(X * X)) <= 1e-12 * np.sum(X * X)
    back = oracle.apply_dense(Lm, T, transpose=True)
    assert np.max(np.abs(back - X)) <= 1e-12 * np.max(np.abs(X))


def test_csr_equals_dense(oracle):
    rng = np.random.default_rng(8)
    for n, levels in ((64, 0), (256, 5), (1024, 0)):
        X = rng.standard_normal((1, 2 * n, 4)).astype(np.float32)
        Lm = oracle.transform_matrix(T_HAAR, n, levels)
        csr = oracle.haar_matrix_csr(n, levels)
        T_d = oracle.apply_dense(Lm, X.astype(np.float64))
        T_s = oracle.apply_csr(csr, n, X)
        assert np.max(np.abs(T_d - T_s)) <= 1e-13 * np.max(np.abs(T_d))
        Y_d = oracle.apply_dense(Lm, T_d, transpose=True)
        Y_s = oracle.apply_csr_transpose(csr, n, T_d)
        assert np.max(np.abs(Y_d - Y_s)) <= 1e-13 * np.max(np.abs(Y_d))
        # CSR holds exactly the non-zeros of the dense matrix
        rp, col, val = csr
        D = np.zeros((n, n))
        for i in range(n):
            D[i, col[rp[i]:rp[i + 1]]] = val[rp[i]:rp[i + 1]]
        assert np.array_equal(D, Lm)


def test_bias_projection_closed_form(oracle):
    """l = L 1 (Method, second equation): Haar l-level => 2^(l/2) on the first n/2^l rows,
    0 elsewhere; DCT => (sqrt n, 0, ..., 0); and L^T (Y_t + l b^T) = L^T Y_t + 1 b^T."""
    n = 64
    ones = np.ones((1, n, 1))
    for levels in (1, 3, 6):
        l = oracle.apply_dense(oracle.transform_matrix(T_HAAR, n, levels), ones)[0, :, 0]
        na = n >> levels
        assert np.allclose(l[:na], 2 ** (levels / 2), rtol=1e-14)
        assert np.max(np.abs(l[na:])) <= 1e-14
    l = oracle.apply_dense(oracle.transform_matrix(T_DCT, n), ones)[0, :, 0]
    assert abs(l[0] - math.sqrt(n)) <= 1e-13 and np.max(np.abs(l[1:])) <= 1e-13
    rng = np.random.default_rng(1)
    Yt = rng.standard_normal((1, n, 5))
    beta = rng.standard_normal(5)
    Lm = oracle.transform_matrix(T_HAAR, n, 3)
    lvec = (Lm @ np.ones(n))[:, None]
    lhs = oracle.apply_dense(Lm, Yt + lvec * beta[None, :], transpose=True)
    rhs = oracle.apply_dense(Lm, Yt, transpose=True) + beta
    assert np.max(np.abs(lhs - rhs)) <= 1e-12


# --------------------------------------------------------------------------------------
# Quantizer (Sec. 2.1, first equation and the range bound that follows it)
# --------------------------------------------------------------------------------------

def test_quantizer_properties(oracle):
    rng = np.random.default_rng(2)
    rows, K = 40, 96
    T = rng.standard_normal((rows, K)) * rng.lognormal(0, 2, size=(rows, 1))
    bits = np.where(np.arange(rows) < 8, 8, 4).astype(np.int32)
    q, s = oracle.quantize_rows(T, bits)
    qmax = (2 ** (bits - 1) - 1)[:, None]
    assert q.dtype == np.int8 and s.dtype == np.float32
    assert np.all(np.abs(q.astype(int)) <= qmax)                  # restricted symmetric range
    am = np.argmax(np.abs(T), axis=1)
    assert np.all(np.abs(q[np.arange(rows), am].astype(int)) == qmax[:, 0])   # absmax -> +-qmax
    assert np.allclose(s, (np.max(np.abs(T), axis=1).astype(np.float32) / qmax[:, 0].astype(np.float32)))
    sd = s.astype(np.float64)[:, None]
    err = T - sd * q
    assert np.all(np.abs(err) <= sd / 2 * (1 + 1e-6))             # no clipping: rounding error only
    # per-token bound: ||Q(t) - t||^2 <= K s^2 / 4 <= K ||t||^2 / (4 qmax^2)
    e2 = np.sum(err * err, axis=1)
    assert np.all(e2 <= K * sd[:, 0] ** 2 / 4 * (1 + 1e-6))
    assert np.all(e2 <= K * np.sum(T * T, axis=1) / (4 * qmax[:, 0] ** 2) * (1 + 1e-6))
    # re-quantizing the de-quantized row is idempotent
    q2, s2 = oracle.quantize_rows(sd * q, bits)
    assert np.array_equal(q2, q)
    assert np.allclose(s2, s, rtol=1e-6)


def test_quantizer_round_half_to_even_and_zero_row(oracle):
    # scale = 7/7 = 1 exactly, so the values are their own pre-rounding codes
    T = np.array([[7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.49, -3.51],
                  [0, 0, 0, 0, 0, 0, 0, 0, 0]])
    q, s = oracle.quantize_rows(T, np.array([4, 4], dtype=np.int32))
    assert s[0] == 1.0 and s[1] == 1.0                                # zero row: scale 1, codes 0
    assert q[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 3, -4]
    assert not q[1].any()
    # 8-bit row
    T = np.array([[127.0, -126.5, 0.49999, 63.5]])
    q, s = oracle.quantize_rows(T, np.array([8], dtype=np.int32))
    assert s[0] == 1.0 and q[0].tolist() == [127, -126, 0, 64]


def test_bit_map_reproduces_printed_effective_bits(oracle):
    """Golden values printed in the paper (tests/golden/effective_bits.txt)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "effective_bits.txt")
    rows = [ln.split("#")[0].split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for k, L, bh, bl, eff in rows:
        bits = oracle.bit_map(int(L), int(L), int(k), int(bh), int(bl))
        assert bits.mean() == float(eff)
        assert np.all(bits[:int(k)] == int(bh)) and np.all(bits[int(k):] == int(bl))
    # blockwise: the first k_hi rows OF EACH BLOCK are the 8-bit ones
    bits = oracle.bit_map(1024, 256, 16)
    assert bits.mean() == 4.25
    assert set(np.nonzero(bits == 8)[0] % 256) == set(range(16))


def test_error_invariance_under_orthogonal_transform(oracle):
    """First step of the proof of Theorem 1: ||L^T Q(LX) - X||_F = ||Q(LX) - LX||_F."""
    cfg = gen.scaled(gen.config_tiny(), L=128, K=64)
    X = gen.make_activation(cfg).astype(np.float64)
    for transform, levels in ((T_HAAR, 0), (T_HAAR, 3), (T_DCT, 0)):
        Lm = oracle.transform_matrix(transform, cfg.L, levels)
        T = oracle.apply_dense(Lm, X)
        q, s = oracle.quantize_rows(T[0], oracle.bit_map(cfg.L, cfg.L, 8))
        Tq = (q * s.astype(np.float64)[:, None])[None]
        lhs = np.linalg.norm(oracle.apply_dense(Lm, Tq, transpose=True) - X)
        rhs = np.linalg.norm(Tq - T)
        assert abs(lhs - rhs) <= 1e-12 * rhs


# --------------------------------------------------------------------------------------
# Integer GEMM and the whole layer
# --------------------------------------------------------------------------------------

def test_gemm_brute_force(oracle):
    rng = np.random.default_rng(4)
    M, N, K = 37, 19, 256
    q = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    wq = rng.integers(-7, 8, size=(N, K), dtype=np.int8)
    acc = oracle.gemm_i32(q, wq)
    ref = q.astype(np.int64) @ wq.astype(np.int64).T
    assert acc.shape == (M, N) and np.array_equal(acc.astype(np.int64), ref)
    assert np.max(np.abs(acc)) <= 127 * 7 * K
    # extreme codes reach the bound exactly
    acc = oracle.gemm_i32(np.full((2, K), 127, np.int8), np.full((3, K), -7, np.int8))
    assert np.all(acc == -127 * 7 * K)


def test_unquantized_pipeline_is_plain_matmul(oracle):
    """(L^-1 (L X)) W^T = L^-1 ((L X) W^T) = X W^T  (Method, second equation)."""
    rng = np.random.default_rng(6)
    B, L, K, N = 2, 64, 48, 24
    X = rng.standard_normal((B, L, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    ref = oracle.matmul_f64(X.reshape(-1, K), W).reshape(B, L, N)
    assert np.max(np.abs(ref - X.astype(np.float64) @ W.astype(np.float64).T)) <= 1e-12
    for transform, n, levels in ((T_HAAR, 64, 0), (T_HAAR, 32, 2), (T_DCT, 16, 0)):
        Lm = oracle.transform_matrix(transform, n, levels)
        T = oracle.apply_dense(Lm, X.astype(np.float64))
        Yt = (T.reshape(-1, K) @ W.astype(np.float64).T).reshape(B, L, N)
        Y = oracle.apply_dense(Lm, Yt, transpose=True)
        assert np.max(np.abs(Y - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_layer_exact_when_codes_are_exact(oracle):
    """Inputs built so that every transformed row is an integer multiple of a power-of-two
    scale with the extreme code present: quantization is then lossless and the STaMP layer
    must return the textbook X W^T (+ bias)."""
    rng = np.random.default_rng(9)
    nblk, K, N = 6, 32, 10
    # block of 4 tokens [u, u, v, v] with 2-level Haar: a_2 = u + v, d_2 = u - v, d_1 = 0
    P = rng.integers(-127, 128, size=(nblk, K)); P[:, 0] = 127      # 8-bit row (k_hi = 1)
    Q = rng.integers(-7, 8, size=(nblk, K)); Q[:, 1] = -7           # 4-bit row
    u, v = (P + Q) / 2.0, (P - Q) / 2.0
    X = np.stack([u, u, v, v], axis=1).reshape(1, 4 * nblk, K).astype(np.float32)
    Wi = rng.integers(-7, 8, size=(N, K)); Wi[:, 2] = 7
    W = (Wi * 2.0 ** -3).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    out = oracle.stamp_linear(X, W, bias, transform=T_HAAR, block=4, levels=2, k_hi=1)
    q = out["q"].reshape(nblk, 4, K)
    assert np.array_equal(q[:, 0], P) and np.array_equal(q[:, 1], Q) and not q[:, 2:].any()
    assert np.array_equal(out["wq"], Wi)
    assert np.all(out["x_scale"].reshape(nblk, 4) == 1.0) and np.all(out["w_scale"] == 2.0 ** -3)
    ref = X[0].astype(np.float64) @ W.astype(np.float64).T + bias.astype(np.float64)
    assert np.max(np.abs(out["Y"] - ref)) <= 1e-12 * np.max(np.abs(ref))


def _python_loop_layer(X, W, bias, n, levels, k_hi):
    """The Algorithm written out with Python floats and loops (tiny sizes only)."""
    L, K = len(X), len(X[0])
    N = len(W)
    r = 1.0 / math.sqrt(2.0)
    T = [[0.0] * K for _ in range(L)]
    for b0 in range(0, L, n):
        for j in range(K):
            v = [X[b0 + t][j] for t in range(n)]
            length = n
            for _ in range(levels):
                a = [(v[2 * i] + v[2 * i + 1]) * r for i in range(length // 2)]
                d = [(v[2 * i] - v[2 * i + 1]) * r for i in range(length // 2)]
                v[:length] = a + d
                length //= 2
            for t in range(n):
                T[b0 + t][j] = v[t]

    def quant(row, qmax):
        """Nearest of the 2 qmax + 1 levels s * k by brute force in exact rational arithmetic; a value closer
        than 2^-20 (relative) to the midpoint of two levels is a tie at fp32 resolution and is reported in
        `ties` instead of being decided here."""
        amax = max(abs(x) for x in row)
        s = float(np.float32(amax) / np.float32(qmax)) if amax > 0 else 1.0
        sf = Fraction(s)
        codes = []
        for x in row:
            xf = Fraction(x)
            dist = sorted((abs(xf - sf * k), k) for k in range(-qmax, qmax + 1))
            (d0, k0), (d1, _) = dist[0], dist[1]
            if d1 - d0 <= sf * Fraction(1, 1 << 20) * max(1, abs(k0)):
                ties.append((x, s))
            codes.append(k0)
        return codes, s

    ties = []

    qs = [quant(T[i], 127 if (i % n) < k_hi else 7) for i in range(L)]
    ws = [quant(W[c], 7) for c in range(N)]
    Yt = [[sum(qs[i][0][k] * ws[c][0][k] for k in range(K)) * qs[i][1] * ws[c][1] for c in range(N)]
          for i in range(L)]
    Y = [[0.0] * N for _ in range(L)]
    for b0 in range(0, L, n):
        for c in range(N):
            v = [Yt[b0 + t][c] for t in range(n)]
            length = n >> levels
            for _ in range(levels):
                a, d = v[:length], v[length:2 * length]
                rec = []
                for i in range(length):
                    rec += [(a[i] + d[i]) * r, (a[i] - d[i]) * r]
                v[:2 * length] = rec
                length *= 2
            for t in range(n):
                Y[b0 + t][c] = v[t] + bias[c]
    return np.array(Y), np.array([x[0] for x in qs]), np.array([x[1] for x in qs]), ties


def test_layer_vs_python_loops(oracle):
    """Brute force on tiny inputs: an independent, loop-by-loop statement of the Algorithm
    (fast in-place Haar instead of the explicit matrix)."""
    rng = np.random.default_rng(12)
    L, K, N, n, levels, k_hi = 16, 6, 5, 8, 3, 2
    X = rng.standard_normal((L, K)).astype(np.float32)
    X[:, 1] *= 20
    W = (rng.standard_normal((N, K)) * 0.1).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    out = oracle.stamp_linear(X[None], W, bias, transform=T_HAAR, block=n, levels=levels, k_hi=k_hi)
    Y, q, s, ties = _python_loop_layer(X.astype(float).tolist(), W.astype(float).tolist(), bias.astype(float).tolist(),
                                       n, levels, k_hi)
    assert not ties          # no value of this input sits on a rounding boundary: the nearest level is unique
    assert np.array_equal(out["q"], q)
    assert np.allclose(out["x_scale"], s, rtol=1e-7)
    assert np.max(np.abs(out["Y"] - Y)) <= 1e-12 * np.max(np.abs(Y))


def test_layer_stages_compose(oracle):
    """The one-call layer equals its exported steps chained in the Algorithm's order."""
    cfg = gen.scaled(gen.config_tiny(), L=64, K=128, N=32)
    X, W = gen.make_activation(cfg), gen.make_weight(cfg)
    out = oracle.stamp_linear(X, W, None, transform=T_DCT, block=32, k_hi=4)
    Lm = oracle.transform_matrix(T_DCT, 32)
    T = oracle.apply_dense(Lm, X.astype(np.float64))
    assert np.array_equal(out["T"], T.reshape(-1, cfg.K))
    q, s = oracle.quantize_rows(T.reshape(-1, cfg.K), oracle.bit_map(cfg.L, 32, 4))
    wq, sw = oracle.quantize_weights(W)
    assert np.array_equal(out["q"], q) and np.array_equal(out["wq"], wq)
    acc = oracle.gemm_i32(q, wq)
    assert np.array_equal(out["acc"], acc)
    Yt = oracle.dequant(acc, s, sw)
    assert np.array_equal(out["Yt"], Yt)
    assert np.array_equal(out["Y"], oracle.apply_dense(Lm, Yt.reshape(1, cfg.L, -1), transpose=True).reshape(cfg.L, -1))


# --------------------------------------------------------------------------------------
# Qualitative claims on the synthetic stand-ins (sanity, not parity criteria)
# --------------------------------------------------------------------------------------

def _sqnr(ref, x):
    return 10 * math.log10(np.sum(ref * ref) / np.sum((ref - x) ** 2))


def test_energy_concentrates_and_stamp_beats_uniform_4bit(oracle):
    cfg = gen.scaled(gen.config_sweep(512, 2048), K=256, N=64)
    X, W = gen.make_activation(cfg), gen.make_weight(cfg)
    ref = oracle.matmul_f64(X[0], W)
    stamp = oracle.stamp_linear(X, W, None, transform=T_HAAR, k_hi=cfg.k_hi, want=("T", "Y"))
    e = np.sum(stamp["T"] ** 2, axis=1)
    L = cfg.L
    # AR(1) with rho = 0.9 decorrelates over ~10 tokens: every level up to 2^5 tokens gains energy
    # over the finer one, and the 8-bit rows (coarsest bands) carry far more energy per token
    band_mean = [e[L >> j:L >> (j - 1)].mean() for j in range(5, 0, -1)]
    assert all(a > b for a, b in zip(band_mean, band_mean[1:]))
    assert e[:cfg.k_hi].mean() > 10 * e[cfg.k_hi:].mean()
    uniform = oracle.stamp_linear(X, W, None, transform=T_ID, k_hi=0, want=("Y",))
    assert _sqnr(ref, stamp["Y"]) > _sqnr(ref, uniform["Y"])


# ---------------------------------------------------------------------------------------------
# 2-D Haar over the patch grid (Sec. "Efficient Energy Concentration"; LVM set-up: 3 levels on a
# 64 x 64 grid leave 64 low-pass tokens)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("h,w,levels", [(8, 8, 3), (16, 8, 2), (4, 16, 1), (64, 64, 3)])
def test_haar2d_orthonormal_and_lowpass_closed_form(oracle, h, w, levels):
    n = h * w
    Lm = oracle.transform_matrix(oracle.T_HAAR2D, n, levels, grid_w=w)
    assert np.abs(Lm @ Lm.T - np.eye(n)).max() <= 1e-12
    # LL_l[y, x] = 2^-l * (sum over the 2^l x 2^l patch): the first n / 4^l rows, raster order
    s = 1 << levels
    for y in range(h // s):
        for x in range(w // s):
            want = np.zeros((h, w))
            want[y * s:(y + 1) * s, x * s:(x + 1) * s] = 2.0 ** -levels
            assert np.array_equal(Lm[y * (w // s) + x], want.reshape(-1))
    # a constant image has no detail: only the low-pass rows respond, with c * 2^l
    t = Lm @ np.full(n, 3.0)
    q = n >> (2 * levels)
    assert np.allclose(t[:q], 3.0 * 2.0 ** levels, rtol=0, atol=1e-12) and np.abs(t[q:]).max() <= 1e-12


def test_haar2d_one_level_is_the_kronecker_product_of_1d_steps(oracle):
    """Independent construction: one 2-D level = (1-D Haar step across rows) (x) (1-D step along a row)."""
    h, w = 4, 8
    Hy = oracle.transform_matrix(oracle.T_HAAR, h, 1)     # rows: [averages | differences], pinned above
    Hx = oracle.transform_matrix(oracle.T_HAAR, w, 1)
    ay, dy, ax, dx = Hy[:h // 2], Hy[h // 2:], Hx[:w // 2], Hx[w // 2:]
    want = np.concatenate([np.kron(ay, ax),    # LL
                           np.kron(ay, dx),    # LH: difference along a row
                           np.kron(dy, ax),    # HL: difference across rows
                           np.kron(dy, dx)])   # HH
    got = oracle.transform_matrix(oracle.T_HAAR2D, h * w, 1, grid_w=w)
    assert np.abs(got - want).max() <= 1e-15


def test_haar2d_levels_nest_and_pipeline_is_plain_matmul(oracle):
    """Level l+1 only re-mixes the low-pass quarter; with the quantizers off the layer is X W^T."""
    h = w = 8
    n = h * w
    L1 = oracle.transform_matrix(oracle.T_HAAR2D, n, 1, grid_w=w)
    L2 = oracle.transform_matrix(oracle.T_HAAR2D, n, 2, grid_w=w)
    assert np.array_equal(L1[n // 4:], L2[n // 4:])                    # level-1 detail bands untouched
    inner = oracle.transform_matrix(oracle.T_HAAR2D, n // 4, 1, grid_w=w // 2)
    assert np.abs(L2[:n // 4] - inner @ L1[:n // 4]).max() <= 1e-15   # the LL grid transformed once more
    rng = np.random.default_rng(7)
    X = rng.standard_normal((2, n, 24))
    W = rng.standard_normal((10, 24))
    T = oracle.apply_dense(L2, X)
    back = oracle.apply_dense(L2, T @ W.T, transpose=True)
    assert np.abs(back - X @ W.T).max() <= 1e-12
    assert abs((T ** 2).sum() - (X ** 2).sum()) <= 1e-10 * (X ** 2).sum()


def test_haar2d_layer_runs_and_marks_the_lowpass_tokens_high_precision(oracle):
    cfg = gen.scaled(gen.config_dit_proj_2d(), B=1, L=256, K=128, N=64, grid=16, levels=2, k_hi=16)
    X, W = gen.make_activation(cfg), gen.make_weight(cfg)
    out = oracle.stamp_linear(X, W, None, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi,
                              grid_w=cfg.grid, want=("T", "q", "Y"))
    # the 16 low-pass tokens (a 4 x 4 grid of 4 x 4 patch sums) are the 8-bit rows and carry most energy
    assert np.abs(out["q"][:16]).max() > 7 and np.abs(out["q"][16:]).max() <= 7
    e = (out["T"] ** 2).sum(axis=1)
    assert e[:16].sum() > 0.9 * e.sum()
    ref = oracle.matmul_f64(X.reshape(-1, cfg.K), W)
    assert np.linalg.norm(out["Y"] - ref) / np.linalg.norm(ref) < 0.2


# ---------------------------------------------------------------------------------------------
# Walsh-Hadamard transform (Sec. "Efficient Energy Concentration": the DCT with only the signs kept)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n", [2, 8, 64, 256])
def test_wht_is_the_sequency_ordered_hadamard_matrix(oracle, n):
    import scipy.linalg
    Wm = oracle.transform_matrix(oracle.T_WHT, n)
    assert np.abs(Wm @ Wm.T - np.eye(n)).max() <= 1e-12
    assert np.array_equal(Wm, Wm.T)                                   # symmetric, hence its own inverse
    assert np.allclose(np.abs(Wm), 1.0 / math.sqrt(n), rtol=0, atol=1e-15)
    changes = (np.diff(np.sign(Wm), axis=1) != 0).sum(axis=1)
    assert np.array_equal(changes, np.arange(n))                      # row u changes sign u times
    # the same rows as the library's natural-order Hadamard matrix, reordered
    Hn = scipy.linalg.hadamard(n) / math.sqrt(n)
    assert {tuple(np.sign(r)) for r in Hn} == {tuple(np.sign(r)) for r in Wm}
    assert np.allclose(Wm[0], 1.0 / math.sqrt(n))                     # row 0 = DC, as for the DCT


def test_wht_rows_follow_the_sign_of_the_cosine_basis_at_low_sequency(oracle):
    """"Retaining only the sign": the first rows of the WHT are the signs of the first DCT rows."""
    n = 64
    Wm = oracle.transform_matrix(oracle.T_WHT, n)
    Cm = oracle.transform_matrix(oracle.T_DCT2, n)
    for u in (0, 1, 2, 4, 8, 16, 32):     # dyadic frequencies: square waves with the cosine's zero crossings
        assert np.array_equal(np.sign(Wm[u]), np.sign(Cm[u]))


def test_wht_layer_runs_blockwise(oracle):
    cfg = gen.scaled(gen.config_llm_down_wht(), B=1, L=512, K=128, N=64)
    X, W = gen.make_activation(cfg), gen.make_weight(cfg)
    out = oracle.stamp_linear(X, W, None, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi,
                              want=("T", "q", "Y"))
    Wm = oracle.transform_matrix(oracle.T_WHT, cfg.block)
    T_np = np.einsum("ut,btk->buk", Wm, X.astype(np.float64).reshape(-1, cfg.block, cfg.K)).reshape(-1, cfg.K)
    assert np.abs(out["T"] - T_np).max() <= 1e-12 * np.abs(T_np).max()
    assert abs((out["T"] ** 2).sum() - (X.astype(np.float64) ** 2).sum()) <= 1e-10 * (X.astype(np.float64) ** 2).sum()
    ref = oracle.matmul_f64(X.reshape(-1, cfg.K), W)
    assert np.linalg.norm(out["Y"] - ref) / np.linalg.norm(ref) < 0.2


# --------------------------------------------------------------------------------------
# Zero-point (asymmetric) activation quantizer: Sec. 2.1, first equation as printed, min-max range
# --------------------------------------------------------------------------------------

def test_asym_quantizer_hand_case_and_constant_rows(oracle):
    # 4 bits: range 3, s = 3/15 = 0.2, z = rne(1/0.2) = 5; x/s = -5, 0, 3, 10 (none near a tie)
    T = np.array([[-1.0, 0.0, 0.6, 2.0],
                  [0.0, 0.0, 0.0, 0.0],          # zero row: s = 1, z = 0, codes 0
                  [3.0, 3.0, 3.0, 3.0]])         # constant row: s = 1, z = -3, codes 0, de-quantizes to 3
    q, s, z = oracle.quantize_rows_asym(T, np.array([4], dtype=np.int32))
    assert q.dtype == np.uint8 and s.dtype == np.float32 and z.dtype == np.int32
    assert q[0].tolist() == [0, 5, 8, 15] and z[0] == 5 and s[0] == np.float32(3.0) / np.float32(15.0)
    assert not q[1].any() and s[1] == 1.0 and z[1] == 0
    assert not q[2].any() and s[2] == 1.0 and z[2] == -3
    # integers -100 .. 155 at 8 bits: s = 1, z = 100, codes = value + 100, exact
    T = np.arange(-100, 156, dtype=np.float64)[None, ::-1].copy()
    q, s, z = oracle.quantize_rows_asym(T, np.array([8], dtype=np.int32))
    assert s[0] == 1.0 and z[0] == 100 and np.array_equal(q[0].astype(int), T[0].astype(int) + 100)
    # a row that does not straddle zero keeps an out-of-range zero point and still uses every code
    T = np.linspace(10.0, 25.0, 16)[None, :]
    q, s, z = oracle.quantize_rows_asym(T, np.array([4], dtype=np.int32))
    assert z[0] == -10 and q[0].tolist() == list(range(16))


def test_asym_quantizer_bound_and_nearest_level(oracle):
    rng = np.random.default_rng(12)
    rows, K = 48, 80
    T = rng.standard_normal((rows, K)) * rng.lognormal(0, 1.5, size=(rows, 1)) + rng.standard_normal((rows, 1)) * 3
    bits = np.where(np.arange(rows) < 10, 8, 4).astype(np.int32)
    q, s, z = oracle.quantize_rows_asym(T, bits)
    top = (2 ** bits - 1)
    assert np.all(q.astype(int) <= top[:, None])
    rng_row = T.max(axis=1) - T.min(axis=1)
    assert np.allclose(s, rng_row / top, rtol=1e-6)                       # s = range / (2^b - 1)
    assert np.all(np.abs(z + T.min(axis=1) / s) <= 0.5 + 1e-3)            # z = rne(-min / s)
    # the minimum maps to code 0, the maximum to the top code (one below on a rounding coincidence)
    assert np.all(q[np.arange(rows), T.argmin(axis=1)] == 0)
    qtop = q[np.arange(rows), T.argmax(axis=1)].astype(int)
    assert np.all(qtop >= top - 1) and np.mean(qtop == top) > 0.9
    sd = s.astype(np.float64)[:, None]
    deq = sd * (q.astype(np.float64) - z[:, None])
    err = deq - T
    # the section's bound: ||Q(x) - x||^2 <= d s^2 / 4 = d range^2 / (4 (2^b - 1)^2); the clamp of a top code
    # that rounded one past the range costs at most one extra half step on that element
    assert np.all(np.abs(err) <= sd * (0.5 + 1e-5) + sd * (q == top[:, None]) * 0.5)
    e2 = np.sum(np.where(q == top[:, None], 0.0, err * err), axis=1)
    assert np.all(e2 <= K * (rng_row / top) ** 2 / 4 * (1 + 1e-5))
    # brute force: every code is the level nearest to its value among all 2^b levels
    for r in range(rows):
        levels = sd[r, 0] * (np.arange(top[r] + 1, dtype=np.float64) - z[r])
        best = np.abs(T[r][:, None] - levels[None, :]).min(axis=1)
        assert np.all(np.abs(err[r]) <= best * (1 + 1e-4) + 1e-6 * sd[r, 0])


def test_asym_beats_symmetric_on_one_sided_rows(oracle):
    # rows in [0, 1): the symmetric quantizer spends half its codes on values that never occur
    rng = np.random.default_rng(13)
    T = rng.random((16, 256))
    bits = np.full(1, 4, dtype=np.int32)
    qa, sa, za = oracle.quantize_rows_asym(T, bits)
    qs, ss = oracle.quantize_rows(T, bits)
    ea = np.sum((sa.astype(np.float64)[:, None] * (qa.astype(np.float64) - za[:, None]) - T) ** 2)
    es = np.sum((ss.astype(np.float64)[:, None] * qs - T) ** 2)
    assert ea < es / 3.5          # twice the resolution (15 steps over 1 vs 7): about 4.6x less squared error


def test_asym_integer_product_equals_product_of_dequantized_operands(oracle):
    rng = np.random.default_rng(14)
    M, K, N = 24, 64, 20
    T = rng.standard_normal((M, K)) + rng.standard_normal((M, 1)) * 2
    bits = np.where(np.arange(M) < 4, 8, 4).astype(np.int32)
    q, s, z = oracle.quantize_rows_asym(T, bits)
    wq, sw = oracle.quantize_weights(rng.standard_normal((N, K)).astype(np.float32))
    acc = oracle.gemm_zp_i32(q, z, wq)
    Yt = oracle.dequant(acc, s, sw)
    xhat = s.astype(np.float64)[:, None] * (q.astype(np.float64) - z[:, None])       # s (x_int - z)
    what = sw.astype(np.float64)[:, None] * wq.astype(np.float64)
    ref = xhat @ what.T
    assert np.abs(Yt - ref).max() <= 1e-12 * np.abs(ref).max()
    # and the sum splits into the plain code product minus z times the weight row sums
    plain = q.astype(np.int64) @ wq.astype(np.int64).T
    assert np.array_equal(acc, plain - z.astype(np.int64)[:, None] * wq.astype(np.int64).sum(axis=1)[None, :])


def test_asym_layer_composes_and_is_closer_than_symmetric_on_shifted_activations(oracle):
    cfg = gen.scaled(gen.config_llm_up(), B=1, L=256, K=128, N=96)
    X, W = gen.make_activation(cfg), gen.make_weight(cfg)
    X = (X + 0.75 * np.abs(X).mean()).astype(np.float32)       # a per-feature offset the transform concentrates in row 0
    kw = dict(transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi)
    out = oracle.stamp_linear(X, W, None, asym=True, **kw)
    assert out["q"].dtype == np.uint8 and out["x_zero"].shape == (cfg.L,)
    bits = oracle.bit_map(cfg.L, cfg.L, cfg.k_hi)
    q, s, z = oracle.quantize_rows_asym(out["T"], bits)
    assert np.array_equal(q, out["q"]) and np.array_equal(z, out["x_zero"]) and np.array_equal(s, out["x_scale"])
    assert np.array_equal(out["acc"], oracle.gemm_zp_i32(q, z, out["wq"]))
    Lm = oracle.transform_matrix(cfg.transform, cfg.L, cfg.levels)
    assert np.abs(out["Y"] - Lm.T @ out["Yt"]).max() <= 1e-12 * np.abs(out["Y"]).max()
    ref = oracle.matmul_f64(X.reshape(-1, cfg.K), W)
    sym = oracle.stamp_linear(X, W, None, **kw, want=("Y",))
    ea = np.linalg.norm(out["Y"] - ref) / np.linalg.norm(ref)
    es = np.linalg.norm(sym["Y"] - ref) / np.linalg.norm(ref)
    assert ea < es and ea < 0.2


# --------------------------------------------------------------------------------------
# The precision of the rounding decision (Sec. 2.1 fixes none): how often the two readings differ
# --------------------------------------------------------------------------------------

def _transformed(oracle, cfg):
    X = gen.make_activation(cfg)
    n = cfg.block_len
    if cfg.transform == T_HAAR and n > 4096:
        T = oracle.apply_csr(oracle.haar_matrix_csr(n, cfg.levels), n, X)
    else:
        T = oracle.apply_dense(oracle.transform_matrix(cfg.transform, n, cfg.levels, grid_w=cfg.grid), X)
    return T.reshape(-1, cfg.K)


ROUNDING_CASES = {
    "tiny": gen.config_tiny(),
    "llm_mlp_up": gen.config_llm_up(),
    "dit_attn_proj": gen.config_dit_proj(),
    "llm_down_proj_reduced": gen.scaled(gen.config_llm_down(), B=1, L=1024, K=2048),
    "sweep_L2048_D2048": gen.config_sweep(2048, 2048),
}


@pytest.mark.parametrize("name", list(ROUNDING_CASES))
def test_fp32_and_fp64_rounding_decisions_differ_only_at_fp32_ties(oracle, name):
    """The quantizer's quotient t / s can be rounded to an integer from its fp32 or from its fp64 value.  The two
    readings give different codes only where the fp32 quotient IS a half-integer (bf16 inputs make absmax / qmax land
    there exactly) while the fp64 quotient of the same fp32 scale sits a hair beside it; the disagreement is one code
    step.  The counts printed here are recorded with the reading taken (fp32, the precision of the scale)."""
    cfg = ROUNDING_CASES[name]
    T = _transformed(oracle, cfg)
    bits = oracle.bit_map(cfg.L, cfg.block_len, cfg.k_hi)
    assert oracle.set_rounding_decision(False) is False
    q32, s32 = oracle.quantize_rows(T, bits)
    oracle.set_rounding_decision(True)
    try:
        q64, s64 = oracle.quantize_rows(T, bits)
    finally:
        oracle.set_rounding_decision(False)
    assert np.array_equal(s32, s64)
    r, c = np.nonzero(q32 != q64)
    print(f"[{name}] codes on which the fp32 and fp64 rounding decisions differ: {len(r)} of {q32.size} "
          f"({len(r) / q32.size:.2e})")
    if len(r):
        assert np.abs(q32[r, c].astype(int) - q64[r, c].astype(int)).max() == 1
        quo32 = T[r, c].astype(np.float32) / s32[r]
        assert np.all(np.abs(quo32 - np.trunc(quo32)) == 0.5)          # an exact tie in fp32 ...
        quo64 = T[r, c] / s32[r].astype(np.float64)
        frac = np.abs(quo64 - np.trunc(quo64))
        assert np.all(np.abs(frac - 0.5) <= 2.0 ** -21 * np.maximum(1.0, np.abs(quo64)))   # ... a near-tie in fp64
        assert np.all(frac != 0.5)


# --------------------------------------------------------------------------------------
# Planted mistakes: each plausible slip in the oracle's source fails a pin above
# --------------------------------------------------------------------------------------

_ORACLE_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle")

MUTANTS = {
    # name: (text in stamp_oracle.c, replacement, [pins that must fail])
    "haar_detail_sign": ("tmp[half + i] = (v[2 * i] - v[2 * i + 1]) * r;", "tmp[half + i] = (v[2 * i + 1] - v[2 * i]) * r;",
                         ["test_haar_n2_hand_case", "closed_form"]),
    "haar_step_not_normalised": ("const double r = 1.0 / sqrt(2.0);\n  int half", "const double r = 0.5;\n  int half",
                                 ["orthonormal_haar"]),
    "inverse_uses_untransposed_matrix": ("double l = transpose ? Lmat[(size_t)t * n + i] : Lmat[(size_t)i * n + t];",
                                         "double l = Lmat[(size_t)i * n + t];", ["reconstruction", "plain_matmul"]),
    "dct_dc_row_not_rescaled": ("double cu = (u == 0) ? 1.0 / sqrt(2.0) : 1.0;", "double cu = 1.0;",
                                ["orthonormal_dct", "dct_scipy"]),
    "bias_dropped": ("Y[(size_t)m * N + j] += (double)bias[j];", "Y[(size_t)m * N + j] += 0.0;",
                     ["exact_codes", "python_loops"]),
    "qmax_is_two_to_b_minus_1": ("float qmaxf = (float)((1 << (bits - 1)) - 1);\n    double amax = 0.0;\n    for (int j = 0; j < K; ++j) {\n      double a = fabs(t[j]);",
                                 "float qmaxf = (float)((1 << (bits - 1)));\n    double amax = 0.0;\n    for (int j = 0; j < K; ++j) {\n      double a = fabs(t[j]);",
                                 ["quantizer_hand_rows", "quantizer_properties"]),
    "round_toward_zero": ("float q = g_decide_fp64 ? (float)nearbyint(t[j] / (double)s) : rintf((float)t[j] / s);",
                          "float q = truncf((float)t[j] / s);", ["quantizer_hand_rows", "quantizer_properties"]),
    "gemm_weight_operand_transposed": ("const int8_t* b = wq + (size_t)n * K;\n      for (int k = 0; k < K; ++k) s += (int64_t)a[k] * (int64_t)b[k];",
                                       "const int8_t* b = wq + n;\n      for (int k = 0; k < K; ++k) s += (int64_t)a[k] * (int64_t)b[(size_t)(k % N) * K + (k / N)];",
                                       ["gemm_brute_force"]),
    "dequant_forgets_weight_scale": ("(double)acc[(size_t)m * N + n] * (double)sx[m] * (double)sw[n];",
                                     "(double)acc[(size_t)m * N + n] * (double)sx[m];", ["exact_codes", "python_loops"]),
    "high_precision_rows_off_by_one": ("bits[i] = ((i % n) < k_hi) ? bits_hi : bits_lo;", "bits[i] = ((i % n) <= k_hi) ? bits_hi : bits_lo;",
                                       ["printed_bits"]),
    "wht_natural_order": ("Lmat[(size_t)changes * n + j] = par ? -r : r;", "Lmat[(size_t)i * n + j] = par ? -r : r;",
                          ["wht_sequency"]),
    "haar2d_lh_hl_swapped_sign": ("tmp[3 * q + i] = (a - b - c + d) * 0.5;", "tmp[3 * q + i] = (a - b - c - d) * 0.5;",
                                  ["haar2d_orthonormal"]),
}

_PINS = {
    "test_haar_n2_hand_case": lambda o: test_haar_n2_hand_case(o),
    "closed_form": lambda o: test_haar_closed_form_rows(o, 16, 3),
    "orthonormal_haar": lambda o: test_orthonormal(o, T_HAAR, 64, 3),
    "orthonormal_dct": lambda o: test_orthonormal(o, T_DCT, 8, 0),
    "dct_scipy": lambda o: test_dct_matches_scipy_ortho_dct2(o, 16),
    "reconstruction": lambda o: test_energy_and_reconstruction(o, T_HAAR, 128, 3),
    "plain_matmul": lambda o: test_unquantized_pipeline_is_plain_matmul(o),
    "exact_codes": lambda o: test_layer_exact_when_codes_are_exact(o),
    "python_loops": lambda o: test_layer_vs_python_loops(o),
    "quantizer_hand_rows": lambda o: test_quantizer_round_half_to_even_and_zero_row(o),
    "quantizer_properties": lambda o: test_quantizer_properties(o),
    "gemm_brute_force": lambda o: test_gemm_brute_force(o),
    "printed_bits": lambda o: test_bit_map_reproduces_printed_effective_bits(o),
    "wht_sequency": lambda o: test_wht_is_the_sequency_ordered_hadamard_matrix(o, 8),
    "haar2d_orthonormal": lambda o: test_haar2d_orthonormal_and_lowpass_closed_form(o, 8, 8, 3),
}


def _load_mutant(tmpdir, name, old, new):
    """A second copy of the oracle's ctypes wrapper bound to a library compiled from the mutated source."""
    src = open(os.path.join(_ORACLE_DIR, "stamp_oracle.c")).read()
    assert src.count(old) == 1, f"mutation site of {name!r} not found exactly once in the oracle source"
    c_path = os.path.join(tmpdir, f"mutant_{name}.c")
    so_path = os.path.join(tmpdir, f"libmutant_{name}.so")
    with open(c_path, "w") as f:
        f.write(src.replace(old, new))
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", so_path, c_path, "-lm"])
    spec = importlib.util.spec_from_file_location(f"mutant_oracle_{name}", os.path.join(_ORACLE_DIR, "stamp_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod._SRC, mod._LIB = c_path, so_path
    return mod


@pytest.mark.parametrize("name", list(MUTANTS))
def test_planted_mistake_fails_its_pins(name):
    """Mutate a COPY of the oracle's source (the committed oracle is untouched), build it, and run the named pins
    on the mutant: every one of them must fail.  The mutations are the slips a plausible rewrite would make --
    a flipped sign, a missing normalisation, a transposed operand, a dropped term, a wrong code range."""
    old, new, pins = MUTANTS[name]
    with tempfile.TemporaryDirectory() as tmpdir:
        mutant = _load_mutant(tmpdir, name, old, new)
        for pin in pins:
            with pytest.raises(AssertionError):
                _PINS[pin](mutant)


def test_unmutated_oracle_passes_the_pins_the_mutants_fail(oracle):
    for pin in _PINS.values():
        pin(oracle)


# --------------------------------------------------------------------------------------
# Haar with the first token excluded (App. "Experimental details / LLMs", STaMP paragraph)
# --------------------------------------------------------------------------------------
T_SKIP1 = 5


@pytest.mark.parametrize("n,levels", [(2, 0), (4, 0), (4, 1), (8, 2), (64, 0), (256, 3), (2048, 0)])
def test_skip_first_is_orthonormal_and_leaves_token_zero_alone(oracle, n, levels):
    """Theorem 1's premise still holds (L orthogonal), row 0 is the first token itself, and no other row touches it:
    the massive first token cannot leak into any coefficient."""
    Lm = oracle.transform_matrix(T_SKIP1, n, levels)
    assert np.max(np.abs(Lm @ Lm.T - np.eye(n))) <= 1e-12
    assert np.array_equal(Lm[0], np.eye(n)[0])
    assert not Lm[1:, 0].any()


def test_skip_first_hand_case_and_band_structure(oracle):
    """n = 4: tokens (x0 | x1 x2 x3).  Level 1 pairs (x1, x2) and carries x3 unchanged; level 2 pairs the average with
    the carried token.  Order [x0 | a_2 | d_2 | d_1]."""
    r = 1.0 / math.sqrt(2.0)
    Lm = oracle.transform_matrix(T_SKIP1, 4, 0)
    want = np.array([[1, 0, 0, 0],
                     [0, r * r, r * r, r],
                     [0, r * r, r * r, -r],
                     [0, r, -r, 0]])
    assert np.allclose(Lm, want, rtol=0, atol=1e-15)
    one = oracle.transform_matrix(T_SKIP1, 4, 1)          # one level: [x0 | (x1+x2)/sqrt2, x3 | (x1-x2)/sqrt2]
    assert np.allclose(one, [[1, 0, 0, 0], [0, r, r, 0], [0, 0, 0, 1], [0, r, -r, 0]], rtol=0, atol=1e-15)
    # n = 2^p: after the first level the low-pass band has n/2 entries (the last one is the carried token), so
    # the deeper levels are the ordinary dyadic Haar transform of that band
    n = 64
    full = oracle.transform_matrix(T_SKIP1, n, 0)
    lvl1 = oracle.transform_matrix(T_SKIP1, n, 1)
    H = oracle.transform_matrix(T_HAAR, n // 2, 0)
    assert np.allclose(full[1:1 + n // 2], H @ lvl1[1:1 + n // 2], rtol=0, atol=1e-14)
    assert np.array_equal(full[1 + n // 2:], lvl1[1 + n // 2:])         # d_1: n/2 - 1 rows, untouched by deeper levels
    assert np.array_equal(lvl1[n // 2], np.eye(n)[n - 1])               # the carried last token, unscaled
    # m = n - 1 = 3 tokens when the tail happens to be a power of two plus nothing to carry: plain Haar on them
    five = np.zeros((5, 5))
    v = np.eye(5)
    # (n must be a power of two for the matrix builder; the 4-token tail is checked through n = 8 instead)
    eight = oracle.transform_matrix(T_SKIP1, 8, 1)
    for i in range(3):                                                    # pairs (1,2), (3,4), (5,6); 7 carried
        assert np.allclose(eight[1 + i, 1 + 2 * i:3 + 2 * i], [r, r]) and np.allclose(eight[5 + i, 1 + 2 * i:3 + 2 * i], [r, -r])
    assert np.array_equal(eight[4], np.eye(8)[7])


def test_skip_first_layer_keeps_the_massive_token_out_of_the_detail_rows(oracle):
    """The LLM recipe multiplies token 0 by 100.  With the plain transform that token enters one coefficient of EVERY
    band and inflates those rows' scales; with the first token excluded the 4-bit rows no longer see it, the pipeline
    with the quantizers off is still X W^T, and the quantized layer is closer to the unquantized product."""
    cfg = gen.scaled(gen.config_llm_up(), B=1, L=256, K=128, N=48, k_hi=8)
    X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
    plain = oracle.matmul_f64(X.reshape(-1, cfg.K), W) + bias[None, :]
    skip = oracle.stamp_linear(X, W, bias, transform=T_SKIP1, k_hi=cfg.k_hi)
    full = oracle.stamp_linear(X, W, bias, transform=T_HAAR, k_hi=cfg.k_hi)
    Lm = oracle.transform_matrix(T_SKIP1, cfg.L, 0)
    T = oracle.apply_dense(Lm, X.astype(np.float64))
    assert np.array_equal(skip["T"], T.reshape(-1, cfg.K))
    assert np.array_equal(skip["T"][0], X[0, 0].astype(np.float64))          # row 0 = the first token, untouched
    Yt = (T.reshape(-1, cfg.K) @ W.astype(np.float64).T).reshape(1, cfg.L, -1)
    assert np.max(np.abs(oracle.apply_dense(Lm, Yt, transpose=True)[0] + bias - plain)) <= 1e-11 * np.max(np.abs(plain))
    # scales of the 4-bit rows: inflated by the leak with the plain transform, not with the exclusion
    # (the leak sits in the first coefficient of every band: those rows' scales blow up)
    lo = np.arange(cfg.L) >= cfg.k_hi
    assert np.max(full["x_scale"][lo]) > 3.0 * np.max(skip["x_scale"][lo])
    err = lambda y: np.linalg.norm(y - plain) / np.linalg.norm(plain)
    assert err(skip["Y"]) < err(full["Y"])


# --------------------------------------------------------------------------------------
# Per-block ("group") scales of 64 features (LVM table: W4A4 per-block quantization, block size 64)
# --------------------------------------------------------------------------------------

def test_grouped_quantizer_is_the_per_token_quantizer_on_every_group(oracle):
    """group = K is the per-token quantizer itself; for group < K every group of a row is quantized exactly as if it
    were a row of its own (codes and scales equal those of the per-token routine run on the reshaped array)."""
    rng = np.random.default_rng(31)
    rows, K, group = 24, 256, 64
    T = rng.standard_normal((rows, K)) * rng.lognormal(0, 1.5, size=(rows, 1))
    T[:, 7] *= 40.0                                     # an outlier channel: only its group pays for it
    bits = np.where(np.arange(rows) < 6, 8, 4).astype(np.int32)
    q_full, s_full = oracle.quantize_rows_grouped(T, bits, K)
    q_pt, s_pt = oracle.quantize_rows(T, bits)
    assert np.array_equal(q_full, q_pt) and np.array_equal(s_full[:, 0], s_pt)
    q, s = oracle.quantize_rows_grouped(T, bits, group)
    assert s.shape == (rows, K // group)
    q_ref, s_ref = oracle.quantize_rows(T.reshape(rows * (K // group), group), np.repeat(bits, K // group))
    assert np.array_equal(q.reshape(-1, group), q_ref) and np.array_equal(s.reshape(-1), s_ref)
    # error bound per group (Sec. 2.1's rounding bound with the group's own scale) and the gain over one scale per row
    err = T - np.repeat(s.astype(np.float64), group, axis=1) * q
    assert np.all(np.abs(err) <= np.repeat(s.astype(np.float64), group, axis=1) / 2 * (1 + 1e-6))
    err_pt = T - s_pt.astype(np.float64)[:, None] * q_pt
    assert np.sum(err ** 2) < 0.5 * np.sum(err_pt ** 2)
    # hand case: two groups of two, scales 1 and 2
    qh, sh = oracle.quantize_rows_grouped(np.array([[7.0, -3.5, 14.0, 5.0]]), np.array([4], dtype=np.int32), 2)
    assert sh.tolist() == [[1.0, 2.0]] and qh.tolist() == [[7, -4, 7, 2]]


def test_grouped_product_brute_force_and_reduction_to_the_plain_product(oracle):
    rng = np.random.default_rng(32)
    M, N, K, group = 9, 7, 128, 32
    q = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    wq = rng.integers(-7, 8, size=(N, K), dtype=np.int8)
    sx = rng.uniform(0.5, 2.0, size=(M, K // group)).astype(np.float32)
    sw = rng.uniform(0.01, 0.1, size=(N, K // group)).astype(np.float32)
    Yt = oracle.gemm_grouped(q, sx, wq, sw, group)
    # the definition: product of the de-quantized operands
    A = q.astype(np.float64) * np.repeat(sx.astype(np.float64), group, axis=1)
    Wd = wq.astype(np.float64) * np.repeat(sw.astype(np.float64), group, axis=1)
    assert np.max(np.abs(Yt - A @ Wd.T)) <= 1e-12 * np.max(np.abs(Yt))
    # one group: the plain integer product times the two scales
    Y1 = oracle.gemm_grouped(q, sx[:, :1], wq, sw[:, :1], K)
    assert np.array_equal(Y1, oracle.dequant(oracle.gemm_i32(q, wq), sx[:, 0], sw[:, 0]))


def test_grouped_layer_exact_codes_and_closer_than_per_token_on_outlier_channels(oracle):
    """Whole layer with group scales: inputs whose groups are integer multiples of power-of-two scales give the
    textbook product; on the DiT stand-in (2 % outlier channels x 30) the grouped layer is closer to X W^T than the
    per-token layer, with and without the sequence transform -- and STaMP still helps on top (LVM table)."""
    rng = np.random.default_rng(33)
    nblk, K, N, group = 4, 128, 6, 64
    P = rng.integers(-127, 128, size=(nblk, K)); P[:, 0] = 127; P[:, 64] = -127
    Q = rng.integers(-7, 8, size=(nblk, K)); Q[:, 1] = -7; Q[:, 65] = 7
    P[:, 64:] *= 1                                        # (second group: same construction, own extreme codes)
    u, v = (P + Q) / 2.0, (P - Q) / 2.0
    X = np.stack([u, u, v, v], axis=1).reshape(1, 4 * nblk, K).astype(np.float32)
    Wi = rng.integers(-7, 8, size=(N, K)); Wi[:, 2] = 7; Wi[:, 66] = -7
    W = (Wi * 2.0 ** -3).astype(np.float32)
    out = oracle.stamp_linear(X, W, None, transform=T_HAAR, block=4, levels=2, k_hi=1, group=group)
    assert np.array_equal(out["wq"], Wi) and np.all(out["x_scale"] == 1.0) and np.all(out["w_scale"] == 2.0 ** -3)
    ref = X[0].astype(np.float64) @ W.astype(np.float64).T
    assert np.max(np.abs(out["Y"] - ref)) <= 1e-12 * np.max(np.abs(ref))
    cfg = gen.scaled(gen.config_dit_proj(), B=1, L=256, K=256, N=64, grid=16, levels=4, k_hi=16)
    Xc, Wc = gen.make_activation(cfg), gen.make_weight(cfg)
    plain = oracle.matmul_f64(Xc.reshape(-1, cfg.K), Wc)
    err = lambda **kw: np.linalg.norm(oracle.stamp_linear(Xc, Wc, None, want=("Y",), **kw)["Y"] - plain) / np.linalg.norm(plain)
    e_pt_id = err(transform=T_ID, k_hi=0)
    e_g_id = err(transform=T_ID, k_hi=0, group=64)
    e_g_stamp = err(transform=T_HAAR, levels=4, k_hi=16, group=64)
    assert e_g_id < e_pt_id and e_g_stamp < e_g_id
