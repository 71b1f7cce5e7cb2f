"""Parity at the full sizes of the named configurations, in the launch configuration the
benchmark times (stamp_linear_fused on bf16 activations with prepared int8 weight codes).

The oracle's integer GEMM is a triple loop, so the output is compared on a sample of output
channels: output channels are independent given the activation codes, and the weight generator
reproduces any subset of rows of the full matrix.  Transformed values are compared on a sample
of input channels (the sequence transform acts on every channel separately); scales and codes
are compared in full.  Tolerances are those of the stage-wise parity tests.
"""
import math

import numpy as np
import pytest

from paper_2510_26771_b200 import inputs as gen
from tests import helpers as H
from tests.test_gpu_parity import check_fused_operand, _fused_y_tol

pytestmark = pytest.mark.gpu

T_TOL = 1e-5
CODE_FRAC = 1e-5
Y_TOL = 1e-3


def _scale_rtol(cfg):
    """A scale is absmax / qmax of a transformed row, so it inherits the tolerance on T.  Haar
    coefficients see at most log2(n) fp32 roundings (1e-6 holds); a DCT coefficient is an fp32 sum
    of n products, whose error grows like sqrt(n) ulp, so only the 1e-5 of T itself is promised.  A 2-D Haar
    coefficient of level l is the result of 3 l fp32 additions (9 roundings for 3 levels): 2e-6."""
    if cfg.transform == gen.T_HAAR2D:
        return 2e-6
    return 1e-5 if cfg.transform in (gen.T_DCT2, gen.T_WHT) else 1e-6

FULL = {
    "llm_mlp_up": gen.config_llm_up(),
    "dit_attn_proj": gen.config_dit_proj(),
    "llm_down_proj": gen.config_llm_down(),
    "dit_attn_proj_2d": gen.config_dit_proj_2d(),
    "llm_down_proj_wht": gen.config_llm_down_wht(),
    "llm_mlp_up_zp": gen.config_llm_up_zp(),
    "llm_mlp_up_skip1": gen.config_llm_up_skip1(),
    "dit_attn_proj_2d_zp": gen.config_dit_proj_2d_zp(),
}
# the throughput sweep: all twelve shapes
for _L in gen.SWEEP_L:
    for _D in gen.SWEEP_D:
        _c = gen.config_sweep(_L, _D)
        FULL[_c.name] = _c


def _oracle_transform_cols(oracle, cfg, Xc):
    """T = L X on a channel subset Xc [B, L, C] with the oracle's explicit matrix."""
    n = cfg.block_len
    if cfg.transform == gen.T_HAAR and n > 4096:
        return oracle.apply_csr(oracle.haar_matrix_csr(n, cfg.levels), n, Xc)
    return oracle.apply_dense(oracle.transform_matrix(cfg.transform, n, cfg.levels, grid_w=cfg.grid), Xc)


@pytest.mark.parametrize("name", list(FULL))
def test_full_size_parity(oracle, name):
    import torch
    from paper_2510_26771_b200 import binding as st
    cfg = FULL[name]
    B, L, K, N, M = cfg.B, cfg.L, cfg.K, cfg.N, cfg.M
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, zero_point=cfg.zero_point)
    X = gen.make_activation(cfg)
    rng = np.random.default_rng(1234)
    ncols = min(N, 64)
    cols = np.sort(rng.choice(N, size=ncols, replace=False))
    Wc = gen.make_weight(cfg, cols)
    bias = gen.make_bias(cfg)
    ref = oracle.stamp_linear(X, Wc, bias[cols], transform=cfg.transform, block=cfg.block, levels=cfg.levels,
                              k_hi=cfg.k_hi, grid_w=cfg.grid, asym=cfg.zero_point, want=("x_scale", "q", "Y"))

    Xd = H.to_device(X, cfg.dtype)
    ws = st.alloc_workspace(c, B, L, K, N)

    # a1 on a sample of input channels
    chans = np.sort(rng.choice(K, size=min(K, 96), replace=False))
    T_ref = _oracle_transform_cols(oracle, cfg, np.ascontiguousarray(X[:, :, chans])).reshape(M, -1)
    T = st.stamp_debug_transform(c, Xd, ws)
    T_s = T.reshape(M, K)[:, torch.from_numpy(chans).cuda()].cpu().numpy().astype(np.float64)
    del T
    assert H.rel_fro(T_s, T_ref) <= T_TOL
    col_max = np.abs(T_ref).max(axis=1, keepdims=True)
    assert np.all(np.abs(T_s - T_ref) <= T_TOL * np.maximum(col_max, 1e-30))

    # a2-a3 in full
    q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
    codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, B, L, K).cpu().numpy().reshape(M, K)
    if cfg.zero_point:
        # stored codes and zero points are offset by half the code range; a zero point within fp32 error of
        # a rounding tie may come out one off, and such a row is compared through its centred codes
        xs, zc = st.split_zero_points(xs)
        half = np.where((np.arange(M) % cfg.block_len) < cfg.k_hi, 128, 8).astype(np.int32)
        dz = zc.cpu().numpy().reshape(-1) + half - ref["x_zero"]
        assert np.abs(dz).max() <= 1 and np.count_nonzero(dz) <= int(math.ceil(CODE_FRAC * M))
        print(f"[{name}] rows with the zero point off by one: {np.count_nonzero(dz)} of {M}")
        codes = (codes.astype(np.int16) + half[:, None] - dz[:, None]).astype(np.int16)
        codes = np.where((dz != 0)[:, None], np.clip(codes, 0, 2 * half[:, None] - 1), codes)
        assert np.allclose(xs.cpu().numpy().reshape(-1), ref["x_scale"], rtol=2 * _scale_rtol(cfg), atol=0)
    else:
        assert np.allclose(xs.cpu().numpy().reshape(-1), ref["x_scale"], rtol=_scale_rtol(cfg), atol=0)
    bad, worst = H.code_mismatch(codes, ref["q"])
    print(f"[{name}] code mismatches {bad} of {codes.size} (max |diff| {worst})")
    assert worst <= 1 and bad <= int(math.ceil(CODE_FRAC * codes.size))
    del codes, q_hi, q_lo

    # the operand the timed route feeds its GEMM (tile / patch order), code by code
    check_fused_operand(st, c, cfg, Xd, ws, ref["q"], ref["x_scale"], ref_zero=ref.get("x_zero"), label=name)

    # the whole layer as the benchmark runs it; fp32 and bf16 output
    Wd = H.to_device(gen.make_weight(cfg), cfg.dtype)
    wq, w_scale = st.stamp_quantize_weights(c, Wd)
    w8 = st.stamp_prepare_weights(c, wq)
    del Wd
    bd = torch.from_numpy(bias).cuda()
    cols_d = torch.from_numpy(cols).cuda()
    Y = st.stamp_linear_fused(c, Xd, w8, st.W_INT8, w_scale, bd, ws)
    Y_s = Y.reshape(M, N)[:, cols_d].cpu().numpy()
    del Y
    err = H.rel_fro(Y_s, ref["Y"])
    print(f"[{name}] output relative Frobenius error {err:.2e} on {ncols} sampled channels")
    # (the tight bound presumes the oracle's codes; a code that sat on a rounding boundary and fell the other way --
    #  allowed up to 1e-5 of them -- moves the output by a code step of its row, far more than fp32 rounding)
    assert err <= (_fused_y_tol(cfg) if bad == 0 else Y_TOL)
    Yb = st.stamp_linear_fused(c, Xd, w8, st.W_INT8, w_scale, bd, ws, out_dtype=torch.bfloat16)
    Yb_s = Yb.reshape(M, N)[:, cols_d].float().cpu().numpy()
    # bf16 output: the fp32 result rounded once (2^-9 relative) on top of the fp32 path's own error
    assert H.rel_fro(Yb_s, ref["Y"]) <= Y_TOL + 2.0 ** -8
    assert np.all(np.abs(Yb_s - Y_s) <= np.abs(Y_s) * 2.0 ** -8 + 1e-30)
    assert st.stamp_last_device_status() == 0
