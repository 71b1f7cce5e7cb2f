"""Parity of the CUDA path against the CPU oracle, stage by stage, through the C ABI.
Tolerances: T within 1e-5 relative; codes bit-exact except at most 1e-5 of them off by +-1
(ties at rounding boundaries); int32 accumulators bit-exact given identical codes; final fp32
output within 1e-3 relative Frobenius error of the fp64 oracle."""
import math

import numpy as np
import pytest

from paper_2510_26771_b200 import inputs as gen
from tests import helpers as H

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


@pytest.fixture(scope="module")
def st():
    import torch
    from paper_2510_26771_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return binding


def _cfg_struct(st, cfg):
    return st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid)


def _oracle_all(oracle, cfg, X, W, bias=None, want=("T", "x_scale", "q", "w_scale", "wq", "acc", "Yt", "Y")):
    return oracle.stamp_linear(X, W, bias, transform=cfg.transform, block=cfg.block, levels=cfg.levels,
                               k_hi=cfg.k_hi, grid_w=cfg.grid, want=want)


def _allowed(count):
    # at most 1e-5 of the codes, rounded up to a whole code
    return int(math.ceil(CODE_FRAC * count))


# Output tolerance of the one-call layer where its inverse is exact fp32 butterflies (Haar, 2-D Haar): with the
# codes equal to the oracle's, what is left is fp32 rounding in the de-quantization and the synthesis (measured
# 6e-8 to 8e-8).  The 1e-3 of the specification is kept for the DCT / Walsh-Hadamard routes, whose layer inverse
# runs on the tensor cores with a split-bf16 operand (about 2^-17 per term).
Y_TOL_HAAR = 1e-5


def _fused_y_tol(cfg):
    return Y_TOL if cfg.transform in (gen.T_DCT2, gen.T_WHT) else Y_TOL_HAAR


def check_fused_operand(st, c, cfg, Xd, ws, ref_q, ref_scale, ref_zero=None, label=""):
    """The codes the one-call layer feeds its GEMM (tile / patch order, mapped back to logical order by the
    library's debug export) against the oracle's, code by code; the per-row factor against scale x 2^(-level/2)
    (1-D Haar; the plain scale above level 8) or scale x 2^(-level) (2-D Haar).  Returns False when the
    configuration keeps its operand in logical order (nothing to map back)."""
    try:
        codes, factor, level, zero = st.stamp_debug_fused_operand(c, Xd, cfg.N, ws)
    except st.StampError as e:
        assert e.status == 2
        return False
    M, K = cfg.M, cfg.K
    codes = codes.cpu().numpy().reshape(M, K).astype(np.int64)
    factor = factor.cpu().numpy().reshape(M).astype(np.float64)
    level = level.cpu().numpy().reshape(M).astype(np.int64)
    zero = zero.cpu().numpy().reshape(M).astype(np.int64)
    if cfg.transform == gen.T_HAAR2D:
        want = ref_scale.astype(np.float64) * 2.0 ** (-level)
    else:
        want = ref_scale.astype(np.float64) * np.where(level > 8, 1.0, 2.0 ** (-level / 2.0))
    assert np.allclose(factor, want, rtol=2e-6, atol=0)
    if ref_zero is not None:
        half = np.where((np.arange(M) % cfg.block_len) < cfg.k_hi, 128, 8).astype(np.int64)
        dz = zero + half - ref_zero
        assert np.abs(dz).max() <= 1 and np.count_nonzero(dz) <= _allowed(M), (np.abs(dz).max(), np.count_nonzero(dz))
        codes = codes + half[:, None] - dz[:, None]      # rows whose zero point sits one off move as a whole
    bad, worst = H.code_mismatch(codes, ref_q.astype(np.int64))
    print(f"[{label}] fused-route operand: {bad} of {codes.size} codes differ from the oracle's (max |diff| {worst})")
    assert worst <= 1 and bad <= _allowed(codes.size), (bad, worst, codes.size)
    return True


CASES = {
    "tiny": gen.config_tiny(),
    # several channel and token tiles with ragged tails (N not a multiple of 128, 3 K blocks)
    "ragged": gen.scaled(gen.config_llm_up(), B=2, L=512, K=384, N=392, k_hi=16),
    # fixed-depth Haar on a 2-D-grid-like input, block smaller than the sequence
    "blocked": gen.scaled(gen.config_dit_proj(), B=1, L=1024, K=256, N=136, grid=32, block=256, levels=6, k_hi=4),
    # one-level transform and the identity (pure mixed-precision quantization)
    "one_level": gen.scaled(gen.config_sweep(512, 2048), L=256, K=128, N=64, levels=1, k_hi=128),
    "identity": gen.scaled(gen.config_sweep(512, 2048), L=192 + 64, K=256, N=128, transform=gen.T_IDENTITY, k_hi=8),
    # wide feature axes: 8 and 4 tokens per CTA in the fused transform+quantize kernel
    "wide_k4096": gen.scaled(gen.config_llm_up(), L=256, K=4096, N=64, k_hi=8),
    "wide_k8192": gen.scaled(gen.config_sweep(512, 8192), L=128, K=8192, N=64, levels=5, k_hi=4),
    # blockwise DCT-II: several blocks per sequence, ragged output-channel tile; a short block
    "dct_blocks": gen.scaled(gen.config_llm_down(), B=2, L=512, K=384, N=136),
    # output width a multiple of 64: the layer's inverse DCT also runs on the tensor cores
    "dct_tensor_inverse": gen.scaled(gen.config_llm_down(), B=1, L=768, K=256, N=192),
    # Walsh-Hadamard blocks: 256 tokens (tensor cores, one exact bf16 term) and a short block (general kernels)
    "wht_blocks": gen.scaled(gen.config_llm_down_wht(), B=2, L=512, K=384, N=192),
    "wht_short_block": gen.scaled(gen.config_llm_down_wht(), B=1, L=256, K=128, N=72, block=64, k_hi=4),
    "dct_short_block": gen.scaled(gen.config_llm_down(), B=1, L=256, K=128, N=64, block=32, k_hi=4),
    # fused inverse epilogue with 5 and 7 levels closed inside a 256-token tile (8 and 6 are covered above)
    "tile_depth5": gen.scaled(gen.config_dit_proj(), B=2, L=512, K=256, N=200, grid=0, block=256, levels=5, k_hi=8,
                              recipe="ar1"),
    "tile_depth7": gen.scaled(gen.config_llm_up(), B=1, L=1024, K=384, N=128, levels=7, k_hi=8),
    # twelve levels over two sequences: the five levels above the tensor-core tile are finished by the transform
    # kernel's own tail, and most of their 32 rows per sequence take 4-bit codes (k_hi below the row count)
    "deep_tail_4bit": gen.scaled(gen.config_llm_up(), B=2, L=4096, K=256, N=64, k_hi=8),
    # the same tail with more (sequence, 64-channel strip) items than the GPU has SMs: it then takes 128-channel strips
    "tail_wide_strips": gen.scaled(gen.config_llm_up(), B=8, L=512, K=1280, N=64, k_hi=2),
    # 2-D Haar over the patch grid: square and oblong grids, one to three levels
    "haar2d_3": gen.scaled(gen.config_dit_proj_2d(), B=2, L=1024, K=256, N=136, grid=32, levels=3, k_hi=16),
    "haar2d_1": gen.scaled(gen.config_dit_proj_2d(), B=1, L=256, K=128, N=64, grid=16, levels=1, k_hi=64),
    # oblong grid (32 wide, 16 high), fp32 input, ragged channel tile: the fused patch-order route again
    "haar2d_oblong": gen.scaled(gen.config_dit_proj_2d(), B=3, L=512, K=128, N=72, grid=32, levels=3, k_hi=8,
                                dtype=gen.F32, recipe="ar1"),
    # the widest patches that still fit in shared memory: 1792 bf16 channels, 896 fp32 channels (224 KB each)
    "haar2d_max_bf16": gen.scaled(gen.config_dit_proj_2d(), B=1, L=256, K=1792, N=64, grid=16, levels=3, k_hi=4),
    # (an AR(1) field: the smooth random field of the patch-grid recipe, kept in fp32, has HH rows 1e6 times
    #  smaller than the values they are differences of, beyond what fp32 butterflies resolve to 1e-5 of the row)
    "haar2d_max_fp32": gen.scaled(gen.config_dit_proj_2d(), B=1, L=256, K=896, N=64, grid=16, levels=3, k_hi=4,
                                  dtype=gen.F32, recipe="ar1"),
    # a patch (64 tokens x 2048 channels) that does not fit in shared memory: row maxima and codes in separate launches
    "haar2d_wide_k": gen.scaled(gen.config_dit_proj_2d(), B=1, L=256, K=2048, N=64, grid=16, levels=3, k_hi=4),
    # Haar with the first token excluded (the LLM setting): full depth with ragged tiles, one level, fp32 blocks
    "skip_first": gen.scaled(gen.config_llm_up_skip1(), B=2, L=512, K=384, N=392, k_hi=16),
    "skip_first_one_level": gen.scaled(gen.config_llm_up_skip1(), B=1, L=256, K=128, N=64, levels=1, k_hi=130),
    "skip_first_fp32_blocks": gen.scaled(gen.config_tiny(), B=2, L=256, K=128, N=72, block=64, levels=3, k_hi=8,
                                         transform=gen.T_HAAR_SKIP1),
    # two levels only: no cluster tree, approximation rows quantized by the same kernel
    "two_levels": gen.scaled(gen.config_dit_proj(), B=2, L=256, K=1152, N=128, grid=16, levels=2, k_hi=64),
}


# cases whose one-call route writes the GEMM operand in tile or patch order
FUSED_ORDER_CASES = {"ragged", "blocked", "wide_k4096", "tile_depth5", "tile_depth7", "deep_tail_4bit", "tail_wide_strips", "haar2d_3",
                     "haar2d_oblong", "haar2d_max_bf16", "haar2d_max_fp32", "haar2d_wide_k"}


@pytest.mark.parametrize("name", list(CASES))
def test_stagewise_parity(st, oracle, name):
    import torch
    cfg = CASES[name]
    c = _cfg_struct(st, cfg)
    X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
    ref = _oracle_all(oracle, cfg, X, W, bias)
    B, L, K, N = cfg.B, cfg.L, cfg.K, cfg.N
    Xd, Wd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype)
    bd = torch.from_numpy(bias).cuda()
    ws = st.alloc_workspace(c, B, L, K, N)

    # a1: transform
    T = st.stamp_debug_transform(c, Xd, ws).cpu().numpy().reshape(-1, K).astype(np.float64)
    row_max = np.abs(ref["T"]).max(axis=1, keepdims=True)
    assert np.all(np.abs(T - ref["T"]) <= T_TOL * np.maximum(row_max, 1e-30))
    assert H.rel_fro(T, ref["T"]) <= T_TOL

    # a2-a3: scales and codes
    q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
    codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, B, L, K).cpu().numpy().reshape(-1, K)
    assert np.allclose(xs.cpu().numpy().reshape(-1), ref["x_scale"], rtol=_scale_rtol(cfg), atol=0)
    bad, worst = H.code_mismatch(codes, ref["q"])
    print(f"[{name}] activation code mismatches: {bad} of {codes.size} (max |diff| {worst})")
    assert worst <= 1 and bad <= _allowed(codes.size), (bad, worst, codes.size)
    act_bad = bad

    # a4: weights
    wq, wsc = st.stamp_quantize_weights(c, Wd)
    w8 = st.stamp_prepare_weights(c, wq)
    assert np.array_equal(wsc.cpu().numpy(), ref["w_scale"])
    bad, worst = H.code_mismatch(w8.cpu().numpy(), ref["wq"])
    assert worst <= 1 and bad <= _allowed(w8.numel()), (bad, worst)
    assert np.array_equal(wq.cpu().numpy(), H.pack_nibbles(w8.cpu().numpy()))

    # a5: integer GEMM, fed the ORACLE's codes: accumulators must be bit-identical
    oq_hi, oq_lo = H.pack_codes(ref["q"], cfg.block_len, cfg.k_hi)
    owq = torch.from_numpy(H.pack_nibbles(ref["wq"])).cuda()
    oqh, oql = torch.from_numpy(oq_hi).cuda(), torch.from_numpy(oq_lo).cuda()
    acc = st.stamp_debug_gemm_i32(c, oqh, oql, owq, st.W_PACKED4, B, L, K, N, ws).cpu().numpy()
    assert np.array_equal(acc, ref["acc"])
    ow8 = torch.from_numpy(ref["wq"]).cuda()
    acc = st.stamp_debug_gemm_i32(c, oqh, oql, ow8, st.W_INT8, B, L, K, N, ws).cpu().numpy()
    assert np.array_equal(acc, ref["acc"])

    # a6: de-quantized transformed-domain output from the oracle's codes and scales
    oxs = torch.from_numpy(ref["x_scale"]).cuda()
    ows = torch.from_numpy(ref["w_scale"]).cuda()
    Yt = st.stamp_linear(c, oqh, oql, oxs, owq, st.W_PACKED4, ows, B, L, K, N, ws).cpu().numpy().reshape(-1, N)
    assert H.rel_fro(Yt, ref["Yt"]) <= 1e-6

    # a7-a8: inverse transform + bias from the oracle's Yt
    Ytd = torch.from_numpy(ref["Yt"].astype(np.float32)).cuda().reshape(B, L, N)
    Y = st.stamp_inverse(c, Ytd, bd, ws).cpu().numpy().reshape(-1, N)
    assert H.rel_fro(Y, ref["Y"]) <= 1e-6
    Yb = st.stamp_inverse(c, Ytd, bd, ws, out_dtype=torch.bfloat16).float().cpu().numpy().reshape(-1, N)
    ref_bf16 = gen.round_to_bf16(ref["Y"].astype(np.float32))
    # bf16 output: compare with the oracle's output rounded to bf16, within one bf16 ulp
    # (plus the fp32 path's own error, 1e-5 of the largest output, where outputs nearly cancel)
    assert np.all(np.abs(Yb - ref_bf16) <= np.abs(ref_bf16) * 2.0 ** -7 + 1e-5 * np.abs(ref_bf16).max())

    # whole layer, chained calls and the fused call
    Yt2 = st.stamp_linear(c, q_hi, q_lo, xs, wq, st.W_PACKED4, wsc, B, L, K, N, ws)
    Y2 = st.stamp_inverse(c, Yt2, bd, ws).cpu().numpy().reshape(-1, N)
    assert H.rel_fro(Y2, ref["Y"]) <= Y_TOL
    both = st.stamp_prepare_weights_both(c, wq)
    assert torch.equal(both[:N * K].view(N, K), w8) and torch.equal(both[N * K:].view(torch.uint8).view(N, K // 2), wq)
    for wfmt, wbuf in ((st.W_PACKED4, wq), (st.W_INT8, w8), (st.W_INT8_AND_PACKED4, both)):
        Y3 = st.stamp_linear_fused(c, Xd, wbuf, wfmt, wsc, bd, ws, n_out=N).cpu().numpy().reshape(-1, N)
        err = H.rel_fro(Y3, ref["Y"])
        print(f"[{name}] one-call layer, output relative Frobenius error {err:.2e}")
        # (the tight bound presumes the oracle's codes; a code on a rounding boundary that fell the other way moves
        #  the output by a whole code step of its row)
        assert err <= (_fused_y_tol(cfg) if act_bad == 0 else Y_TOL)
    assert st.stamp_last_launch_count() > 0
    # the operand of the one-call layer's GEMM, code by code (routes that reorder it)
    mapped = check_fused_operand(st, c, cfg, Xd, ws, ref["q"], ref["x_scale"], label=name)
    assert mapped == (name in FUSED_ORDER_CASES), name
    assert st.stamp_last_device_status() == 0


ZP_CASES = {
    # full-depth Haar with ragged tiles, blockwise DCT and Walsh-Hadamard, the patch-grid Haar, no transform
    "zp_haar": gen.scaled(gen.config_llm_up(), B=2, L=512, K=384, N=392, k_hi=16),
    "zp_haar_fp32_blocks": gen.scaled(gen.config_tiny(), B=1, L=256, K=128, N=72, block=64, levels=3, k_hi=8),
    "zp_dct": gen.scaled(gen.config_llm_down(), B=1, L=512, K=256, N=136),
    "zp_wht": gen.scaled(gen.config_llm_down_wht(), B=1, L=256, K=128, N=64, block=64, k_hi=4),
    "zp_haar2d": gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=256, N=128, grid=32, levels=3, k_hi=16),
    "zp_skip_first": gen.scaled(gen.config_llm_up_skip1(), B=1, L=256, K=128, N=72, k_hi=8),
    "zp_identity": gen.scaled(gen.config_sweep(512, 2048), L=256, K=256, N=128, transform=gen.T_IDENTITY, k_hi=8),
}


@pytest.mark.parametrize("name", list(ZP_CASES))
def test_zero_point_stagewise_parity(st, oracle, name):
    """Zero-point activation codes (Sec. 2.1, first equation, min-max range) against the oracle.  The library
    stores codes and zero points offset by half the code range; the oracle keeps the unsigned ones."""
    import torch
    cfg = ZP_CASES[name]
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, zero_point=True)
    X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
    # a per-feature offset, so that rows (above all the low-pass ones) are far from symmetric about zero
    X = gen.round_to_bf16((X + 0.5 * np.abs(X).mean()).astype(np.float32)) if cfg.dtype == 1 else (X + 0.5).astype(np.float32)
    ref = oracle.stamp_linear(X, W, bias, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi,
                              grid_w=cfg.grid, asym=True)
    B, L, K, N = cfg.B, cfg.L, cfg.K, cfg.N
    M = B * L
    Xd, Wd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype)
    bd = torch.from_numpy(bias).cuda()
    ws = st.alloc_workspace(c, B, L, K, N)
    half = np.where((np.arange(M) % cfg.block_len) < cfg.k_hi, 128, 8).astype(np.int64)

    # scales, zero points, codes
    q_hi, q_lo, xbuf = st.stamp_quantize(c, Xd, ws)
    xs, zc = st.split_zero_points(xbuf)
    xs, zc = xs.cpu().numpy().reshape(-1), zc.cpu().numpy().reshape(-1).astype(np.int64)
    codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, B, L, K).cpu().numpy().reshape(-1, K).astype(np.int64)
    assert np.allclose(xs, ref["x_scale"], rtol=2 * _scale_rtol(cfg), atol=0)
    dz = zc + half - ref["x_zero"]
    # a zero point is a rounded quotient: within fp32 error of a tie it may come out one off, and the row's
    # codes move with it -- compare such rows through the centred codes c - zc = x_int - z
    # (same budget as for the codes: at most 1e-5 of the rows, rounded up to a whole row)
    assert np.abs(dz).max() <= 1 and np.count_nonzero(dz) <= _allowed(M), (np.abs(dz).max(), np.count_nonzero(dz))
    same = dz == 0
    bad, worst = H.code_mismatch((codes + half[:, None])[same], ref["q"][same].astype(np.int64))
    print(f"[{name}] zero-point code mismatches: {bad} of {codes.size} (max |diff| {worst}); rows with z off by one: "
          f"{np.count_nonzero(dz)}")
    assert worst <= 1 and bad <= _allowed(codes.size), (bad, worst, codes.size)
    centred = codes - zc[:, None]
    centred_ref = ref["q"].astype(np.int64) - ref["x_zero"].astype(np.int64)[:, None]
    assert np.abs(centred - centred_ref).max() <= 1
    assert codes.min() >= -128 and codes.max() <= 127 and np.all(np.abs(codes[half == 8]) <= 8)

    # integer GEMM on the oracle's codes in the stored (offset) form: the plain code product, bit-identical
    oc = (ref["q"].astype(np.int64) - half[:, None]).astype(np.int8)
    ozc = (ref["x_zero"].astype(np.int64) - half).astype(np.int32)
    oq_hi, oq_lo = H.pack_codes(oc, cfg.block_len, cfg.k_hi)
    oqh, oql = torch.from_numpy(oq_hi).cuda(), torch.from_numpy(oq_lo).cuda()
    ow8 = torch.from_numpy(ref["wq"]).cuda()
    acc = st.stamp_debug_gemm_i32(c, oqh, oql, ow8, st.W_INT8, B, L, K, N, ws).cpu().numpy()
    assert np.array_equal(acc, oracle.gemm_i32(oc, ref["wq"]))

    # de-quantized transformed-domain output with the zero-point term, from the oracle's codes, scales, zero points
    oxbuf = torch.empty((2, B, L), dtype=torch.float32, device="cuda")
    oxbuf[0].copy_(torch.from_numpy(ref["x_scale"]).reshape(B, L))
    oxbuf[1].view(torch.int32).copy_(torch.from_numpy(ozc).reshape(B, L))
    ows = torch.from_numpy(ref["w_scale"]).cuda()
    owq = torch.from_numpy(H.pack_nibbles(ref["wq"])).cuda()
    for wfmt, wbuf in ((st.W_PACKED4, owq), (st.W_INT8, ow8)):
        Yt = st.stamp_linear(c, oqh, oql, oxbuf, wbuf, wfmt, ows, B, L, K, N, ws).cpu().numpy().reshape(-1, N)
        assert H.rel_fro(Yt, ref["Yt"]) <= 1e-6

    # whole layer: chained calls and the one-call form
    wq, wsc = st.stamp_quantize_weights(c, Wd)
    w8 = st.stamp_prepare_weights(c, wq)
    Yt2 = st.stamp_linear(c, q_hi, q_lo, xbuf, wq, st.W_PACKED4, wsc, B, L, K, N, ws)
    Y2 = st.stamp_inverse(c, Yt2, bd, ws).cpu().numpy().reshape(-1, N)
    assert H.rel_fro(Y2, ref["Y"]) <= Y_TOL
    for wfmt, wbuf in ((st.W_PACKED4, wq), (st.W_INT8, w8)):
        Y3 = st.stamp_linear_fused(c, Xd, wbuf, wfmt, wsc, bd, ws).cpu().numpy().reshape(-1, N)
        assert H.rel_fro(Y3, ref["Y"]) <= _fused_y_tol(cfg)
    mapped = check_fused_operand(st, c, cfg, Xd, ws, ref["q"], ref["x_scale"], ref_zero=ref["x_zero"], label=name)
    assert mapped == (name == "zp_haar2d")
    assert st.stamp_last_device_status() == 0
    # what the zero point buys on these one-sided rows: closer to the unquantized product than symmetric codes
    plain = oracle.matmul_f64(X.reshape(-1, K), W) + bias[None, :]
    sym = _oracle_all(oracle, cfg, X, W, bias, want=("Y",))["Y"]
    assert H.rel_fro(Y3, plain) < H.rel_fro(sym, plain)


def test_zero_point_constant_and_zero_rows(st):
    """No transform, rows that are constant: scale 1, stored code -2^(b-1) everywhere, zero point -rne(value) - 2^(b-1)."""
    import torch
    c = st.make_config(st.T_IDENTITY, 0, 0, 2, zero_point=True)
    ws = st.alloc_workspace(c, 1, 4, 128, 8)
    X = torch.zeros((1, 4, 128), device="cuda")
    X[0, 1] = 3.0
    X[0, 3] = -2.0
    q_hi, q_lo, xbuf = st.stamp_quantize(c, X, ws)
    xs, zc = st.split_zero_points(xbuf)
    codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, 1, 4, 128).cpu().numpy().reshape(4, 128)
    assert torch.all(xs == 1.0)
    assert zc.cpu().numpy().reshape(-1).tolist() == [-128, -3 - 128, -8, 2 - 8]
    assert np.all(codes[:2] == -128) and np.all(codes[2:] == -8)


def test_transform_then_inverse_is_identity(st):
    """Quantizers off: L^T (L X) = X on the device (uses the activation as its own 'output')."""
    import torch
    cfg = gen.scaled(gen.config_llm_up(), B=1, L=2048, K=256, N=256)
    c = _cfg_struct(st, cfg)
    X = gen.make_activation(cfg)
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    T = st.stamp_debug_transform(c, H.to_device(X, cfg.dtype), ws)
    back = st.stamp_inverse(c, T, None, ws).cpu().numpy()
    assert np.max(np.abs(back - X)) <= 2e-6 * np.max(np.abs(X))
    # energy preservation on the device result
    e_t = float((T.double() ** 2).sum())
    e_x = float((X.astype(np.float64) ** 2).sum())
    assert abs(e_t - e_x) <= 1e-6 * e_x


def test_host_buffer_call_matches_device_call(st):
    """stamp_linear_fused_host = the same layer with the two copies enqueued around it."""
    import torch
    cfg = gen.scaled(gen.config_llm_up(), B=1, L=512, K=256, N=264)
    c = _cfg_struct(st, cfg)
    X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
    Xd, Wd, bd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype), torch.from_numpy(bias).cuda()
    wq, wsc = st.stamp_quantize_weights(c, Wd)
    w8 = st.stamp_prepare_weights(c, wq)
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    want = st.stamp_linear_fused(c, Xd, w8, st.W_INT8, wsc, bd, ws, out_dtype=torch.bfloat16)
    X_host = Xd.cpu().pin_memory()
    Y_host = torch.empty((cfg.B, cfg.L, cfg.N), dtype=torch.bfloat16).pin_memory()
    ws_h = torch.empty(st.stamp_workspace_bytes_host(c, cfg.B, cfg.L, cfg.K, cfg.N, st.BF16, st.BF16), dtype=torch.uint8,
                       device="cuda")
    st.stamp_linear_fused_host(c, X_host, w8, st.W_INT8, wsc, bd, Y_host, ws_h)
    torch.cuda.synchronize()
    assert torch.equal(Y_host, want.cpu())
    assert st.stamp_last_device_status() == 0


def test_edge_cases(st, oracle):
    """Zero activations (scale 1, codes 0), k_hi = 0 and k_hi = block."""
    import torch
    base = gen.scaled(gen.config_tiny(), L=128, K=128, N=64, levels=0)
    for k_hi in (0, 128):
        cfg = gen.scaled(base, k_hi=k_hi)
        c = _cfg_struct(st, cfg)
        X, W = gen.make_activation(cfg), gen.make_weight(cfg)
        ref = _oracle_all(oracle, cfg, X, W, want=("q", "Y"))
        ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
        Xd, Wd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype)
        q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
        codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, cfg.B, cfg.L, cfg.K).cpu().numpy().reshape(-1, cfg.K)
        bad, worst = H.code_mismatch(codes, ref["q"])
        assert worst <= 1 and bad <= 1
        wq, wsc = st.stamp_quantize_weights(c, Wd)
        Y = st.stamp_linear_fused(c, Xd, wq, st.W_PACKED4, wsc, None, ws).cpu().numpy().reshape(-1, cfg.N)
        assert H.rel_fro(Y, ref["Y"]) <= Y_TOL
    cfg = base
    c = _cfg_struct(st, cfg)
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    Xz = torch.zeros((1, cfg.L, cfg.K), device="cuda")
    q_hi, q_lo, xs = st.stamp_quantize(c, Xz, ws)
    assert torch.all(xs == 1.0) and not q_hi.any() and not q_lo.any()


def test_zero_activations_give_the_bias_on_every_route(st):
    """All-zero input: every row has scale 1 (range 0) and codes 0 (stored -2^(b-1) with zero points), so the
    layer returns the bias exactly -- on the fused Haar route (with rows above the GEMM tiles), the fused 2-D
    route with symmetric and with zero-point codes, the tensor-core DCT route and the general zero-point route."""
    import torch
    routes = {
        "haar_tiled": (gen.scaled(gen.config_llm_up(), B=1, L=1024, K=256, N=136), False),
        "haar2d_patch": (gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=256, N=136, grid=32, k_hi=16), False),
        "haar2d_patch_zp": (gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=256, N=136, grid=32, k_hi=16), True),
        "dct_tensor": (gen.scaled(gen.config_llm_down(), B=1, L=512, K=256, N=192), False),
        "haar_zp_general": (gen.scaled(gen.config_llm_up(), B=1, L=512, K=256, N=136), True),
    }
    for name, (cfg, zp) in routes.items():
        c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, zero_point=zp)
        W, bias = gen.make_weight(cfg), gen.make_bias(cfg)
        wq, wsc = st.stamp_quantize_weights(c, H.to_device(W, cfg.dtype))
        bd = torch.from_numpy(bias).cuda()
        ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
        Xz = torch.zeros((cfg.B, cfg.L, cfg.K), dtype=torch.bfloat16, device="cuda")
        Y = st.stamp_linear_fused(c, Xz, wq, st.W_PACKED4, wsc, bd, ws)
        assert torch.equal(Y.reshape(-1, cfg.N), bd.expand(cfg.M, cfg.N)), name
        assert st.stamp_last_device_status() == 0


def test_fused_call_can_be_captured_in_a_cuda_graph(st):
    """The one-call layer makes no synchronising call and allocates nothing, so a stream capture records it
    (dependent launches included) and the replayed graph gives the same output as the direct call."""
    import torch
    for cfg in (gen.scaled(gen.config_llm_up(), B=1, L=1024, K=256, N=264),
                gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=256, N=136, grid=32, k_hi=16)):
        c = _cfg_struct(st, cfg)
        X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
        Xd, Wd, bd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype), torch.from_numpy(bias).cuda()
        wq, wsc = st.stamp_quantize_weights(c, Wd)
        w8 = st.stamp_prepare_weights(c, wq)
        ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
        want = st.stamp_linear_fused(c, Xd, w8, st.W_INT8, wsc, bd, ws, out_dtype=torch.bfloat16).clone()
        out = torch.zeros_like(want)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                st.stamp_linear_fused(c, Xd, w8, st.W_INT8, wsc, bd, ws, out=out)
        for _ in range(3):
            out.zero_()
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, want)
        assert st.stamp_last_device_status() == 0



def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable(st):
    """Failure detection without a fault: a kernel waits on a barrier nobody completes; its bounded wait gives up
    after about a millisecond, the status word reads time-out exactly once, and the library keeps working."""
    import torch
    assert st.stamp_last_device_status() == 0
    st.stamp_debug_expire_wait(2_000_000)
    assert st.stamp_last_device_status() == 5          # STAMP_ERR_TIMEOUT ...
    assert "wait" in st.status_string(5)
    assert st.stamp_last_device_status() == 0          # ... reported once, then cleared
    # the context is intact: a layer call still gives the right answer
    cfg = gen.scaled(gen.config_llm_up(), B=1, L=512, K=256, N=136)
    c = _cfg_struct(st, cfg)
    W, bias = gen.make_weight(cfg), gen.make_bias(cfg)
    wq, wsc = st.stamp_quantize_weights(c, H.to_device(W, cfg.dtype))
    bd = torch.from_numpy(bias).cuda()
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    Xz = torch.zeros((cfg.B, cfg.L, cfg.K), dtype=torch.bfloat16, device="cuda")
    Y = st.stamp_linear_fused(c, Xz, wq, st.W_PACKED4, wsc, bd, ws)
    assert torch.equal(Y.reshape(-1, cfg.N), bd.expand(cfg.M, cfg.N))
    assert st.stamp_last_device_status() == 0


@pytest.mark.parametrize("name", ["tiny", "ragged", "blocked", "dct_blocks", "haar2d_oblong", "wide_k8192"])
def test_guard_bands_around_workspace_and_output_stay_intact(st, name):
    """Canaries: the workspace and the output are carved out of larger allocations whose margins hold a pattern.  After
    the public calls have run on ragged shapes (tiles that hang over the edge in every direction) the margins must
    be untouched -- no kernel writes outside the buffers it was given."""
    import torch
    cfg = CASES[name]
    c = _cfg_struct(st, cfg)
    B, L, K, N = cfg.B, cfg.L, cfg.K, cfg.N
    X, W, bias = gen.make_activation(cfg), gen.make_weight(cfg), gen.make_bias(cfg)
    Xd, Wd, bd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype), torch.from_numpy(bias).cuda()
    guard = 1 << 16
    need = st.stamp_workspace_bytes(c, B, L, K, N)
    raw = torch.full((need + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = raw[guard:guard + need]
    assert ws.data_ptr() % 256 == 0
    for out_dtype, esz in ((torch.float32, 4), (torch.bfloat16, 2)):
        ybytes = B * L * N * esz
        yraw = torch.full((ybytes + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
        Y = yraw[guard:guard + ybytes].view(out_dtype).reshape(B, L, N)
        wq, wsc = st.stamp_quantize_weights(c, Wd)
        q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
        Yt = st.stamp_linear(c, q_hi, q_lo, xs, wq, st.W_PACKED4, wsc, B, L, K, N, ws)
        st.stamp_inverse(c, Yt, bd, ws, out=Y)
        st.stamp_linear_fused(c, Xd, wq, st.W_PACKED4, wsc, bd, ws, out=Y)
        st.stamp_debug_transform(c, Xd, ws)
        torch.cuda.synchronize()
        assert bool((raw[:guard] == 0xA5).all()) and bool((raw[guard + need:] == 0xA5).all()), "workspace overrun"
        assert bool((yraw[:guard] == 0x5A).all()) and bool((yraw[guard + ybytes:] == 0x5A).all()), "output overrun"
    assert st.stamp_last_device_status() == 0


GROUP_CASES = {
    # the LVM table's setting on the DiT stand-in: 3-level 2-D Haar, 64 low-pass tokens at 8 bits, blocks of 64 features
    "g64_haar2d": (gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=256, N=136, grid=32, k_hi=16), 64),
    # 1-D Haar with ragged tiles; a larger block; no transform at all (plain per-block W4A4)
    "g64_haar": (gen.scaled(gen.config_llm_up(), B=2, L=512, K=384, N=392, k_hi=16), 64),
    "g128_haar": (gen.scaled(gen.config_llm_up(), B=1, L=256, K=384, N=72, k_hi=8), 128),
    "g64_identity": (gen.scaled(gen.config_sweep(512, 2048), L=256, K=256, N=128, transform=gen.T_IDENTITY, k_hi=0), 64),
    # more than 128 groups per row (the tensor-core product's scale table holds 128): the CUDA-core product
    "g64_long_k": (gen.scaled(gen.config_llm_up(), B=1, L=128, K=8320, N=64, k_hi=8), 64),
    # blocks of 256 features: a ring stage of the tensor-core product is part of one group
    "g256_haar": (gen.scaled(gen.config_llm_up(), B=1, L=512, K=1024, N=256, k_hi=8), 256),
    # the DiT projection at full size (all 1152 output channels on the GPU, 64 of them through the oracle)
    "g64_dit_full": (gen.config_dit_proj_2d(), 64),
}


@pytest.mark.parametrize("name", list(GROUP_CASES))
def test_group_scale_parity(st, oracle, name):
    """Per-block scales of 64 (128) features for activations and weights against the oracle: weight scales equal,
    activation scales within the tolerance of T, codes within the tie budget, the product of the oracle's codes and
    scales within fp32 rounding, the one-call layer within the output tolerance."""
    import torch
    cfg, group = GROUP_CASES[name]
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, group=group)
    B, L, K, N, M = cfg.B, cfg.L, cfg.K, cfg.N, cfg.M
    X, bias = gen.make_activation(cfg), gen.make_bias(cfg)
    cols = np.arange(N) if N <= 512 else np.sort(np.random.default_rng(7).choice(N, size=64, replace=False))
    W = gen.make_weight(cfg)
    ref = oracle.stamp_linear(X, W[cols], bias[cols], transform=cfg.transform, block=cfg.block, levels=cfg.levels,
                              k_hi=cfg.k_hi, grid_w=cfg.grid, group=group, want=("x_scale", "q", "w_scale", "wq", "Yt", "Y"))
    Xd, Wd, bd = H.to_device(X, cfg.dtype), H.to_device(W, cfg.dtype), torch.from_numpy(bias).cuda()
    ws = st.alloc_workspace(c, B, L, K, N)
    # weights
    wq, wsc = st.stamp_quantize_weights(c, Wd)
    assert wsc.shape == (N, K // group)
    assert np.array_equal(wsc.cpu().numpy()[cols], ref["w_scale"])
    w8 = st.stamp_prepare_weights(c, wq)
    bad, worst = H.code_mismatch(w8.cpu().numpy()[cols], ref["wq"])
    assert worst <= 1 and bad <= _allowed(ref["wq"].size), (bad, worst)
    # activations
    q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
    assert xs.shape == (B, L, K // group)
    assert np.allclose(xs.cpu().numpy().reshape(M, -1), ref["x_scale"], rtol=_scale_rtol(cfg), atol=0)
    codes = st.stamp_debug_unpack_codes(c, q_hi, q_lo, B, L, K).cpu().numpy().reshape(M, K)
    bad, worst = H.code_mismatch(codes, ref["q"])
    print(f"[{name}] group-scaled activation code mismatches: {bad} of {codes.size} (max |diff| {worst})")
    assert worst <= 1 and bad <= _allowed(codes.size), (bad, worst)
    # product fed the oracle's codes and scales (all output channels of the oracle's subset)
    if N <= 512:
        oq_hi, oq_lo = H.pack_codes(ref["q"], cfg.block_len, cfg.k_hi)
        Yt = st.stamp_linear(c, torch.from_numpy(oq_hi).cuda(), torch.from_numpy(oq_lo).cuda(),
                             torch.from_numpy(ref["x_scale"]).cuda().reshape(B, L, -1),
                             torch.from_numpy(H.pack_nibbles(ref["wq"])).cuda(), st.W_PACKED4,
                             torch.from_numpy(ref["w_scale"]).cuda(), B, L, K, N, ws).cpu().numpy().reshape(M, N)
        assert H.rel_fro(Yt, ref["Yt"]) <= 1e-6
    # the layer: chained calls and the one-call form
    Yt2 = st.stamp_linear(c, q_hi, q_lo, xs, wq, st.W_PACKED4, wsc, B, L, K, N, ws)
    Y2 = st.stamp_inverse(c, Yt2, bd, ws).cpu().numpy().reshape(M, N)[:, cols]
    Y3 = st.stamp_linear_fused(c, Xd, w8, st.W_INT8, wsc, bd, ws).cpu().numpy().reshape(M, N)[:, cols]
    e2, e3 = H.rel_fro(Y2, ref["Y"]), H.rel_fro(Y3, ref["Y"])
    print(f"[{name}] output relative Frobenius error: chained {e2:.2e}, one call {e3:.2e}")
    assert e2 <= (Y_TOL_HAAR if bad == 0 else Y_TOL) and e3 <= (Y_TOL_HAAR if bad == 0 else Y_TOL)
    assert st.stamp_last_device_status() == 0


def test_group_scale_arguments_are_checked(st):
    import ctypes
    lib = st.lib()
    out = ctypes.c_size_t(0)
    ok = st.make_config(st.T_HAAR, 0, 0, 16, group=64)
    assert lib.stamp_workspace_bytes(ctypes.byref(ok), 1, 256, 256, 64, ctypes.byref(out)) == 0
    for bad_group in (48, 96, 192):                      # not 64 * 2^i, or not a divisor of K
        c = st.make_config(st.T_HAAR, 0, 0, 16, group=bad_group)
        assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 256, 384, 64, ctypes.byref(out)) == 2
    c = st.make_config(st.T_HAAR, 0, 0, 16, group=64, zero_point=True)
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 256, 256, 64, ctypes.byref(out)) == 2
    c = st.make_config(st.T_HAAR, 0, 0, 16, group=64)
    c.w_gran = st.G_PER_CHANNEL                          # group set but the granularity fields disagree
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 256, 256, 64, ctypes.byref(out)) == 1


def test_kv_cache_round_trip(st, oracle):
    """STaMP on a KV cache (LLM table: KV at 4 bits, 64 transformed tokens at 8; scales per token and head): the
    cache [B, H, L, 128] is quantized as B * H sequences of 128 features, read back with stamp_dequantize and
    stamp_inverse, and compared with the oracle's L^T Q(L X); it is closer to the cache than plain 4-bit codes."""
    import torch
    B, Hh, L, Dh = 2, 4, 1024, 128
    cfg = gen.scaled(gen.config_llm_up(), B=B * Hh, L=L, K=Dh, N=Dh, k_hi=64, first_token_gain=1.0, recipe="ar1")
    X = gen.make_activation(cfg)                                  # [B * H, L, 128], correlated along tokens
    Lm = oracle.transform_matrix(cfg.transform, L, 0)
    T = oracle.apply_dense(Lm, X.astype(np.float64))
    bits = oracle.bit_map(L, L, cfg.k_hi)
    q, s = oracle.quantize_rows(T.reshape(-1, Dh), bits)
    Tq = (q * s.astype(np.float64)[:, None]).reshape(B * Hh, L, Dh)
    ref = oracle.apply_dense(Lm, Tq, transpose=True)
    c = st.make_config(cfg.transform, 0, 0, cfg.k_hi)
    ws = st.alloc_workspace(c, B * Hh, L, Dh, Dh)
    Xd = H.to_device(X, cfg.dtype)
    q_hi, q_lo, xs = st.stamp_quantize(c, Xd, ws)
    Td = st.stamp_dequantize(c, q_hi, q_lo, xs, B * Hh, L, Dh)
    assert H.rel_fro(Td.cpu().numpy(), Tq) <= 1e-6
    back = st.stamp_inverse(c, Td, None, ws).cpu().numpy()
    assert H.rel_fro(back, ref) <= 1e-6
    # against the cache itself: STaMP 8/4 beats plain 4-bit per-token codes on these correlated sequences
    q4, s4 = oracle.quantize_rows(X.reshape(-1, Dh).astype(np.float64), np.array([4], dtype=np.int32))
    plain4 = (q4 * s4.astype(np.float64)[:, None]).reshape(X.shape)
    assert H.rel_fro(back, X) < H.rel_fro(plain4, X)
    assert st.stamp_last_device_status() == 0
