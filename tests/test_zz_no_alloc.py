"""The allocation-free inverse call (stamp_inverse_noalloc) against the ordinary stamp_inverse.

Some users of the library cannot allocate device memory where they call it -- an operator
plug-in inside a serving loop whose framework owns all device memory, or a callback where a
cudaMalloc would stall the device -- and have no workspace to pass.  For them the library
carries its own few MB of scratch per GPU.  This file checks, through the C ABI, that the
variant gives the same output as the call with a caller-owned workspace, on two calls in a row
with different inputs (the shared scratch keeps the first call's partial sums when the second
one starts), and that a problem whose partial sums exceed the built-in array is refused.

The file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2510_26771_b200 import inputs as gen
from tests import helpers as H


@pytest.mark.gpu
def test_noalloc_inverse_matches_workspace_inverse_twice():
    import torch
    from paper_2510_26771_b200 import binding as st
    assert torch.cuda.is_available()
    st.lib()
    # full-depth Haar over 2048 tokens: three coarse-to-fine passes, so both scratch regions are used
    cfg = gen.scaled(gen.config_llm_up(), B=2, L=2048, K=128, N=264)
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi)
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    g = torch.Generator(device="cuda").manual_seed(5)
    bias = torch.randn(cfg.N, device="cuda", generator=g)
    for call in range(2):
        Yt = torch.randn((cfg.B, cfg.L, cfg.N), device="cuda", generator=g) * (1.0 + 9.0 * call)
        for out_dtype in (torch.float32, torch.bfloat16):
            want = st.stamp_inverse(c, Yt, bias, ws, out_dtype=out_dtype)
            got = st.stamp_inverse_noalloc(c, Yt, bias, out_dtype=out_dtype)
            assert st.stamp_last_launch_count() == 3
            torch.cuda.synchronize()
            assert H.rel_fro(got.float().cpu().numpy(), want.float().cpu().numpy()) <= 1e-6
    assert st.stamp_last_device_status() == 0


@pytest.mark.gpu
def test_noalloc_inverse_other_transforms_and_the_oracle():
    """The other layouts of the built-in scratch: a DCT block (the dense matrix lives there), a two-pass Haar
    inverse (one region of partial sums), the 2-D Haar transform (no scratch at all) -- each against the call
    with a caller-owned workspace, and one of them against the oracle's L^T Yt + bias as well."""
    import torch
    from oracle import stamp_oracle as orc
    from paper_2510_26771_b200 import binding as st
    st.lib()
    orc.build()
    g = torch.Generator(device="cuda").manual_seed(11)
    cases = {
        "dct_block_256": gen.scaled(gen.config_llm_down(), B=1, L=512, K=128, N=136),
        "haar_8_levels": gen.scaled(gen.config_llm_up(), B=2, L=256, K=128, N=72),
        "haar2d": gen.scaled(gen.config_dit_proj_2d(), B=1, L=1024, K=128, N=72, grid=32, k_hi=16),
    }
    for name, cfg in cases.items():
        c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid)
        ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
        bias = torch.randn(cfg.N, device="cuda", generator=g)
        for call in range(2):
            Yt = torch.randn((cfg.B, cfg.L, cfg.N), device="cuda", generator=g)
            want = st.stamp_inverse(c, Yt, bias, ws)
            got = st.stamp_inverse_noalloc(c, Yt, bias)
            torch.cuda.synchronize()
            assert H.rel_fro(got.cpu().numpy(), want.cpu().numpy()) <= 1e-6, name
        Lm = orc.transform_matrix(cfg.transform, cfg.block_len, cfg.levels, grid_w=cfg.grid)
        ref = orc.apply_dense(Lm, Yt.double().cpu().numpy(), transpose=True) + bias.double().cpu().numpy()
        assert H.rel_fro(got.cpu().numpy(), ref) <= (1e-5 if cfg.transform == gen.T_DCT2 else 1e-6), name
    assert st.stamp_last_device_status() == 0


def test_noalloc_inverse_refuses_oversized_problems():
    """Host-side: the size check comes before any CUDA call, so it needs no GPU."""
    from paper_2510_26771_b200 import build as stamp_build
    stamp_build.build()
    from paper_2510_26771_b200 import binding as st
    lib = st.lib()
    c = st.make_config(st.T_HAAR, 0, 0, 64)
    fake = ctypes.c_void_p(4096)  # never dereferenced: the call is refused first
    # (32768/32 + 32768/1024) tokens x 8192 channels x 4 bytes = 33 MiB of partial sums > 4 MiB
    rc = lib.stamp_inverse_noalloc(ctypes.byref(c), fake, None, 1, 32768, 8192, fake, 0, None)
    assert rc == 6 and "scratch" in st.status_string(rc)
    assert lib.stamp_inverse_noalloc(ctypes.byref(c), None, None, 1, 2048, 256, fake, 0, None) == 1
    # a DCT block of 2048 tokens: its dense matrix alone is 16 MiB
    d = st.make_config(st.T_DCT2, 2048, 0, 16)
    assert lib.stamp_inverse_noalloc(ctypes.byref(d), fake, None, 1, 2048, 256, fake, 0, None) == 6
    d = st.make_config(st.T_DCT2, 1024, 0, 16)                       # 4 MiB: fits exactly (refused only for the null pointer)
    assert lib.stamp_inverse_noalloc(ctypes.byref(d), None, None, 1, 1024, 256, fake, 0, None) == 1
    e = st.make_config(st.T_HAAR_SKIP1, 0, 0, 16)
    assert lib.stamp_inverse_noalloc(ctypes.byref(e), fake, None, 1, 2048, 256, fake, 0, None) == 2
