"""The seeded generators: determinism, storage rounding, and the stated statistics."""
import numpy as np

from paper_2510_26771_b200 import inputs as gen


def test_deterministic_and_bf16_exact():
    cfg = gen.scaled(gen.config_llm_up(), L=128, K=256, N=64)
    a, b = gen.make_activation(cfg), gen.make_activation(cfg)
    assert np.array_equal(a, b) and a.shape == (1, 128, 256)
    assert np.array_equal(gen.round_to_bf16(a), a)            # already bf16-representable
    bits = gen.bf16_bits(a)
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(back, a)


def test_round_to_bf16_ties_to_even():
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -1.0 - 2 ** -8], dtype=np.float32)
    assert gen.round_to_bf16(x).tolist() == [1.0, 1.0 + 2 ** -6, 1.0, -1.0]


def test_weight_subset_matches_full():
    cfg = gen.scaled(gen.config_llm_up(), K=128, N=700)
    full = gen.make_weight(cfg)
    rows = np.array([0, 5, 255, 256, 699])
    assert np.array_equal(gen.make_weight(cfg, rows), full[rows])
    assert abs(full.std() - cfg.w_std) < 0.1 * cfg.w_std


def test_tiny_config_statistics():
    cfg = gen.config_tiny()
    x = gen.make_activation(cfg)
    assert x.shape == (1, 64, 256) and x.dtype == np.float32
    ch_rms = np.sqrt((x[0].astype(np.float64) ** 2).mean(axis=0))
    assert (ch_rms > 8 * np.median(ch_rms)).sum() == 4            # exactly 4 outlier channels (x20)


def test_first_token_and_correlation():
    cfg = gen.scaled(gen.config_llm_up(), L=512, K=256)
    x = gen.make_activation(cfg)[0].astype(np.float64)
    assert np.abs(x[0]).mean() > 20 * np.abs(x[1:]).mean()          # massive first token
    body = x[1:]
    r = (body[1:] * body[:-1]).sum() / (body[1:] ** 2).sum()
    assert 0.9 < r < 0.99                                           # AR(1), rho = 0.95


def test_grf_is_spatially_smooth():
    cfg = gen.scaled(gen.config_dit_proj(), B=1, K=16, N=16)
    x = gen.make_activation(cfg)[0].astype(np.float64).reshape(64, 64, 16)
    horiz = (x[:, 1:] * x[:, :-1]).mean() / (x ** 2).mean()
    vert = (x[1:] * x[:-1]).mean() / (x ** 2).mean()
    assert horiz > 0.95 and vert > 0.95
