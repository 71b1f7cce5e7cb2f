"""Seeded synthetic inputs for the STaMP linear layer.

This module only draws random activations and weights with the statistics the
paper describes for LLM / LVM activations (strong local correlation along the
token axis, a few outlier channels, a massive first token, a 2-D patch grid
flattened in raster order).  It holds none of the method's arithmetic: no
sequence transform, no quantizer, no matmul.  Both the CPU oracle's tests and
the CUDA path's tests draw their inputs from here so that they see the same
bytes.

All arrays are returned as float32 numpy arrays whose values are already
rounded to the storage dtype of the configuration (bf16 or fp32), so the exact
same real numbers reach the oracle (upcast to fp64) and the GPU (as bf16 bits).
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
from scipy.signal import lfilter

# transform identifiers (values match the public C header's stamp_transform)
T_IDENTITY, T_HAAR, T_DCT2, T_HAAR2D, T_WHT, T_HAAR_SKIP1 = 0, 1, 2, 3, 4, 5
# storage dtypes (values match stamp_dtype)
F32, BF16 = 0, 1


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    """One STaMP linear-layer workload: shapes, transform and bit allocation."""
    name: str
    B: int                 # batch items (independent sequences)
    L: int                 # tokens per sequence (paper: s)
    K: int                 # input features (paper: d)
    N: int                 # output features
    dtype: int             # F32 or BF16 storage of X and W
    transform: int         # T_HAAR / T_DCT2 / T_IDENTITY
    block: int             # tokens per transform block (0 => whole sequence)
    levels: int            # Haar levels (0 => full depth)
    k_hi: int              # first k_hi transformed tokens of each block at 8 bits
    seed: int
    recipe: str            # which generator below
    rho: float = 0.9
    outlier_frac: float = 0.0
    outlier_count: int = 0     # exact count (overrides frac when > 0)
    outlier_gain: float = 1.0
    first_token_gain: float = 1.0
    w_std: float = 0.02
    grid: int = 0              # patch-grid side for the GRF recipe
    length_scale: float = 8.0
    zero_point: bool = False   # activation codes with a per-token zero point (min-max range)

    @property
    def M(self) -> int:
        return self.B * self.L

    @property
    def block_len(self) -> int:
        return self.block if self.block else self.L


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    out = ((bits + bias) >> np.uint32(16)) << np.uint32(16)
    return out.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are exactly representable in bf16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _store(x: np.ndarray, dtype: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_to_bf16(x) if dtype == BF16 else x


def ar1(rng: np.random.Generator, B: int, L: int, K: int, rho: float) -> np.ndarray:
    """Stationary AR(1) along the token axis, independent per channel and batch item:
    x_0 = e_0 / sqrt(1 - rho^2), x_t = rho x_{t-1} + e_t, e ~ N(0, 1)."""
    out = np.empty((B, L, K), dtype=np.float32)
    for b in range(B):
        e = rng.standard_normal((L, K), dtype=np.float32)
        e[0] /= np.float32(np.sqrt(1.0 - rho * rho))
        out[b] = lfilter([1.0], [1.0, -rho], e.astype(np.float64), axis=0).astype(np.float32)
    return out


def gaussian_random_field(rng: np.random.Generator, B: int, grid: int, K: int,
                          length_scale: float) -> np.ndarray:
    """Per channel: white noise on a grid x grid patch lattice, smoothed by a periodic
    Gaussian kernel (sigma = length_scale patches, applied in the FFT domain),
    renormalised to unit variance, flattened in raster order to grid*grid tokens."""
    f = np.fft.fftfreq(grid)
    g = np.exp(-2.0 * (np.pi * length_scale) ** 2 * (f[:, None] ** 2 + f[None, :] ** 2))
    out = np.empty((B, grid * grid, K), dtype=np.float32)
    for b in range(B):
        chunk = 128
        for c0 in range(0, K, chunk):
            c1 = min(K, c0 + chunk)
            w = rng.standard_normal((c1 - c0, grid, grid))
            s = np.fft.ifft2(np.fft.fft2(w, axes=(1, 2)) * g[None], axes=(1, 2)).real
            s /= s.std(axis=(1, 2), keepdims=True)
            out[b, :, c0:c1] = s.reshape(c1 - c0, grid * grid).T.astype(np.float32)
    return out


def _apply_outliers(rng: np.random.Generator, x: np.ndarray, cfg: LayerConfig) -> None:
    K = x.shape[-1]
    n = cfg.outlier_count if cfg.outlier_count > 0 else int(round(cfg.outlier_frac * K))
    if n > 0:
        ch = rng.choice(K, size=n, replace=False)
        x[..., ch] *= np.float32(cfg.outlier_gain)


def make_activation(cfg: LayerConfig) -> np.ndarray:
    """X [B, L, K] float32 (values rounded to cfg.dtype)."""
    rng = np.random.default_rng(cfg.seed)
    if cfg.recipe in ("ar1", "ar1_first_token"):
        x = ar1(rng, cfg.B, cfg.L, cfg.K, cfg.rho)
        _apply_outliers(rng, x, cfg)
        if cfg.recipe == "ar1_first_token":
            x[:, 0, :] *= np.float32(cfg.first_token_gain)
    elif cfg.recipe == "grf":
        assert cfg.grid * cfg.grid == cfg.L
        x = gaussian_random_field(rng, cfg.B, cfg.grid, cfg.K, cfg.length_scale)
        _apply_outliers(rng, x, cfg)
    elif cfg.recipe == "ar1_student":
        x = ar1(rng, cfg.B, cfg.L, cfg.K, cfg.rho)
        scale = np.abs(rng.standard_t(3.0, size=cfg.K)).astype(np.float32)
        x *= scale[None, None, :]
    elif cfg.recipe == "white":
        x = rng.standard_normal((cfg.B, cfg.L, cfg.K), dtype=np.float32)
    else:
        raise ValueError(f"unknown recipe {cfg.recipe!r}")
    return _store(x, cfg.dtype)


def make_weight(cfg: LayerConfig, rows: Optional[np.ndarray] = None) -> np.ndarray:
    """W [N, K] float32 ~ N(0, w_std^2) (values rounded to cfg.dtype).

    `rows` selects a subset of output channels; the draw is made row by row from a
    per-row child stream so that a subset equals the same rows of the full matrix."""
    idx = np.arange(cfg.N) if rows is None else np.asarray(rows)
    w = np.empty((len(idx), cfg.K), dtype=np.float32)
    # one generator per block of 256 rows keeps full-matrix generation fast while any
    # subset of rows still reproduces the full matrix's values
    blk = 256
    cache_id, cache = -1, None
    for j, n in enumerate(idx):
        bid = int(n) // blk
        if bid != cache_id:
            r = np.random.default_rng([cfg.seed, 7919, bid])
            cache = r.standard_normal((blk, cfg.K), dtype=np.float32)
            cache_id = bid
        w[j] = cache[int(n) % blk]
    w *= np.float32(cfg.w_std)
    return _store(w, cfg.dtype)


def make_bias(cfg: LayerConfig) -> np.ndarray:
    rng = np.random.default_rng([cfg.seed, 104729])
    return rng.standard_normal(cfg.N).astype(np.float32) * np.float32(0.1)


# ----------------------------------------------------------------------------------
# The named workloads
# ----------------------------------------------------------------------------------

def config_tiny() -> LayerConfig:
    return LayerConfig("tiny", B=1, L=64, K=256, N=256, dtype=F32, transform=T_HAAR, block=0,
                       levels=3, k_hi=8, seed=0, recipe="ar1", rho=0.9, outlier_count=4,
                       outlier_gain=20.0, w_std=1.0 / 16.0)


def config_llm_up() -> LayerConfig:
    return LayerConfig("llm_mlp_up", B=1, L=2048, K=4096, N=11008, dtype=BF16, transform=T_HAAR,
                       block=0, levels=0, k_hi=64, seed=1, recipe="ar1_first_token", rho=0.95,
                       outlier_frac=0.01, outlier_gain=50.0, first_token_gain=100.0, w_std=0.02)


def config_dit_proj() -> LayerConfig:
    return LayerConfig("dit_attn_proj", B=2, L=4096, K=1152, N=1152, dtype=BF16, transform=T_HAAR,
                       block=0, levels=6, k_hi=64, seed=2, recipe="grf", outlier_frac=0.02,
                       outlier_gain=30.0, w_std=0.03, grid=64, length_scale=8.0)


def config_llm_down_wht() -> LayerConfig:
    """The down-projection workload with the Walsh-Hadamard transform in place of the DCT (same blocks)."""
    return dataclasses.replace(config_llm_down(), name="llm_down_proj_wht", transform=T_WHT)


def config_llm_up_zp() -> LayerConfig:
    """The MLP up-projection workload with zero-point (asymmetric, min-max) activation codes."""
    return dataclasses.replace(config_llm_up(), name="llm_mlp_up_zp", zero_point=True)


def config_llm_up_skip1() -> LayerConfig:
    """The MLP up-projection workload as the paper runs LLMs: the massive first token is left out of the sequence
    transform (and is one of the 8-bit rows)."""
    return dataclasses.replace(config_llm_up(), name="llm_mlp_up_skip1", transform=T_HAAR_SKIP1)


def config_dit_proj_2d() -> LayerConfig:
    """The DiT projection with the paper's own LVM transform: 3-level 2-D Haar over the 64 x 64 patch grid,
    whose 64 low-pass tokens are the 8-bit ones."""
    return dataclasses.replace(config_dit_proj(), name="dit_attn_proj_2d", transform=T_HAAR2D, levels=3)


def config_dit_proj_2d_zp() -> LayerConfig:
    """The paper's LVM activation setting in full: 3-level 2-D Haar over the patch grid, 64 low-pass tokens at
    8 bits, zero-point (asymmetric, min-max) codes."""
    return dataclasses.replace(config_dit_proj_2d(), name="dit_attn_proj_2d_zp", zero_point=True)


def config_llm_down() -> LayerConfig:
    return LayerConfig("llm_down_proj", B=4, L=4096, K=14336, N=4096, dtype=BF16, transform=T_DCT2,
                       block=256, levels=0, k_hi=16, seed=3, recipe="ar1_student", rho=0.9,
                       w_std=0.01)


SWEEP_L = (512, 2048, 8192, 32768)
SWEEP_D = (2048, 4096, 8192)


def config_sweep(L: int, D: int, levels: int = 0) -> LayerConfig:
    idx = SWEEP_L.index(L) * len(SWEEP_D) + SWEEP_D.index(D)
    return LayerConfig(f"sweep_L{L}_D{D}", B=1, L=L, K=D, N=D, dtype=BF16, transform=T_HAAR,
                       block=0, levels=levels, k_hi=L // 32, seed=100 + idx, recipe="ar1", rho=0.9,
                       outlier_frac=0.01, outlier_gain=50.0, w_std=0.02)


def named_configs() -> dict:
    return {c.name: c for c in (config_tiny(), config_llm_up(), config_dit_proj(), config_llm_down(), config_dit_proj_2d(), config_llm_down_wht(),
                                config_llm_up_zp(), config_dit_proj_2d_zp(), config_llm_up_skip1())}


def scaled(cfg: LayerConfig, **kw) -> LayerConfig:
    """A copy of cfg with some fields replaced (used for reduced-size parity cases)."""
    return dataclasses.replace(cfg, **kw)
