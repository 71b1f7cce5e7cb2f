// Debug export of the fused route's GEMM operand: the transform+quantize kernels of the one-call layer write
// their codes in the row order the GEMM's fused inverse epilogue consumes (tile order for the 1-D Haar chain,
// patch order for the 2-D Haar transform).  These kernels map every LOGICAL transformed row back to where that
// route stored it and copy its codes (and the per-row factor the epilogue multiplies with), so that the codes
// of the timed route can be compared one by one with a reference in logical order.  The index arithmetic here
// is written from the layout's definition, independently of the kernels that produce and consume the operand.
#pragma once
#include "common.cuh"

namespace stamp {

// 1-D Haar, `levels` levels over blocks of n tokens, tile order.  Logical row i of a block is the
// approximation value a_levels[i] for i < n >> levels, else the detail d_j[i - (n >> j)] of the level j with
// n >> j <= i < n >> (j - 1).  Rows of levels above 8 live in the table that follows the M tile rows, in
// logical order (they are the first n / 256 logical rows of a block).  Inside the 256-row tile that holds the
// original tokens [256 t, 256 t + 256): the details of levels 1..5 of 32-token chunk c sit at rows
// 32 c + 2^(5 - j) + (index inside the chunk), and the tile's coarse values (levels 6..8, approximation
// first, then details from the coarsest level down) at rows 32 q, q = 0..7.
__device__ __forceinline__ long debug_tiled_row(long M, int n, int levels, long r, int* level_out) {
  const long blk = r / n;
  const int i = static_cast<int>(r - blk * n);
  int j, idx;
  bool approx = false;
  if (i < (n >> levels)) {
    j = levels;
    idx = i;
    approx = true;
  } else {
    j = levels;
    while ((n >> (j - 1)) <= i) --j;   // n >> j <= i < n >> (j - 1)
    idx = i - (n >> j);
  }
  *level_out = j;
  if (j > 8) return M + blk * (n >> 8) + i;
  const long first_token = blk * n + ((long)idx << j);   // first original token the coefficient covers
  const long tile = first_token >> 8;
  const int in_tile = idx & ((256 >> j) - 1);            // index among the tile's coefficients of level j
  int row;
  if (j <= 5 && !approx) {
    const int per_chunk = 32 >> j;                        // level-j details per 32-token chunk
    row = 32 * (in_tile / per_chunk) + per_chunk + (in_tile % per_chunk);
  } else if (approx) {
    row = 32 * in_tile;                                   // approximation band: the first coarse slots (or slot 0 of a chunk)
  } else {
    row = 32 * ((256 >> j) + in_tile);                    // detail of level 6..8: after the coarser bands
  }
  return tile * 256 + row;
}

// One CTA per logical row.  codes [M, K] int8, factor [M] float (scale x 2^(-j/2) for tile rows, the plain
// scale for rows of levels above 8), level [M] int.
__global__ void __launch_bounds__(256) k_debug_gather_tiled(const int8_t* __restrict__ a8, const float* __restrict__ sx_epi,
                                                            const float* __restrict__ sx_top, long M, int n, int levels,
                                                            int K, int8_t* __restrict__ codes, float* __restrict__ factor,
                                                            int* __restrict__ level) {
  const long r = blockIdx.x;
  int j;
  const long prow = debug_tiled_row(M, n, levels, r, &j);
  const int4* src = reinterpret_cast<const int4*>(a8 + prow * (long)K);
  int4* dst = reinterpret_cast<int4*>(codes + r * (long)K);
  for (int k = threadIdx.x; k < K / 16; k += blockDim.x) dst[k] = src[k];
  if (threadIdx.x == 0) {
    factor[r] = prow >= M ? sx_top[prow - M] : sx_epi[prow];
    level[r] = j;
  }
}

// 2-D Haar, three levels, patch order: rows [64 p, 64 p + 64) hold 8 x 8 patch p (patches in raster order of the
// block's patch grid, blocks in order); row 0 the patch's LL_3 value, row 4^(3-l) + 3 * cell + band the level-l
// detail `band` (0 LH, 1 HL, 2 HH) of the patch's cell (row-major over its (8 >> l) x (8 >> l) cells).
// Logical order of a block: [LL_3 | LH_3 | HL_3 | HH_3 | LH_2 | ... | HH_1], every band in raster order of its grid.
__global__ void __launch_bounds__(256) k_debug_gather_patch(const int8_t* __restrict__ a8, const float* __restrict__ sx_epi,
                                                            const int* __restrict__ zp_epi, long M, int n, int w, int K,
                                                            int8_t* __restrict__ codes, float* __restrict__ factor,
                                                            int* __restrict__ level, int* __restrict__ zero) {
  const long r = blockIdx.x;
  const long blk = r / n;
  const int i = static_cast<int>(r - blk * n);
  const int patches_per_row = w >> 3;
  const int patches_per_block = n >> 6;
  int l = 3, band = -1, pos = i;
  if (i >= (n >> 6)) {
    l = 3;
    while ((n >> (2 * (l - 1))) <= i) --l;   // n >> 2l <= i < n >> 2(l-1)
    const int q = n >> (2 * l);
    band = i / q - 1;
    pos = i - (band + 1) * q;
  }
  const int gw = w >> l;
  const int gy = pos / gw, gx = pos - gy * gw;
  const int sh = 3 - l;
  const int py = gy >> sh, px = gx >> sh;
  const int cells = 8 >> l;
  const int cell = (gy & (cells - 1)) * cells + (gx & (cells - 1));
  const int idx = band < 0 ? 0 : (1 << (2 * sh)) + 3 * cell + band;
  const long prow = 64 * (blk * patches_per_block + (long)py * patches_per_row + px) + idx;
  const int4* src = reinterpret_cast<const int4*>(a8 + prow * (long)K);
  int4* dst = reinterpret_cast<int4*>(codes + r * (long)K);
  for (int k = threadIdx.x; k < K / 16; k += blockDim.x) dst[k] = src[k];
  if (threadIdx.x == 0) {
    factor[r] = sx_epi[prow];
    level[r] = l;
    if (zero) zero[r] = zp_epi ? zp_epi[prow] : 0;
  }
}

}  // namespace stamp
