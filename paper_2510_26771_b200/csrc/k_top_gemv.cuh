// The few transformed tokens above the GEMM's 256-token tiles (Haar levels > 8), for short
// sequences: when a layer has at most 16 such rows, their product with the weights is a skinny
// GEMV-like contraction bound by reading the weights once, not worth a tensor-core launch plus a
// separate inverse pass.  One kernel does, per output channel:
//   acc[r] = sum_k top_codes[r, k] * w8[ch, k]          (dp4a, int32: Algorithm line "Y <- X W^T")
//   yt[r]  = acc[r] * x_scale[r]                        (weight scales are applied by the main GEMM)
//   a8[.]  = inverse Haar of the (levels - 8) top levels over each block's rows (orthonormal)
// and writes a8v [R, n_out]: the level-8 approximation coefficient of every 256-token tile, which
// the main GEMM's fused epilogue continues from.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

constexpr int TOPG_THREADS = 256;
constexpr int TOPG_CH_PER_WARP = 4;

// R = total top rows (nseq * rows_per_block), rows_per_block = 2^top_levels.
//   codes [R, K] int8, x_scale [R], w8 [n_out, K] int8, a8v [R, n_out] float
template <int R>
__global__ void __launch_bounds__(TOPG_THREADS, (R <= 4 ? 3 : (R <= 8 ? 4 : 2))) k_top_gemv(const int8_t* __restrict__ codes,
                                                           const float* __restrict__ x_scale,
                                                           const int8_t* __restrict__ w8, int K, int n_out,
                                                           int top_levels, float* __restrict__ a8v) {
  extern __shared__ __align__(16) uint8_t topg_smem[];   // [R, K] codes
  ptx::grid_dependency_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  {
    const uint4* src = reinterpret_cast<const uint4*>(codes);
    uint4* dst = reinterpret_cast<uint4*>(topg_smem);
    for (int i = threadIdx.x; i < R * K / 16; i += TOPG_THREADS) dst[i] = src[i];
  }
  __syncthreads();
  const int ch0 = (blockIdx.x * (TOPG_THREADS / 32) + warp) * TOPG_CH_PER_WARP;
  if (ch0 >= n_out) return;
  int acc[TOPG_CH_PER_WARP][R];
#pragma unroll
  for (int c = 0; c < TOPG_CH_PER_WARP; ++c)
#pragma unroll
    for (int r = 0; r < R; ++r) acc[c][r] = 0;
  // The kernel is bound by the weight bytes in flight per SM, not by arithmetic.  With few rows (R <= 4) the
  // accumulators leave room for two 512-byte steps of every channel per iteration (eight 16-byte loads per lane in
  // flight: measured 0.077 -> 0.060 ms per layer step at R = 2, K = 8192); from R = 8 on one step per iteration is
  // as fast or faster (the second set of loads would cost occupancy).
  constexpr int NSTEP = (R <= 4) ? 2 : 1;
  for (int k0 = lane * 16; k0 < K; k0 += NSTEP * 32 * 16) {
    const bool second = NSTEP == 2 && k0 + 32 * 16 < K;
    uint4 w[TOPG_CH_PER_WARP][NSTEP];
#pragma unroll
    for (int c = 0; c < TOPG_CH_PER_WARP; ++c) {
      const int ch = min(ch0 + c, n_out - 1);   // a ragged last group re-reads the last channel, stores are guarded
      const uint4* wp = reinterpret_cast<const uint4*>(w8 + (long)ch * K + k0);
      w[c][0] = __ldg(wp);
      if (NSTEP == 2) w[c][NSTEP - 1] = second ? __ldg(wp + 32) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < NSTEP; ++u) {
      if (u == 1 && !second) break;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const uint4 a = *reinterpret_cast<const uint4*>(topg_smem + r * K + k0 + u * 32 * 16);
#pragma unroll
        for (int c = 0; c < TOPG_CH_PER_WARP; ++c) {
          int s = acc[c][r];
          s = __dp4a(static_cast<int>(a.x), static_cast<int>(w[c][u].x), s);
          s = __dp4a(static_cast<int>(a.y), static_cast<int>(w[c][u].y), s);
          s = __dp4a(static_cast<int>(a.z), static_cast<int>(w[c][u].z), s);
          s = __dp4a(static_cast<int>(a.w), static_cast<int>(w[c][u].w), s);
          acc[c][r] = s;
        }
      }
    }
  }
  // sum over the lanes; lane c then owns channel ch0 + c
  float y[R];
#pragma unroll
  for (int r = 0; r < R; ++r) y[r] = 0.f;
#pragma unroll
  for (int c = 0; c < TOPG_CH_PER_WARP; ++c)
#pragma unroll
    for (int r = 0; r < R; ++r) {
      int s = acc[c][r];
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == c) y[r] = static_cast<float>(s) * __ldg(x_scale + r);
    }
  if (lane >= TOPG_CH_PER_WARP || ch0 + lane >= n_out) return;
  // inverse Haar over each block's rows [a | d_top | ... ] (orthonormal steps), in place
  const int rb = 1 << top_levels;
  const float rs = 0.70710678118654752440f;
#pragma unroll 1
  for (int b0 = 0; b0 < R; b0 += rb) {
    float cur[R], nxt[R];
    cur[0] = y[b0];
    for (int len = 1; len < rb; len <<= 1) {
      for (int i = 0; i < len; ++i) {
        const float d = y[b0 + len + i];
        nxt[2 * i] = (cur[i] + d) * rs;
        nxt[2 * i + 1] = (cur[i] - d) * rs;
      }
      for (int i = 0; i < 2 * len; ++i) cur[i] = nxt[i];
    }
    for (int i = 0; i < rb; ++i) a8v[(long)(b0 + i) * n_out + ch0 + lane] = cur[i];
  }
}

}  // namespace stamp
