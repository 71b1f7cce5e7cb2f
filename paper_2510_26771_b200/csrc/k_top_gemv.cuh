// The few transformed tokens above the GEMM's 256-token tiles (Haar levels > 8), for short
// sequences: when a layer has at most 16 such rows, their product with the weights is a skinny
// GEMV-like contraction bound by reading the weights once, not worth a tensor-core launch plus a
// separate inverse pass.  One kernel does, per output channel:
//   acc[r] = sum_k top_codes[r, k] * w8[ch, k]          (dp4a, int32: the product step of Algorithm 1)
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

// Eight two's-complement nibbles of a word (nibble 0 = lowest = even feature first) -> eight int8 in two words.
__device__ __forceinline__ void topg_unpack8(uint32_t w, uint32_t& b0, uint32_t& b1) {
  uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;      // features 0, 2, 4, 6 / 1, 3, 5, 7
  lo |= (lo & 0x08080808u) * 0x1Eu;                                // sign-extend every byte: bit 3 -> bits 4..7
  hi |= (hi & 0x08080808u) * 0x1Eu;
  b0 = __byte_perm(lo, hi, 0x5140);
  b1 = __byte_perm(lo, hi, 0x7362);
}

// R = total top rows (nseq * rows_per_block), rows_per_block = 2^top_levels.
//   codes [R, K] int8, x_scale [R], w8 [n_out, K] int8, a8v [R, n_out] float
// PACKED: the weights are read as packed 4-bit codes [n_out, K / 2] instead (half the bytes of what is a pure
// weight stream) and expanded in registers; a lane then covers 32 features per 16-byte load.
template <int R, bool PACKED = false>
__global__ void __launch_bounds__(TOPG_THREADS, (R <= 4 ? 3 : (R <= 8 ? 4 : 2))) k_top_gemv(const int8_t* __restrict__ codes,
                                                           const float* __restrict__ x_scale,
                                                           const int8_t* __restrict__ w8, int K, int n_out,
                                                           int top_levels, float* __restrict__ a8v) {
  extern __shared__ __align__(16) uint8_t topg_smem[];   // [R, K] codes
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();   // the next kernel may set itself up on SMs as they fall free; it still waits for this grid to finish
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
  constexpr int FPL = PACKED ? 32 : 16;     // features per lane and 16-byte load
  for (int k0 = lane * FPL; k0 < K; k0 += NSTEP * 32 * FPL) {
    const bool second = NSTEP == 2 && k0 + 32 * FPL < K;
    uint4 w[TOPG_CH_PER_WARP][NSTEP];
#pragma unroll
    for (int c = 0; c < TOPG_CH_PER_WARP; ++c) {
      const int ch = min(ch0 + c, n_out - 1);   // a ragged last group re-reads the last channel, stores are guarded
      const uint4* wp = PACKED ? reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(w8) + (long)ch * (K / 2) + k0 / 2)
                               : reinterpret_cast<const uint4*>(w8 + (long)ch * K + k0);
      w[c][0] = __ldg(wp);
      if (NSTEP == 2) w[c][NSTEP - 1] = second ? __ldg(wp + 32) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < NSTEP; ++u) {
      if (u == 1 && !second) break;
      if constexpr (PACKED) {
#pragma unroll
        for (int c = 0; c < TOPG_CH_PER_WARP; ++c) {
          uint32_t b[8];
          topg_unpack8(w[c][u].x, b[0], b[1]);
          topg_unpack8(w[c][u].y, b[2], b[3]);
          topg_unpack8(w[c][u].z, b[4], b[5]);
          topg_unpack8(w[c][u].w, b[6], b[7]);
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const uint4 a0 = *reinterpret_cast<const uint4*>(topg_smem + r * K + k0 + u * 32 * FPL);
            const uint4 a1 = *reinterpret_cast<const uint4*>(topg_smem + r * K + k0 + u * 32 * FPL + 16);
            int s = acc[c][r];
            s = __dp4a(static_cast<int>(a0.x), static_cast<int>(b[0]), s);
            s = __dp4a(static_cast<int>(a0.y), static_cast<int>(b[1]), s);
            s = __dp4a(static_cast<int>(a0.z), static_cast<int>(b[2]), s);
            s = __dp4a(static_cast<int>(a0.w), static_cast<int>(b[3]), s);
            s = __dp4a(static_cast<int>(a1.x), static_cast<int>(b[4]), s);
            s = __dp4a(static_cast<int>(a1.y), static_cast<int>(b[5]), s);
            s = __dp4a(static_cast<int>(a1.z), static_cast<int>(b[6]), s);
            s = __dp4a(static_cast<int>(a1.w), static_cast<int>(b[7]), s);
            acc[c][r] = s;
          }
        }
      } else {
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
