// 2-D Haar DWT over the patch grid of image tokens (Sec. "Efficient Energy Concentration": for
// images the wavelet transform runs over both spatial axes and a quarter of the tokens stays
// low-pass per level; LVM set-up: 3 levels on a 64 x 64 grid leave the 64 low-pass tokens that get
// 8 bits).  A transform block of n tokens is a grid of h = n / w rows by w columns in raster order.
// One level maps every 2 x 2 cell (a b / c d) to
//     LL = (a + b + c + d) / 2    LH = (a - b + c - d) / 2    HL = (a + b - c - d) / 2    HH = (a - b - c + d) / 2
// (orthonormal; all factors are powers of two) and recurses on the LL grid.  Output order:
//     [LL_l | LH_l | HL_l | HH_l | LH_(l-1) | HL_(l-1) | HH_(l-1) | ... | LH_1 | HL_1 | HH_1],
// each band in raster order of its (h >> level) x (w >> level) grid.
//
// General-shape kernels: a thread owns two adjacent channels of one 2^LV x 2^LV patch, holds it in
// registers (compile-time indices only) and writes the fp32 coefficients to their logical rows;
// the row quantizer reads them.  LV <= 3.
#pragma once
#include "common.cuh"

namespace stamp {

// Logical row, inside a block of n tokens, of the level-l coefficient of `band` (0 = LH, 1 = HL,
// 2 = HH; the low-pass band of the last level is band -1) at grid position (gy, gx).
__device__ __forceinline__ int haar2d_row(int n, int w, int l, int band, int gy, int gx) {
  const int q = n >> (2 * l);
  return (band + 1) * q + gy * (w >> l) + gx;
}

//   in      [nblk, n, K]  TIn        T  [nblk * n, K] float     rowmax [nblk * n] uint bits or nullptr
template <int LV, typename TIn>
__global__ void __launch_bounds__(128) k_haar2d_fwd(const TIn* __restrict__ in, int n, int w, long npatch, int K,
                                                     float* __restrict__ T, unsigned* __restrict__ rowmax) {
  constexpr int S = 1 << LV;
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= K) return;  // whole warps only: K/2 is a multiple of 32
  const int pw = w / S, ph = (n / w) / S;   // patches per grid row / column
  for (long pt = blockIdx.y; pt < npatch; pt += gridDim.y) {
    const long blk = pt / (pw * ph);
    const int pi = static_cast<int>(pt - blk * (pw * ph));
    const int py = pi / pw, px = pi - py * pw;
    const TIn* src = in + ((blk * n + (long)(py * S) * w + px * S) * K + c);
    float2 v[S][S];
#pragma unroll
    for (int y = 0; y < S; ++y)
#pragma unroll
      for (int x = 0; x < S; ++x) v[y][x] = load2(src + ((long)y * w + x) * K);
    float* Tb = T + (blk * n) * (long)K + c;
    unsigned* rm = rowmax ? rowmax + blk * n : nullptr;
    auto emit = [&](int row, float2 t) {
      store2(Tb + (long)row * K, t.x, t.y);
      if (rm) {
        const unsigned m = __reduce_max_sync(0xffffffffu, max(absbits(t.x), absbits(t.y)));
        if ((threadIdx.x & 31) == 0) atomicMax(rm + row, m);
      }
    };
#pragma unroll
    for (int l = 1; l <= LV; ++l) {
      const int st = 1 << (l - 1);
#pragma unroll
      for (int y = 0; y < S; y += 2 * st)
#pragma unroll
        for (int x = 0; x < S; x += 2 * st) {
          const float2 a = v[y][x], b = v[y][x + st], cc = v[y + st][x], d = v[y + st][x + st];
          const int gy = (py * S + y) >> l, gx = (px * S + x) >> l;
          v[y][x] = make_float2(0.5f * ((a.x + b.x) + (cc.x + d.x)), 0.5f * ((a.y + b.y) + (cc.y + d.y)));
          emit(haar2d_row(n, w, l, 0, gy, gx), make_float2(0.5f * ((a.x - b.x) + (cc.x - d.x)), 0.5f * ((a.y - b.y) + (cc.y - d.y))));
          emit(haar2d_row(n, w, l, 1, gy, gx), make_float2(0.5f * ((a.x + b.x) - (cc.x + d.x)), 0.5f * ((a.y + b.y) - (cc.y + d.y))));
          emit(haar2d_row(n, w, l, 2, gy, gx), make_float2(0.5f * ((a.x - b.x) - (cc.x - d.x)), 0.5f * ((a.y - b.y) - (cc.y - d.y))));
        }
    }
    emit(haar2d_row(n, w, LV, -1, py, px), v[0][0]);
  }
}

//   Yt [nblk * n, N] float (logical rows)      out [nblk * n, N] TOut, bias added
template <int LV, typename TOut>
__global__ void __launch_bounds__(128) k_haar2d_inv(const float* __restrict__ Yt, int n, int w, long npatch, int N,
                                                     const float* __restrict__ bias, TOut* __restrict__ out) {
  constexpr int S = 1 << LV;
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= N) return;
  const int pw = w / S, ph = (n / w) / S;
  float b0 = 0.f, b1 = 0.f;
  if (bias != nullptr) {
    b0 = bias[c];
    b1 = bias[c + 1];
  }
  for (long pt = blockIdx.y; pt < npatch; pt += gridDim.y) {
    const long blk = pt / (pw * ph);
    const int pi = static_cast<int>(pt - blk * (pw * ph));
    const int py = pi / pw, px = pi - py * pw;
    const float* Yb = Yt + (blk * n) * (long)N + c;
    float2 v[S][S];
    v[0][0] = load2(Yb + (long)haar2d_row(n, w, LV, -1, py, px) * N);
#pragma unroll
    for (int l = LV; l >= 1; --l) {
      const int st = 1 << (l - 1);
#pragma unroll
      for (int y = 0; y < S; y += 2 * st)
#pragma unroll
        for (int x = 0; x < S; x += 2 * st) {
          const int gy = (py * S + y) >> l, gx = (px * S + x) >> l;
          const float2 ll = v[y][x];
          const float2 lh = load2(Yb + (long)haar2d_row(n, w, l, 0, gy, gx) * N);
          const float2 hl = load2(Yb + (long)haar2d_row(n, w, l, 1, gy, gx) * N);
          const float2 hh = load2(Yb + (long)haar2d_row(n, w, l, 2, gy, gx) * N);
          // the 4 x 4 cell matrix is symmetric and orthonormal: its inverse is itself
          v[y][x] = make_float2(0.5f * ((ll.x + lh.x) + (hl.x + hh.x)), 0.5f * ((ll.y + lh.y) + (hl.y + hh.y)));
          v[y][x + st] = make_float2(0.5f * ((ll.x - lh.x) + (hl.x - hh.x)), 0.5f * ((ll.y - lh.y) + (hl.y - hh.y)));
          v[y + st][x] = make_float2(0.5f * ((ll.x + lh.x) - (hl.x + hh.x)), 0.5f * ((ll.y + lh.y) - (hl.y + hh.y)));
          v[y + st][x + st] = make_float2(0.5f * ((ll.x - lh.x) - (hl.x - hh.x)), 0.5f * ((ll.y - lh.y) - (hl.y - hh.y)));
        }
    }
    TOut* dst = out + ((blk * n + (long)(py * S) * w + px * S) * N + c);
#pragma unroll
    for (int y = 0; y < S; ++y)
#pragma unroll
      for (int x = 0; x < S; ++x) store2(dst + ((long)y * w + x) * N, v[y][x].x + b0, v[y][x].y + b1);
  }
}

}  // namespace stamp
