// Blockwise DCT-II along the token axis (Sec. "Efficient Energy Concentration": the DCT as the
// real Fourier basis that approximates the KLT of a Toeplitz autocorrelation), general-shape
// kernels: the orthonormal DCT-II matrix of one transform block is generated on the device and
// applied (or its transpose, for L^-1 = L^T) as a dense fp32 product per block.
//   C[u][t] = c_u sqrt(2/n) cos(pi (2t+1) u / (2n)),  c_0 = 1/sqrt 2, c_u = 1 otherwise;
// row 0 is the DC row, so the low frequencies are the first transformed tokens.
#pragma once
#include "common.cuh"

namespace stamp {

// The n x n matrix in fp32, each entry rounded once from an fp64 evaluation.  The angle is
// reduced in integer arithmetic first ((2t+1) u mod 4n), so cospi() sees an exact argument.
__global__ void __launch_bounds__(256) k_dct_matrix(int n, float* __restrict__ C) {
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long)n * n) return;
  const int u = static_cast<int>(idx / n), t = static_cast<int>(idx - (long)u * n);
  const long a = ((long)(2 * t + 1) * u) % (4L * n);
  const double cu = (u == 0) ? 0.70710678118654752440 : 1.0;
  C[idx] = static_cast<float>(cu * sqrt(2.0 / n) * cospi(static_cast<double>(a) / (2.0 * n)));
}

// Sign (+1 / -1) of entry (u, t) of the sequency-ordered Walsh-Hadamard matrix of size 2^bits: row u is
// the natural-order Hadamard row  bit_reverse(gray(u)),  whose entry t is (-1)^popcount(row & t); that
// row changes sign exactly u times (Sec. "Efficient Energy Concentration": the DCT reduced to its signs).
__host__ __device__ __forceinline__ int wht_sign(int u, int t, int bits) {
  const unsigned g = static_cast<unsigned>(u) ^ (static_cast<unsigned>(u) >> 1);
  unsigned row = 0;
  for (int b = 0; b < bits; ++b) row |= ((g >> b) & 1u) << (bits - 1 - b);
  unsigned x = row & static_cast<unsigned>(t);
  x ^= x >> 16; x ^= x >> 8; x ^= x >> 4; x ^= x >> 2; x ^= x >> 1;
  return (x & 1u) ? -1 : 1;
}

// The n x n Walsh-Hadamard matrix (sequency order, orthonormal) in fp32.
__global__ void __launch_bounds__(256) k_wht_matrix(int n, int bits, float* __restrict__ C) {
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long)n * n) return;
  const int u = static_cast<int>(idx / n), t = static_cast<int>(idx - (long)u * n);
  C[idx] = static_cast<float>(wht_sign(u, t, bits) / sqrt(static_cast<double>(n)));
}

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) {
  return __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(p)) << 16);
}
__device__ __forceinline__ void st_from_float(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_from_float(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// out[blk*n + r, c] = sum_t A[r][t] * in[blk*n + t, c] (+ bias[c]),  A = C (TRANSPOSE = false:
// the transform) or C^T (TRANSPOSE = true: its inverse).  One CTA computes a 64-row x 64-column
// tile of one transform block; a thread owns 4 rows x 4 columns (columns strided by 16 so that a
// warp's accesses to a token row are contiguous).  fp32 FMAs, reduction over t in order.
//   rowmax [nblk * n] uint bit patterns of the per-row |out| maxima (atomicMax), or nullptr.
template <bool TRANSPOSE, typename TIn, typename TOut>
__global__ void __launch_bounds__(256) k_dct_apply(const float* __restrict__ C, int n, const TIn* __restrict__ in,
                                                   int cols, TOut* __restrict__ out, const float* __restrict__ bias,
                                                   unsigned* __restrict__ rowmax) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN];
  const int row_tiles = (n + BM - 1) / BM;
  const long blk = blockIdx.x / row_tiles;
  const int r0 = (blockIdx.x - blk * row_tiles) * BM;
  const int c0 = blockIdx.y * BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const TIn* in_blk = in + blk * (long)n * cols;
  float acc[4][4] = {};
  for (int t0 = 0; t0 < n; t0 += BK) {
    // A tile: BK x BM (k-major in shared memory), 1024 values over 256 threads
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = threadIdx.x + i * 256;
      int kk, rr;
      if (TRANSPOSE) {  // A[r][t] = C[t][r]: consecutive threads walk r, contiguous in C
        kk = e / BM;
        rr = e - kk * BM;
      } else {          // A[r][t] = C[r][t]: consecutive threads walk t
        rr = e / BK;
        kk = e - rr * BK;
      }
      const int r = r0 + rr, t = t0 + kk;
      float v = 0.f;
      if (r < n && t < n) v = TRANSPOSE ? C[(long)t * n + r] : C[(long)r * n + t];
      As[kk][rr] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = threadIdx.x + i * 256;
      const int kk = e / BN, cc = e - kk * BN;
      const int t = t0 + kk, c = c0 + cc;
      Bs[kk][cc] = (t < n && c < cols) ? ld_as_float(in_blk + (long)t * cols + c) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty * 4 + i;
    unsigned m = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + tx + 16 * j;
      if (r < n && c < cols) {
        float v = acc[i][j];
        if (bias) v += bias[c];
        st_from_float(out + (blk * n + r) * (long)cols + c, v);
        m = max(m, absbits(acc[i][j]));
      }
    }
    if (rowmax) {  // the 16 lanes that share this row sit in one half-warp
      m = max(m, __shfl_xor_sync(0xffffffffu, m, 8));
      m = max(m, __shfl_xor_sync(0xffffffffu, m, 4));
      m = max(m, __shfl_xor_sync(0xffffffffu, m, 2));
      m = max(m, __shfl_xor_sync(0xffffffffu, m, 1));
      if (tx == 0 && r < n) atomicMax(rowmax + blk * n + r, m);
    }
  }
}

}  // namespace stamp
