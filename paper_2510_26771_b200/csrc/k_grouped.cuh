// Per-block ("group") scales along the feature axis for activations and weights (the LVM table's setting: W4A4
// per-block quantization with block size 64; App. "Experimental details / LVMs").  Every run of `group` consecutive
// features of a row has its own scale = absmax / qmax and is quantized with the symmetric round-to-nearest
// quantizer of Sec. 2.1; the product is de-quantized group by group:
//     Yt[m, n] = sum_g ( sum_{k in g} q[m, k] wq[n, k] ) * sx[m, g] * sw[n, g].
// General-shape kernels: quantizers that read materialised rows, and a CUDA-core dp4a product
// that scales its integer partial sums after every group (the tensor-core product of k_gemm_grouped_tc.cuh takes the
// shapes it can; this one the rest).  group = 64 * 2^i, K a multiple of group.
#pragma once
#include "common.cuh"
#include "k_generic.cuh"

namespace stamp {

// One CTA of 256 threads per row; a warp owns a run of 64 features (two per lane) at a time.
//   src row: K values (float: materialised T; or the weight dtype)      scale row: K / group
// Output (any of): a8 row (one code per int8), q_hi row (int8), q_lo row (nibble pairs, low nibble = even k).
template <typename TIn>
__device__ __forceinline__ void quant_row_grouped(const TIn* __restrict__ src, int K, int group, float qmax,
                                                  float* __restrict__ scale_row, int8_t* __restrict__ dst8,
                                                  uint8_t* __restrict__ dst4, unsigned* smax /* [K / 64] shared */) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
  const int n64 = K >> 6;
  for (int b = warp; b < n64; b += nwarp) {
    const float2 v = load2(src + 64 * b + 2 * lane);
    const unsigned m = __reduce_max_sync(0xffffffffu, max(absbits(v.x), absbits(v.y)));
    if (lane == 0) smax[b] = m;
  }
  __syncthreads();
  const int per = group >> 6;           // 64-feature runs per group
  const int qm = static_cast<int>(qmax);
  for (int b = warp; b < n64; b += nwarp) {
    const int g = b / per;
    unsigned m = 0;
    for (int t = 0; t < per; ++t) m = max(m, smax[g * per + t]);
    const float amax = __uint_as_float(m);
    const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
    const float inv = __fdiv_rn(1.0f, scale);
    if (lane == 0 && b == g * per) scale_row[g] = scale;
    const float2 v = load2(src + 64 * b + 2 * lane);
    const int q0 = max(-qm, min(qm, __float2int_rn(div_by_scale(v.x, scale, inv))));
    const int q1 = max(-qm, min(qm, __float2int_rn(div_by_scale(v.y, scale, inv))));
    if (dst8) *reinterpret_cast<char2*>(dst8 + 64 * b + 2 * lane) = make_char2((signed char)q0, (signed char)q1);
    if (dst4) dst4[32 * b + lane] = static_cast<uint8_t>((q0 & 0xF) | ((q1 & 0xF) << 4));
  }
}

// Activations: T [M, K] fp32 in logical order -> codes + scales [M, K / group].
__global__ void __launch_bounds__(256) k_quant_rows_grouped(const float* __restrict__ T, int K, int n, int k_hi, int qmax_hi,
                                                            int qmax_lo, int group, int8_t* __restrict__ a8,
                                                            int8_t* __restrict__ q_hi, uint8_t* __restrict__ q_lo,
                                                            float* __restrict__ x_scale) {
  extern __shared__ unsigned qg_smax[];
  const long r = blockIdx.x;
  const long s = r / n;
  const int i = static_cast<int>(r - s * n);
  const bool hi = i < k_hi;
  int8_t* d8 = a8 ? a8 + r * (long)K : (q_hi && hi) ? q_hi + (s * k_hi + i) * (long)K : nullptr;
  uint8_t* d4 = (q_lo && !hi) ? q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2) : nullptr;
  quant_row_grouped(T + r * (long)K, K, group, static_cast<float>(hi ? qmax_hi : qmax_lo), x_scale + r * (long)(K / group), d8,
                    d4, qg_smax);
}

// Weights (offline): W [N, K] -> packed 4-bit codes [N, K / 2] + scales [N, K / group].
template <typename TW>
__global__ void __launch_bounds__(256) k_quant_weights_grouped(const TW* __restrict__ W, int K, int qmax_w, int group,
                                                               uint8_t* __restrict__ wq, float* __restrict__ w_scale) {
  extern __shared__ unsigned qg_smax[];
  const long r = blockIdx.x;
  quant_row_grouped(W + r * (long)K, K, group, static_cast<float>(qmax_w), w_scale + r * (long)(K / group), nullptr,
                    wq + r * (long)(K / 2), qg_smax);
}

// Yt [M, N] fp32 from a8 [M, K], w8 [N, K] (one code per int8) and the two scale tables.  A CTA of 256 threads
// computes 64 tokens x 64 channels, a thread 4 x 4 of them; K advances 64 features at a time through shared memory
// (rows padded to 68 bytes), dp4a into int32, and at the end of every group the partial sums are scaled into the
// fp32 accumulators.
constexpr int GG_TILE = 64;
constexpr int GG_PITCH = 68;   // bytes per staged row: 64 codes + 4 of padding (17 words: spreads the rows over the banks)
__global__ void __launch_bounds__(256) k_gemm_grouped(const int8_t* __restrict__ a8, const int8_t* __restrict__ w8,
                                                      const float* __restrict__ sx, const float* __restrict__ sw, long M,
                                                      int N, int K, int group, float* __restrict__ Yt) {
  __shared__ __align__(16) uint8_t sa[GG_TILE * GG_PITCH];
  __shared__ __align__(16) uint8_t sb[GG_TILE * GG_PITCH];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const long tok0 = (long)blockIdx.y * GG_TILE;
  const int ch0 = blockIdx.x * GG_TILE;
  const int ng = K / group, steps = group >> 6;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int g = 0; g < ng; ++g) {
    int part[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) part[i][j] = 0;
    for (int st = 0; st < steps; ++st) {
      const int k0 = g * group + st * 64;
      __syncthreads();   // the previous step's reads are done
      // stage 64 rows x 64 bytes of either operand: thread t copies 16 bytes of row t / 4
      {
        const int row = threadIdx.x >> 2, part16 = threadIdx.x & 3;
        int4 va = make_int4(0, 0, 0, 0), vb = make_int4(0, 0, 0, 0);
        if (tok0 + row < M) va = *reinterpret_cast<const int4*>(a8 + (tok0 + row) * (long)K + k0 + 16 * part16);
        if (ch0 + row < N) vb = *reinterpret_cast<const int4*>(w8 + (long)(ch0 + row) * K + k0 + 16 * part16);
        int* pa = reinterpret_cast<int*>(sa + row * GG_PITCH + 16 * part16);
        int* pb = reinterpret_cast<int*>(sb + row * GG_PITCH + 16 * part16);
        pa[0] = va.x; pa[1] = va.y; pa[2] = va.z; pa[3] = va.w;
        pb[0] = vb.x; pb[1] = vb.y; pb[2] = vb.z; pb[3] = vb.w;
      }
      __syncthreads();
#pragma unroll 4
      for (int k4 = 0; k4 < 16; ++k4) {
        int a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const int*>(sa + (4 * ty + i) * GG_PITCH + 4 * k4);
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const int*>(sb + (4 * tx + j) * GG_PITCH + 4 * k4);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) part[i][j] = __dp4a(a[i], b[j], part[i][j]);
      }
    }
    float fa[4], fb[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) fa[i] = (tok0 + 4 * ty + i < M) ? sx[(tok0 + 4 * ty + i) * (long)ng + g] : 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) fb[j] = (ch0 + 4 * tx + j < N) ? sw[(long)(ch0 + 4 * tx + j) * ng + g] : 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(static_cast<float>(part[i][j]), fa[i] * fb[j], acc[i][j]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long tok = tok0 + 4 * ty + i;
    if (tok >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int ch = ch0 + 4 * tx + j;
      if (ch < N) Yt[tok * (long)N + ch] = acc[i][j];
    }
  }
}

}  // namespace stamp
