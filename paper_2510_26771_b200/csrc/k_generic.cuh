// General-shape kernels: multi-pass Haar analysis / synthesis along the token axis with the
// transformed activations materialised in fp32, the row quantizer that reads them, code
// (un)packing and the offline weight quantizer.  These serve the debug exports, every shape the
// specialised kernels do not cover, and the unfused API calls.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

// ------------------------------------------------------------------------------------------
// Haar analysis, P levels per pass (Sec. "Efficient Energy Concentration": each DWT step moves
// the averages to the first half and the differences to the second half of the tokens).
//
// One thread owns two adjacent channels of one group of G = 2^P consecutive input tokens and
// runs the butterflies in registers on UNNORMALISED sums; a coefficient of global level j is
// multiplied once by 2^(-(j + norm_off)/2) when it is written (norm_off > 0 when the input rows are
// themselves sums over 2^norm_off tokens produced by another kernel and T is the compact table of
// the remaining coarse rows).  Detail rows go to their logical row of T,
// [a | d_levels | ... | d_1]; the group's running sum goes to `aout` for the next pass, or, in
// the last pass, to the approximation rows of T.
//   in      [nseq, Lin, K]      TIn (first pass: X; later passes: unnormalised sums, float)
//   T       [nseq * n, K]       float
//   aout    [nseq, Lin >> P, K] float, or nullptr in the last pass
//   rowmax  [nseq * n]          uint bit patterns of per-row |T| maxima (atomicMax), or nullptr
// ------------------------------------------------------------------------------------------
template <int P, typename TIn>
__global__ void __launch_bounds__(128) k_haar_fwd_pass(const TIn* __restrict__ in, int Lin, long ngroups, int K,
                                                       float* __restrict__ T, int n, int lvl0, int norm_off,
                                                       float* __restrict__ aout, unsigned* __restrict__ rowmax) {
  constexpr int G = 1 << P;
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= K) return;  // whole warps only: K/2 is a multiple of 32
  const int gps = Lin >> P;  // groups per transform block
  for (long grp = blockIdx.y; grp < ngroups; grp += gridDim.y) {
    const long s = grp / gps;
    const int g = static_cast<int>(grp - s * gps);
    float a0[G], a1[G];
    const TIn* src = in + ((s * Lin + (long)g * G) * K + c);
#pragma unroll
    for (int t = 0; t < G; ++t) {
      const float2 v = load2(src + (long)t * K);
      a0[t] = v.x;
      a1[t] = v.y;
    }
    float* Tseq = T + (s * n) * (long)K + c;
    unsigned* rm = rowmax ? rowmax + s * n : nullptr;
#pragma unroll
    for (int l = 1; l <= P; ++l) {
      const int half = G >> l;
      const int j = lvl0 + l;
      const HaarNorm nrm = haar_norm(j + norm_off);
      const int row0 = (n >> j) + g * half;
#pragma unroll
      for (int i = 0; i < half; ++i) {
        const float d0 = mul_norm(a0[2 * i] - a0[2 * i + 1], nrm);
        const float d1 = mul_norm(a1[2 * i] - a1[2 * i + 1], nrm);
        const float s0 = a0[2 * i] + a0[2 * i + 1];
        const float s1 = a1[2 * i] + a1[2 * i + 1];
        a0[i] = s0;
        a1[i] = s1;
        store2(Tseq + (long)(row0 + i) * K, d0, d1);
        if (rm) {
          const unsigned m = __reduce_max_sync(0xffffffffu, max(absbits(d0), absbits(d1)));
          if ((threadIdx.x & 31) == 0) atomicMax(rm + row0 + i, m);
        }
      }
    }
    if (aout) {
      store2(aout + ((s * gps + g) * (long)K + c), a0[0], a1[0]);
    } else {
      const HaarNorm nrm = haar_norm(lvl0 + P + norm_off);
      const float v0 = mul_norm(a0[0], nrm), v1 = mul_norm(a1[0], nrm);
      store2(Tseq + (long)g * K, v0, v1);
      if (rm) {
        const unsigned m = __reduce_max_sync(0xffffffffu, max(absbits(v0), absbits(v1)));
        if ((threadIdx.x & 31) == 0) atomicMax(rm + g, m);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Haar synthesis (L^-1 = L^T), P levels per pass, coarse to fine.  A thread owns two adjacent
// output channels of one group: it starts from the group's coarse value, already carrying all
// coarser contributions, and per level adds / subtracts the detail coefficient pre-multiplied
// by 2^(-j/2):  v[2i] = v[i] + d'_j[i],  v[2i+1] = v[i] - d'_j[i].
//   Yt    [nseq * n, N]            float, transformed domain (logical row order)
//   ain   [nseq, n >> (jlo+P), N]  float partial sums from the coarser pass; nullptr in the
//                                  first pass (the approximation rows of Yt are read instead)
//   out   jlo > 0 : [nseq, n >> jlo, N] float partial sums for the next pass
//         jlo == 0: Y [nseq * n, N] TOut, bias added
// norm_off: a level-j coefficient carries 2^(-(j + norm_off)/2) (-1 when the rows belong to a transform that sits one
// level above the table's row order: the dyadic part of the first-token-excluded Haar transform).
// ------------------------------------------------------------------------------------------
template <int P, typename TOut>
__global__ void __launch_bounds__(128) k_haar_inv_pass(const float* __restrict__ Yt, const float* __restrict__ ain,
                                                       int n, int jlo, long ngroups, int N,
                                                       const float* __restrict__ bias, void* __restrict__ out_,
                                                       int norm_off) {
  constexpr int G = 1 << P;
  ptx::grid_dependency_wait();
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= N) return;
  const int gps = n >> (jlo + P);
  float b0 = 0.f, b1 = 0.f;
  if (jlo == 0 && bias != nullptr) {
    b0 = bias[c];
    b1 = bias[c + 1];
  }
  for (long grp = blockIdx.y; grp < ngroups; grp += gridDim.y) {
    const long s = grp / gps;
    const int g = static_cast<int>(grp - s * gps);
    const float* Yseq = Yt + (s * n) * (long)N + c;
    // In-place synthesis with compile-time register indices: the running value of the token range
    // [i, i + 2^l) sits in v[i]; adding / subtracting the level-l detail splits it into the two halves
    // v[i] and v[i + 2^(l-1)], so after level 1 the registers are in natural token order.
    float v0[G], v1[G];
    if (ain) {
      const float2 a = load2(ain + ((s * gps + g) * (long)N + c));
      v0[0] = a.x;
      v1[0] = a.y;
    } else {
      const HaarNorm nrm = haar_norm(jlo + P + norm_off);
      const float2 a = load2(Yseq + (long)g * N);
      v0[0] = mul_norm(a.x, nrm);
      v1[0] = mul_norm(a.y, nrm);
    }
#pragma unroll
    for (int l = P; l >= 1; --l) {
      const int span = 1 << l;               // tokens covered by one level-l coefficient
      const int j = jlo + l;
      const HaarNorm nrm = haar_norm(j + norm_off);
      const int row0 = (n >> j) + g * (G >> l);
#pragma unroll
      for (int i = 0; i < G; i += span) {
        const float2 d = load2(Yseq + (long)(row0 + i / span) * N);
        const float d0 = mul_norm(d.x, nrm), d1 = mul_norm(d.y, nrm);
        const float p0 = v0[i], p1 = v1[i];
        v0[i] = p0 + d0;
        v0[i + span / 2] = p0 - d0;
        v1[i] = p1 + d1;
        v1[i + span / 2] = p1 - d1;
      }
    }
    if (jlo == 0) {
      TOut* dst = static_cast<TOut*>(out_) + ((s * n + (long)g * G) * N + c);
#pragma unroll
      for (int t = 0; t < G; ++t) store2(dst + (long)t * N, v0[t] + b0, v1[t] + b1);
    } else {
      float* dst = static_cast<float*>(out_) + ((s * (long)(n >> jlo) + (long)g * G) * N + c);
#pragma unroll
      for (int t = 0; t < G; ++t) store2(dst + (long)t * N, v0[t], v1[t]);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Haar transform that leaves the first token of every block alone (App. "Experimental details / LLMs": the first
// token of an LLM sequence holds massive outliers, stays at 8 bits and is not transformed).  The n - 1 tokens that
// remain are an odd number: the first level pairs (x1, x2), (x3, x4), ... and carries the last token, which has no
// partner, into the low-pass band unchanged; that band then has n / 2 entries and every deeper level is an ordinary
// dyadic step.  Row order of a block: [x0 | a_l | d_l | ... | d_2 | d_1 (n/2 - 1 rows)].
// First level, forward: writes x0 and the d_1 rows to T (with their maxima), the low-pass band to a1 [nseq, n/2, K]
// (or, when the transform has one level only, to its rows of T).  One thread per channel pair and token pair.
// a1 holds UN-NORMALISED sums x_{2i+1} + x_{2i+2}, as the deeper passes expect of their input (every coefficient
// is then rounded once, when it is written); the carried token enters that band as x * sqrt 2.
// ------------------------------------------------------------------------------------------
template <typename TIn>
__global__ void __launch_bounds__(128) k_skip1_fwd_level1(const TIn* __restrict__ X, int n, long npairs, int K,
                                                          float* __restrict__ T, float* __restrict__ a1, int one_level,
                                                          unsigned* __restrict__ rowmax) {
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= K) return;
  const int half = n >> 1;
  const HaarNorm nrm = haar_norm(1);
  for (long pr = blockIdx.y; pr < npairs; pr += gridDim.y) {
    const long s = pr / half;
    const int i = static_cast<int>(pr - s * half);
    const TIn* xb = X + (s * n) * (long)K + c;
    float* Tb = T + (s * n) * (long)K + c;
    unsigned* rm = rowmax ? rowmax + s * n : nullptr;
    auto put = [&](int row, float v0, float v1) {
      store2(Tb + (long)row * K, v0, v1);
      if (rm) {
        const unsigned m = __reduce_max_sync(0xffffffffu, max(absbits(v0), absbits(v1)));
        if ((threadIdx.x & 31) == 0) atomicMax(rm + row, m);
      }
    };
    constexpr float SQRT2_HI = 1.41421354f, SQRT2_LO = 2.4203235e-8f;   // fp32(sqrt 2) and what it leaves out
    float lo0, lo1;       // low-pass entry: un-normalised (times sqrt 2) unless this is the only level
    if (i < half - 1) {
      const float2 p = load2(xb + (long)(1 + 2 * i) * K), q = load2(xb + (long)(2 + 2 * i) * K);
      lo0 = p.x + q.x;
      lo1 = p.y + q.y;
      if (one_level) {
        lo0 = mul_norm(lo0, nrm);
        lo1 = mul_norm(lo1, nrm);
      }
      put(1 + half + i, mul_norm(p.x - q.x, nrm), mul_norm(p.y - q.y, nrm));
    } else {
      const float2 p = load2(xb + (long)(n - 1) * K);   // no partner: carried as it is
      lo0 = one_level ? p.x : fmaf(p.x, SQRT2_HI, p.x * SQRT2_LO);
      lo1 = one_level ? p.y : fmaf(p.y, SQRT2_HI, p.y * SQRT2_LO);
      const float2 z = load2(xb);                        // and the excluded first token
      put(0, z.x, z.y);
    }
    if (one_level)
      put(1 + i, lo0, lo1);
    else
      store2(a1 + (s * half + i) * (long)K + c, lo0, lo1);
  }
}

// First level, inverse: Y[x0] = Yt row 0; (x_{2i+1}, x_{2i+2}) = (a1[i] +- d_1[i]) / sqrt 2; x_{n-1} = a1[n/2 - 1]; bias added.
// a1 [nseq, n/2, N] is the low-pass band rebuilt by the dyadic passes, as they leave it: a_1 / sqrt 2 (for a one-level
// transform a1 is null and a_1 itself is read from rows 1.. of Yt).
template <typename TOut>
__global__ void __launch_bounds__(128) k_skip1_inv_level1(const float* __restrict__ Yt, const float* __restrict__ a1, int n,
                                                          long npairs, int N, const float* __restrict__ bias,
                                                          TOut* __restrict__ Y) {
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= N) return;
  const int half = n >> 1;
  const HaarNorm nrm = haar_norm(1);
  const float b0 = bias ? bias[c] : 0.f, b1 = bias ? bias[c + 1] : 0.f;
  for (long pr = blockIdx.y; pr < npairs; pr += gridDim.y) {
    const long s = pr / half;
    const int i = static_cast<int>(pr - s * half);
    const float* yb = Yt + (s * n) * (long)N + c;
    TOut* ob = Y + (s * n) * (long)N + c;
    constexpr float SQRT2_HI = 1.41421354f, SQRT2_LO = 2.4203235e-8f;
    float2 a = a1 ? load2(a1 + (s * half + i) * (long)N + c) : load2(yb + (long)(1 + i) * N);
    if (i < half - 1) {
      const float2 d = load2(yb + (long)(1 + half + i) * N);
      const float d0 = mul_norm(d.x, nrm), d1 = mul_norm(d.y, nrm);
      if (!a1) {
        a.x = mul_norm(a.x, nrm);
        a.y = mul_norm(a.y, nrm);
      }
      store2(ob + (long)(1 + 2 * i) * N, a.x + d0 + b0, a.y + d1 + b1);
      store2(ob + (long)(2 + 2 * i) * N, a.x - d0 + b0, a.y - d1 + b1);
    } else {
      if (a1) {   // a_1 / sqrt 2 -> the carried token
        a.x = fmaf(a.x, SQRT2_HI, a.x * SQRT2_LO);
        a.y = fmaf(a.y, SQRT2_HI, a.y * SQRT2_LO);
      }
      store2(ob + (long)(n - 1) * N, a.x + b0, a.y + b1);
      const float2 z = load2(yb);
      store2(ob, z.x + b0, z.y + b1);
    }
  }
}

// t / scale from a pre-computed reciprocal plus one Newton correction: q0 = t * inv,
// q0 + (t - q0 * scale) * inv.  Two FMAs instead of a division, and the quotient is the correctly
// rounded one except in rare half-ulp cases, so codes only differ from a true division when the
// quotient itself sits within one fp32 ulp of a rounding boundary.
__device__ __forceinline__ float div_by_scale(float t, float scale, float inv) {
  const float q0 = t * inv;
  return fmaf(fmaf(-q0, scale, t), inv, q0);
}

// ------------------------------------------------------------------------------------------
// Row quantizer (Sec. 2.1, first equation, symmetric form) reading materialised T.
// One CTA per materialised row: scale = absmax / qmax (IEEE fp32 division), codes =
// clamp(rne(t / scale)).  Writes any of: the int8 operand row for the GEMM (a8), the
// public packed outputs (q_hi rows as int8, q_lo rows as nibble pairs), the scale.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_quant_rows(const float* __restrict__ T, const unsigned* __restrict__ rowmax,
                                                    int K, int n_src, int n, int k_hi, int qmax_hi, int qmax_lo,
                                                    int8_t* __restrict__ a8, int8_t* __restrict__ q_hi,
                                                    uint8_t* __restrict__ q_lo, float* __restrict__ x_scale) {
  // T / rowmax hold the first n_src rows of every block of n logical rows
  const long rs = blockIdx.x;
  const long s = rs / n_src;
  const int i = static_cast<int>(rs - s * n_src);
  const long r = s * n + i;
  const bool hi = i < k_hi;
  const float qmax = static_cast<float>(hi ? qmax_hi : qmax_lo);
  const float amax = __uint_as_float(rowmax[rs]);
  const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
  const float inv = __fdiv_rn(1.0f, scale);
  if (threadIdx.x == 0) x_scale[r] = scale;
  const float4* src = reinterpret_cast<const float4*>(T + rs * (long)K);
  char4* dst8 = a8 ? reinterpret_cast<char4*>(a8 + r * (long)K) : nullptr;
  char4* dsth = (q_hi && hi) ? reinterpret_cast<char4*>(q_hi + (s * k_hi + i) * (long)K) : nullptr;
  uint16_t* dstl =
      (q_lo && !hi) ? reinterpret_cast<uint16_t*>(q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2)) : nullptr;
  for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
    const float4 t = src[k4];
    int q0 = __float2int_rn(div_by_scale(t.x, scale, inv)), q1 = __float2int_rn(div_by_scale(t.y, scale, inv));
    int q2 = __float2int_rn(div_by_scale(t.z, scale, inv)), q3 = __float2int_rn(div_by_scale(t.w, scale, inv));
    const int qm = static_cast<int>(qmax);
    q0 = max(-qm, min(qm, q0));
    q1 = max(-qm, min(qm, q1));
    q2 = max(-qm, min(qm, q2));
    q3 = max(-qm, min(qm, q3));
    const char4 c = make_char4((signed char)q0, (signed char)q1, (signed char)q2, (signed char)q3);
    if (dst8) dst8[k4] = c;
    if (dsth) dsth[k4] = c;
    if (dstl)
      dstl[k4] = static_cast<uint16_t>((q0 & 0xF) | ((q1 & 0xF) << 4) | ((q2 & 0xF) << 8) | ((q3 & 0xF) << 12));
  }
}

// ------------------------------------------------------------------------------------------
// Row quantizer in the zero-point form the first equation of Sec. 2.1 prints, min-max range:
//   s = (max - min) / (2^b - 1)  (1 when the row is constant),  z = rne(-min / s),
//   x_int = clamp(rne(t / s) + z, 0, 2^b - 1).
// Codes are STORED offset by half the code range, c = x_int - 2^(b-1), so that they use the same
// signed byte / nibble formats (and the same signed tensor-core operand) as the symmetric codes; the
// zero point written out is that of the stored code, zc = z - 2^(b-1), and t ~ s * (c - zc).
// One CTA per materialised row; the row is read twice (min/max, then codes), the second time from L2.
// CTAs past the `rows` token rows take the weight row sums of the correction term instead (eight weight rows per
// CTA, one per warp: rs_out[j] = sum_k rs_w8[j, k]), so that the two independent reads share one launch.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_quant_rows_zp(const float* __restrict__ T, long rows, int K, int n, int k_hi,
                                                       int8_t* __restrict__ a8, int8_t* __restrict__ q_hi,
                                                       uint8_t* __restrict__ q_lo, float* __restrict__ x_scale,
                                                       int* __restrict__ x_zero, const int8_t* __restrict__ rs_w8,
                                                       int rs_rows, int* __restrict__ rs_out) {
  __shared__ float red_mn[8], red_mx[8];
  if (blockIdx.x >= rows) {
    const int j = static_cast<int>(blockIdx.x - rows) * 8 + (threadIdx.x >> 5);
    if (j >= rs_rows) return;
    const int* src = reinterpret_cast<const int*>(rs_w8 + (long)j * K);
    int acc = 0;
    for (int k4 = threadIdx.x & 31; k4 < K / 4; k4 += 32) acc = __dp4a(__ldg(src + k4), 0x01010101, acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) rs_out[j] = acc;
    return;
  }
  const long r = blockIdx.x;
  const long s = r / n;
  const int i = static_cast<int>(r - s * n);
  const bool hi = i < k_hi;
  const int half = hi ? 128 : 8;
  const int top = 2 * half - 1;
  const float4* src = reinterpret_cast<const float4*>(T + r * (long)K);
  float mn = __int_as_float(0x7f800000), mx = -mn;
  for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
    const float4 t = src[k4];
    mn = fminf(fminf(mn, t.x), fminf(t.y, fminf(t.z, t.w)));
    mx = fmaxf(fmaxf(mx, t.x), fmaxf(t.y, fmaxf(t.z, t.w)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  if ((threadIdx.x & 31) == 0) {
    red_mn[threadIdx.x >> 5] = mn;
    red_mx[threadIdx.x >> 5] = mx;
  }
  __syncthreads();
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    mn = fminf(mn, red_mn[w]);
    mx = fmaxf(mx, red_mx[w]);
  }
  float scale = __fdiv_rn(mx - mn, static_cast<float>(top));
  if (!(scale > 0.f)) scale = 1.0f;
  const float inv = __fdiv_rn(1.0f, scale);
  float zf = rintf(__fdiv_rn(-mn, scale));
  zf = fminf(fmaxf(zf, -1073741824.0f), 1073741824.0f);
  const int z = static_cast<int>(zf);
  if (threadIdx.x == 0) {
    x_scale[r] = scale;
    x_zero[r] = z - half;
  }
  char4* dst8 = a8 ? reinterpret_cast<char4*>(a8 + r * (long)K) : nullptr;
  char4* dsth = (q_hi && hi) ? reinterpret_cast<char4*>(q_hi + (s * k_hi + i) * (long)K) : nullptr;
  uint16_t* dstl =
      (q_lo && !hi) ? reinterpret_cast<uint16_t*>(q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2)) : nullptr;
  for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
    const float4 t = src[k4];
    int q0 = __float2int_rn(div_by_scale(t.x, scale, inv)) + z, q1 = __float2int_rn(div_by_scale(t.y, scale, inv)) + z;
    int q2 = __float2int_rn(div_by_scale(t.z, scale, inv)) + z, q3 = __float2int_rn(div_by_scale(t.w, scale, inv)) + z;
    q0 = max(0, min(top, q0)) - half;
    q1 = max(0, min(top, q1)) - half;
    q2 = max(0, min(top, q2)) - half;
    q3 = max(0, min(top, q3)) - half;
    const char4 c = make_char4((signed char)q0, (signed char)q1, (signed char)q2, (signed char)q3);
    if (dst8) dst8[k4] = c;
    if (dsth) dsth[k4] = c;
    if (dstl)
      dstl[k4] = static_cast<uint16_t>((q0 & 0xF) | ((q1 & 0xF) << 4) | ((q2 & 0xF) << 8) | ((q3 & 0xF) << 12));
  }
}

// Sum of every row of an int8 matrix [rows, K] (the weight row sums of the zero-point correction
//   sum_k (c - zc) w = sum_k c w  -  zc * sum_k w).  One warp per row.
__global__ void __launch_bounds__(256) k_row_sums_i8(const int8_t* __restrict__ w8, int rows, int K,
                                                     int* __restrict__ out) {
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= rows) return;
  const int* src = reinterpret_cast<const int*>(w8 + (long)r * K);
  int acc = 0;
  for (int k4 = threadIdx.x & 31; k4 < K / 4; k4 += 32) acc = __dp4a(src[k4], 0x01010101, acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) out[r] = acc;
}

// Sign-extend the two nibbles of a byte.
__device__ __forceinline__ int nib_lo(uint32_t b) { return (static_cast<int>(b << 28)) >> 28; }
__device__ __forceinline__ int nib_hi(uint32_t b) { return (static_cast<int>(b << 24)) >> 28; }

// Public code format -> one int8 per code, logical token order.  One CTA per token.
__global__ void __launch_bounds__(256) k_unpack_codes(const int8_t* __restrict__ q_hi, const uint8_t* __restrict__ q_lo,
                                                      int K, int n, int k_hi, int8_t* __restrict__ out) {
  const long r = blockIdx.x;
  const long s = r / n;
  const int i = static_cast<int>(r - s * n);
  char4* dst = reinterpret_cast<char4*>(out + r * (long)K);
  if (i < k_hi) {
    const char4* src = reinterpret_cast<const char4*>(q_hi + (s * k_hi + i) * (long)K);
    for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) dst[k4] = src[k4];
  } else {
    const uint16_t* src = reinterpret_cast<const uint16_t*>(q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2));
    for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
      const uint32_t u = src[k4];
      dst[k4] = make_char4((signed char)nib_lo(u), (signed char)nib_hi(u), (signed char)nib_lo(u >> 8),
                           (signed char)nib_hi(u >> 8));
    }
  }
}

// One int8 per code, logical token order -> the public code format (inverse of k_unpack_codes).
__global__ void __launch_bounds__(256) k_pack_codes(const int8_t* __restrict__ codes, int K, int n, int k_hi,
                                                    int8_t* __restrict__ q_hi, uint8_t* __restrict__ q_lo) {
  const long r = blockIdx.x;
  const long s = r / n;
  const int i = static_cast<int>(r - s * n);
  const char4* src = reinterpret_cast<const char4*>(codes + r * (long)K);
  if (i < k_hi) {
    char4* dst = reinterpret_cast<char4*>(q_hi + (s * k_hi + i) * (long)K);
    for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) dst[k4] = src[k4];
  } else {
    uint16_t* dst = reinterpret_cast<uint16_t*>(q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2));
    for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
      const char4 c = src[k4];
      dst[k4] = static_cast<uint16_t>((c.x & 0xF) | ((c.y & 0xF) << 4) | ((c.z & 0xF) << 8) | ((c.w & 0xF) << 12));
    }
  }
}

// De-quantization of stored activation codes back to transformed values (Sec. 2.1: s (x_int - z)): what a reader
// of a STaMP-quantized KV cache does before the inverse sequence transform.  One CTA per logical row.
//   T[r, k] = x_scale[r (, k / group)] * (code[r, k] - zero[r])        zero: null for symmetric codes
__global__ void __launch_bounds__(256) k_dequant_rows(const int8_t* __restrict__ q_hi, const uint8_t* __restrict__ q_lo,
                                                      const float* __restrict__ x_scale, const int* __restrict__ x_zero,
                                                      int K, int n, int k_hi, int group, float* __restrict__ T) {
  const long r = blockIdx.x;
  const long s = r / n;
  const int i = static_cast<int>(r - s * n);
  const int zc = x_zero ? x_zero[r] : 0;
  const int ng = group ? K / group : 1;
  const float* sc = x_scale + r * (long)ng;
  float* dst = T + r * (long)K;
  if (i < k_hi) {
    const int8_t* src = q_hi + (s * k_hi + i) * (long)K;
    for (int k = threadIdx.x; k < K; k += blockDim.x) dst[k] = sc[group ? k / group : 0] * static_cast<float>(src[k] - zc);
  } else {
    const uint8_t* src = q_lo + (s * (n - k_hi) + (i - k_hi)) * (long)(K / 2);
    for (int k2 = threadIdx.x; k2 < K / 2; k2 += blockDim.x) {
      const uint32_t u = src[k2];
      const int c0 = static_cast<int>(u << 28) >> 28, c1 = static_cast<int>(u << 24) >> 28;   // sign-extended nibbles
      const float f = sc[group ? (2 * k2) / group : 0];
      dst[2 * k2] = f * static_cast<float>(c0 - zc);
      dst[2 * k2 + 1] = f * static_cast<float>(c1 - zc);
    }
  }
}

// Packed 4-bit rows -> int8 rows (weights). One CTA per row.
__global__ void __launch_bounds__(256) k_unpack_rows4(const uint8_t* __restrict__ packed, int K, int8_t* __restrict__ out) {
  const long r = blockIdx.x;
  const uint16_t* src = reinterpret_cast<const uint16_t*>(packed + r * (long)(K / 2));
  char4* dst = reinterpret_cast<char4*>(out + r * (long)K);
  for (int k4 = threadIdx.x; k4 < K / 4; k4 += blockDim.x) {
    const uint32_t u = src[k4];
    dst[k4] = make_char4((signed char)nib_lo(u), (signed char)nib_hi(u), (signed char)nib_lo(u >> 8),
                         (signed char)nib_hi(u >> 8));
  }
}

// Offline weight quantizer: per output channel absmax / qmax, round to nearest, packed nibbles.
template <typename TW>
__global__ void __launch_bounds__(256) k_quant_weights(const TW* __restrict__ W, int K, int qmax_w,
                                                       uint8_t* __restrict__ wq, float* __restrict__ w_scale) {
  __shared__ unsigned red[8];
  const long r = blockIdx.x;
  const TW* src = W + r * (long)K;
  unsigned m = 0;
  for (int k2 = threadIdx.x; k2 < K / 2; k2 += blockDim.x) {
    const float2 v = load2(src + 2 * k2);
    m = max(m, max(absbits(v.x), absbits(v.y)));
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) m = max(m, red[w]);
  const float amax = __uint_as_float(m);
  const float qmax = static_cast<float>(qmax_w);
  const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
  if (threadIdx.x == 0) w_scale[r] = scale;
  uint8_t* dst = wq + r * (long)(K / 2);
  for (int k2 = threadIdx.x; k2 < K / 2; k2 += blockDim.x) {
    const float2 v = load2(src + 2 * k2);
    // offline path: a true division keeps the codes identical to a plain w / scale
    int q0 = max(-qmax_w, min(qmax_w, __float2int_rn(__fdiv_rn(v.x, scale))));
    int q1 = max(-qmax_w, min(qmax_w, __float2int_rn(__fdiv_rn(v.y, scale))));
    dst[k2] = static_cast<uint8_t>((q0 & 0xF) | ((q1 & 0xF) << 4));
  }
}

}  // namespace stamp
