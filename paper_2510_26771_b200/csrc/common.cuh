// Shared host/device helpers of the STaMP CUDA library: resolved problem description,
// storage-type loads, Haar normalisation constants, the device status word.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "stamp.h"

namespace stamp {

// Device status word: kernels raise it with atomicMax when a bounded wait expires; the host
// reads and clears it in stamp_last_device_status().
__device__ int g_device_status = 0;

__device__ __forceinline__ void raise_device_status(int code) { atomicMax(&g_device_status, code); }

// A validated problem: everything the launchers need, resolved from stamp_config + sizes.
struct Problem {
  int B, L, K, N;
  int transform;   // stamp_transform
  int n;           // tokens per transform block (power of two, divides L)
  int levels;      // resolved Haar levels (0 for identity / DCT)
  int k_hi;        // 8-bit rows per block
  int grid_w;      // 2-D Haar: patch-grid width of a block (0 otherwise)
  int act_zp;      // 1: zero-point activation codes (min-max range), 0: symmetric
  int group;       // > 0: one scale per `group` features for activations and weights (0: per token / per channel)
  int nseq;        // B * (L / n): independent transform blocks
  long M;          // B * L tokens
  int qmax_hi, qmax_lo, qmax_w;
  long n_hi_rows() const { return (long)nseq * k_hi; }
  long n_lo_rows() const { return M - n_hi_rows(); }
};

// Multiplication by 2^(-j/2).  Even j: an exact power of two.  Odd j: 1/sqrt(2) is split into
// an fp32 head and tail, v * head + v * tail in one FMA, so the product is rounded once (to within
// a hair of the correctly rounded v / sqrt 2) instead of inheriting the constant's rounding error.
struct HaarNorm {
  float hi, lo;
};
__host__ __device__ __forceinline__ HaarNorm haar_norm(int j) {
  HaarNorm h;
  float p = 1.0f;
  for (int i = 0; i < (j >> 1); ++i) p *= 0.5f;  // unrolled / folded where j is a constant
  if (j & 1) {
    h.hi = 0.707106769084930419921875f * p;       // fp32(1/sqrt 2)
    h.lo = 1.2101617101e-8f * p;                  // 1/sqrt 2 - fp32(1/sqrt 2)
  } else {
    h.hi = p;
    h.lo = 0.0f;
  }
  return h;
}
__device__ __forceinline__ float mul_norm(float v, const HaarNorm& h) { return fmaf(v, h.hi, v * h.lo); }

// Two adjacent channels of one token as floats.
__device__ __forceinline__ float2 load2(const float* p) { return *reinterpret_cast<const float2*>(p); }
__device__ __forceinline__ float2 load2(const __nv_bfloat16* p) {
  const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}
__device__ __forceinline__ void store2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16* p, float a, float b) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}

// Bits of a non-negative float compare like unsigned integers.
__device__ __forceinline__ unsigned absbits(float v) { return __float_as_uint(fabsf(v)); }

}  // namespace stamp
