// Fused Haar transform + per-token mixed-precision quantizer (Algorithm lines "X <- L X" and
// "x_i <- Q(x_i; b_i)") for bf16 activations: one pass over X in HBM.
//
// Why it can be one pass.  The per-token scale needs a whole transformed ROW (all K channels),
// the transform needs whole COLUMNS (all tokens).  A Haar detail coefficient of level j only
// depends on 2^j consecutive tokens, so a CTA that owns G = 2^m consecutive tokens x all K
// channels owns every detail row of levels 1..m of its token range completely: it can take the
// row maxima, quantize and store them without any other CTA.  A thread-block cluster of CS CTAs
// along the token axis extends this by log2(CS) more levels: the level-m running sums (one
// fp32 row per CTA) are combined pairwise up a tree through distributed shared memory.  Only
// the level-D sums (D = m + log2 CS, 1/2^D of the data) leave the cluster, as fp32, for the
// small kernels that finish the remaining levels.
//
// Per CTA:
//   1. one bulk asynchronous copy brings the G x K bf16 slab (contiguous in X) into shared memory
//   2. pass 1: butterflies in registers on un-normalised sums, running |.| maxima of the G-1
//      detail rows; the level-m sums go to an fp32 row in shared memory
//   3. block reduction -> per-row scale = absmax / qmax (the 2^(-j/2) factor applied to the maximum,
//      which is the maximum of the scaled values because the scaling is monotone)
//   4. pass 2: butterflies again from shared memory, 2^(-j/2), t / scale with the same
//      Newton-corrected reciprocal as the general quantizer, round-to-nearest-even by the
//      1.5 * 2^23 trick, byte / nibble packing, coalesced stores
//   5. cluster tree for levels m+1..D
#pragma once
#include "common.cuh"
#include "k_generic.cuh"
#include "ptx.cuh"

namespace stamp {

struct TqParams {
  const __nv_bfloat16* X;  // [M, K]
  int K;
  int n;           // tokens per transform block
  int levels;      // total Haar levels of the transform
  int k_hi;        // 8-bit rows per block
  int qmax_hi, qmax_lo;
  int tree_steps;  // levels handled by the cluster tree (log2 of the cluster size)
  int8_t* a8;      // [M, K] one code per int8, logical row order (GEMM operand) or nullptr
  int8_t* q_hi;    // public outputs (either may be nullptr)
  uint8_t* q_lo;
  float* x_scale;  // [M]
  float* T_out;    // [M, K] fp32 transformed values (debug export) or nullptr
  float* atop;     // [M >> D, K] un-normalised level-D sums when levels > D, else nullptr
};

constexpr int TQ_THREADS = 256;
constexpr float TQ_MAGIC = 12582912.0f;  // 1.5 * 2^23: adding it rounds to the nearest integer (ties to even)
constexpr long long TQ_WAIT_LIMIT = 2000000000LL;

__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 f2sub(float2 a, float2 b) { return __ffma2_rn(b, f2(-1.0f), a); }
__device__ __forceinline__ float2 f2amax(float2 m, float2 v) {
  return make_float2(fmaxf(m.x, fabsf(v.x)), fmaxf(m.y, fabsf(v.y)));
}
template <bool ODD>
__device__ __forceinline__ float2 mul_norm2(float2 v, const HaarNorm& h) {
  if (ODD) return __ffma2_rn(v, f2(h.hi), __fmul2_rn(v, f2(h.lo)));
  return __fmul2_rn(v, f2(h.hi));
}
// t / scale: same arithmetic as div_by_scale(), two lanes at a time
__device__ __forceinline__ float2 div2(float2 t, float scale, float inv) {
  const float2 q0 = __fmul2_rn(t, f2(inv));
  const float2 r = __ffma2_rn(q0, f2(-scale), t);
  return __ffma2_rn(r, f2(inv), q0);
}
// low byte of each word = two's complement code
__device__ __forceinline__ uint32_t pack4_s8(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}
// low nibble of a | low nibble of b << 4, in the low byte
__device__ __forceinline__ uint32_t pack2_s4(uint32_t a, uint32_t b) { return (a & 0xFu) | ((b << 4) & 0xF0u); }

struct RowOut {
  float scale, inv;
  int row;   // global logical row
  int hi;    // 1: 8-bit row
};

// Quantize CH consecutive channels (starting at channel c0) of one transformed row and store
// the codes (and optionally the fp32 values).  t holds CH/2 channel pairs.
template <int CH>
__device__ __forceinline__ void emit_codes(const TqParams& p, const RowOut& ro, int c0, const float2 (&t)[CH / 2]) {
  uint32_t b[CH];
#pragma unroll
  for (int i = 0; i < CH / 2; ++i) {
    const float2 q = __fadd2_rn(div2(t[i], ro.scale, ro.inv), f2(TQ_MAGIC));
    b[2 * i] = __float_as_uint(q.x);
    b[2 * i + 1] = __float_as_uint(q.y);
  }
  const long row = ro.row;
  if (p.T_out) {
    float2* dst = reinterpret_cast<float2*>(p.T_out + row * p.K + c0);
#pragma unroll
    for (int i = 0; i < CH / 2; ++i) dst[i] = t[i];
  }
  uint32_t w8[CH / 4];
#pragma unroll
  for (int i = 0; i < CH / 4; ++i) w8[i] = pack4_s8(b[4 * i], b[4 * i + 1], b[4 * i + 2], b[4 * i + 3]);
  if (p.a8) {
    if (CH == 8) *reinterpret_cast<uint2*>(p.a8 + row * p.K + c0) = make_uint2(w8[0], w8[CH / 4 - 1]);
    else *reinterpret_cast<uint32_t*>(p.a8 + row * p.K + c0) = w8[0];
  }
  if (p.q_hi || p.q_lo) {
    const long s = row / p.n;
    const int i = static_cast<int>(row - s * p.n);
    if (ro.hi) {
      if (p.q_hi) {
        int8_t* dst = p.q_hi + (s * p.k_hi + i) * p.K + c0;
        if (CH == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(w8[0], w8[CH / 4 - 1]);
        else *reinterpret_cast<uint32_t*>(dst) = w8[0];
      }
    } else if (p.q_lo) {
      uint8_t* dst = p.q_lo + (s * (p.n - p.k_hi) + (i - p.k_hi)) * (long)(p.K / 2) + c0 / 2;
      uint32_t w = 0;
#pragma unroll
      for (int k = 0; k < CH / 2; ++k) w |= pack2_s4(b[2 * k], b[2 * k + 1]) << (8 * k);
      if (CH == 8) *reinterpret_cast<uint32_t*>(dst) = w;
      else *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(w);
    }
  }
}

// Maximum over the CTA of a non-negative value (result valid in every thread).
__device__ __forceinline__ float block_max(float v, unsigned* red) {
  const unsigned m = __reduce_max_sync(0xffffffffu, __float_as_uint(v));
  __syncthreads();  // previous users of `red` are done
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  unsigned r = red[0];
#pragma unroll
  for (int w = 1; w < TQ_THREADS / 32; ++w) r = max(r, red[w]);
  return __uint_as_float(r);
}

__device__ __forceinline__ RowOut make_row(const TqParams& p, float amax, long row) {
  RowOut ro;
  const int i = static_cast<int>(row % p.n);
  ro.hi = i < p.k_hi;
  const float qmax = static_cast<float>(ro.hi ? p.qmax_hi : p.qmax_lo);
  ro.scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
  ro.inv = __fdiv_rn(1.0f, ro.scale);
  ro.row = static_cast<int>(row);
  return ro;
}

// Quantize one full row held as un-normalised fp32 values in shared memory (a tree-level detail
// row or the final approximation row): absmax, scale, codes.  `unnorm_max` is the CTA-wide
// maximum of |row| (already reduced).
template <bool ODD>
__device__ __forceinline__ void emit_smem_row(const TqParams& p, const float* row_s, const HaarNorm& h, float unnorm_max,
                                              long out_row) {
  const float amax = ODD ? fmaf(unnorm_max, h.hi, unnorm_max * h.lo) : unnorm_max * h.hi;
  const RowOut ro = make_row(p, amax, out_row);
  if (threadIdx.x == 0) p.x_scale[out_row] = ro.scale;
  for (int o = threadIdx.x; o < p.K / 8; o += TQ_THREADS) {
    const float4 u0 = *reinterpret_cast<const float4*>(row_s + o * 8);
    const float4 u1 = *reinterpret_cast<const float4*>(row_s + o * 8 + 4);
    float2 t[4] = {make_float2(u0.x, u0.y), make_float2(u0.z, u0.w), make_float2(u1.x, u1.y),
                   make_float2(u1.z, u1.w)};
#pragma unroll
    for (int i = 0; i < 4; ++i) t[i] = mul_norm2<ODD>(t[i], h);
    emit_codes<8>(p, ro, o * 8, t);
  }
}

__device__ __forceinline__ void emit_smem_row_dyn(const TqParams& p, const float* row_s, int level, float unnorm_max,
                                                  long out_row) {
  const HaarNorm h = haar_norm(level);
  if (level & 1) emit_smem_row<true>(p, row_s, h, unnorm_max, out_row);
  else emit_smem_row<false>(p, row_s, h, unnorm_max, out_row);
}

// In-register butterflies of G tokens x CH channels (un-normalised).  `visit(l, i, d)` receives
// every detail coefficient vector (CH/2 channel pairs) of local level l, index i; on return
// v[0] holds the level-m sums.
template <int G, int CH, typename Visit>
__device__ __forceinline__ void butterflies(float2 (&v)[G][CH / 2], Visit&& visit) {
  int l = 1;
#pragma unroll
  for (int half = G / 2; half >= 1; half >>= 1, ++l) {
#pragma unroll
    for (int i = 0; i < half; ++i) {
      float2 d[CH / 2];
#pragma unroll
      for (int c = 0; c < CH / 2; ++c) {
        d[c] = f2sub(v[2 * i][c], v[2 * i + 1][c]);
        v[i][c] = __fadd2_rn(v[2 * i][c], v[2 * i + 1][c]);
      }
      visit(l, i, d);
    }
  }
}

template <int G, int CH>
__device__ __forceinline__ void load_tile(const __nv_bfloat16* xs, int K, int c0, float2 (&v)[G][CH / 2]) {
#pragma unroll
  for (int t = 0; t < G; ++t) {
    uint32_t w[CH / 2];
    if (CH == 8) {
      const uint4 u = *reinterpret_cast<const uint4*>(xs + (long)t * K + c0);
      w[0] = u.x; w[1] = u.y; w[CH / 2 - 2] = u.z; w[CH / 2 - 1] = u.w;
    } else {
      const uint2 u = *reinterpret_cast<const uint2*>(xs + (long)t * K + c0);
      w[0] = u.x; w[1] = u.y;
    }
#pragma unroll
    for (int c = 0; c < CH / 2; ++c) v[t][c] = make_float2(__uint_as_float(w[c] << 16), __uint_as_float(w[c] & 0xFFFF0000u));
  }
}

// Shared memory: [G*K bf16 slab | K floats level-m sums | small]
template <int G>
__global__ void __launch_bounds__(TQ_THREADS) k_haar_tq(TqParams p) {
  constexpr int M_LOCAL = (G == 4) ? 2 : (G == 8) ? 3 : 4;
  constexpr int CH = (G == 16) ? 4 : 8;
  extern __shared__ __align__(16) uint8_t smem_tq[];
  const int K = p.K;
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_tq);
  float* arow = reinterpret_cast<float*>(smem_tq + (size_t)G * K * 2);
  float* drow = reinterpret_cast<float*>(smem_tq);  // reuses the slab once pass 2 is done
  uint8_t* tail = smem_tq + (size_t)G * K * 2 + (size_t)K * 4;
  uint64_t* bar = reinterpret_cast<uint64_t*>(tail);
  unsigned* red = reinterpret_cast<unsigned*>(tail + 16);            // [8]
  unsigned* red_rows = reinterpret_cast<unsigned*>(tail + 16 + 32);  // [8 warps][16 rows]
  RowOut* rows = reinterpret_cast<RowOut*>(tail + 16 + 32 + 8 * 16 * 4);  // [16]
  __shared__ uint32_t abort_word;

  const int tid = threadIdx.x;
  const long tok0 = (long)blockIdx.x * G;         // first token of this CTA
  const long s = tok0 / p.n;                      // transform block index
  const int t_in = static_cast<int>(tok0 - s * p.n);  // token offset inside the block
  const long row_base = s * p.n;

  // ---- 1. bring the slab in
  if (tid == 0) {
    abort_word = 0;
    ptx::mbar_init(bar, 1);
    ptx::fence_mbar_init();
    const uint32_t bytes = static_cast<uint32_t>((size_t)G * K * 2);
    ptx::mbar_arrive_expect_tx(bar, bytes);
    // pieces of at most 64 KB (a multiple of 16 bytes: K % 128 == 0)
    const uint8_t* src = reinterpret_cast<const uint8_t*>(p.X + tok0 * K);
    for (uint32_t off = 0; off < bytes; off += 65536u) {
      const uint32_t len = (bytes - off < 65536u) ? (bytes - off) : 65536u;
      ptx::bulk_load(smem_tq + off, src + off, len, bar);
    }
  }
  __syncthreads();
  bool ok = ptx::mbar_wait_bounded(bar, 0, &abort_word, TQ_WAIT_LIMIT);
  if (!__syncthreads_and(ok)) {
    if (tid == 0) raise_device_status(STAMP_ERR_TIMEOUT);
    // the tree below needs every CTA of the cluster at its barriers: keep going through them
    // without touching data
    ok = false;
  }

  // ---- 2. pass 1: row maxima of un-normalised details, level-m sums
  float rmax[G];
#pragma unroll
  for (int r = 0; r < G; ++r) rmax[r] = 0.f;
  if (ok) {
    for (int o = tid; o < K / CH; o += TQ_THREADS) {
      float2 v[G][CH / 2];
      load_tile<G, CH>(xs, K, o * CH, v);
      butterflies<G, CH>(v, [&](int l, int i, const float2(&d)[CH / 2]) {
        float2 m = f2(0.f);
#pragma unroll
        for (int c = 0; c < CH / 2; ++c) m = f2amax(m, d[c]);
        const int r = (G - (G >> (l - 1))) + i;
        rmax[r] = fmaxf(rmax[r], fmaxf(m.x, m.y));
      });
#pragma unroll
      for (int c = 0; c < CH / 2; ++c) *reinterpret_cast<float2*>(arow + o * CH + 2 * c) = v[0][c];
    }
  }
  // ---- 3. reduce the G-1 maxima over the CTA, build the row table
  {
    const int warp = tid >> 5;
#pragma unroll
    for (int r = 0; r < G - 1; ++r) {
      const unsigned m = __reduce_max_sync(0xffffffffu, __float_as_uint(rmax[r]));
      if ((tid & 31) == 0) red_rows[warp * 16 + r] = m;
    }
    __syncthreads();
    if (tid < G - 1) {
      unsigned m = red_rows[tid];
#pragma unroll
      for (int w = 1; w < TQ_THREADS / 32; ++w) m = max(m, red_rows[w * 16 + tid]);
      // local row tid -> (level l, index i)
      int l = 1, base = 0;
      while (tid >= base + (G >> l)) {
        base += G >> l;
        ++l;
      }
      const int i = tid - base;
      const HaarNorm h = haar_norm(l);
      const float um = __uint_as_float(m);
      const float amax = (l & 1) ? fmaf(um, h.hi, um * h.lo) : um * h.hi;
      const long row = row_base + (p.n >> l) + (t_in >> l) + i;
      const RowOut ro = make_row(p, amax, row);
      rows[tid] = ro;
      if (ok) p.x_scale[row] = ro.scale;
    }
    __syncthreads();
  }
  // ---- 4. pass 2: recompute, normalise, quantize, store
  if (ok) {
    for (int o = tid; o < K / CH; o += TQ_THREADS) {
      float2 v[G][CH / 2];
      load_tile<G, CH>(xs, K, o * CH, v);
      butterflies<G, CH>(v, [&](int l, int i, const float2(&d)[CH / 2]) {
        const int r = (G - (G >> (l - 1))) + i;
        const HaarNorm h = haar_norm(l);
        float2 t[CH / 2];
#pragma unroll
        for (int c = 0; c < CH / 2; ++c) t[c] = (l & 1) ? mul_norm2<true>(d[c], h) : mul_norm2<false>(d[c], h);
        emit_codes<CH>(p, rows[r], o * CH, t);
      });
    }
  }

  // ---- 5. cluster tree: levels m+1 .. m+tree_steps, then the level-D sums
  const uint32_t rank = (p.tree_steps > 0) ? ptx::cluster_ctarank() : 0u;
  const uint32_t arow_addr = ptx::smem_u32(arow);
  for (int step = 0; step < p.tree_steps; ++step) {
    ptx::cluster_sync();  // partner's sums are complete and visible; everyone is done with the slab
    const int level = M_LOCAL + step + 1;
    if ((rank & ((2u << step) - 1u)) == 0u && ok) {
      const uint32_t partner = ptx::mapa(arow_addr, rank + (1u << step));
      float m = 0.f;
      for (int i = tid; i < K / 4; i += TQ_THREADS) {
        const float4 a = *reinterpret_cast<const float4*>(arow + 4 * i);
        const float4 b = ptx::ld_dsmem_f4(partner + 16u * i);
        const float4 d = make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
        *reinterpret_cast<float4*>(drow + 4 * i) = d;
        *reinterpret_cast<float4*>(arow + 4 * i) = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(d.x), fabsf(d.y))), fmaxf(fabsf(d.z), fabsf(d.w)));
      }
      m = block_max(m, red);
      emit_smem_row_dyn(p, drow, level, m, row_base + (p.n >> level) + (t_in >> level));
    }
  }
  if (p.tree_steps > 0) ptx::cluster_sync();  // nobody leaves while a partner may still read its sums
  if (rank == 0 && ok) {
    const int D = M_LOCAL + p.tree_steps;
    if (p.levels == D) {
      float m = 0.f;
      for (int i = tid; i < K / 4; i += TQ_THREADS) {
        const float4 a = *reinterpret_cast<const float4*>(arow + 4 * i);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(a.x), fabsf(a.y))), fmaxf(fabsf(a.z), fabsf(a.w)));
      }
      m = block_max(m, red);
      emit_smem_row_dyn(p, arow, D, m, row_base + (t_in >> D));
    } else if (p.atop) {
      float4* dst = reinterpret_cast<float4*>(p.atop + (tok0 >> D) * K);
      __syncthreads();
      for (int i = tid; i < K / 4; i += TQ_THREADS) dst[i] = *reinterpret_cast<const float4*>(arow + 4 * i);
    }
  }
}

template <int G>
constexpr size_t tq_smem_bytes(int K) {
  return (size_t)G * K * 2 + (size_t)K * 4 + 16 + 32 + 8 * 16 * 4 + 16 * sizeof(RowOut);
}

}  // namespace stamp
