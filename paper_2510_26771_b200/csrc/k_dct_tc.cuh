// Blockwise 256-point DCT-II along the token axis on the tensor cores (Sec. "Efficient Energy
// Concentration": the DCT as energy-compacting sequence transform; configuration with blocks of 256
// tokens).  Per transform block the transform is the dense product  T = C X  (C the orthonormal
// 256 x 256 DCT-II matrix, X the block's 256 tokens x channels), a real contraction over tokens.
//
// Precision.  The activations are bf16, i.e. exact tensor-core operands.  C is split into three
// bf16 terms C = C1 + C2 + C3 (24 significant bits), so  C X = C1 X + C2 X + C3 X  accumulated in
// fp32 in tensor memory reproduces an fp32 evaluation of the transform: every product is exact and
// only the accumulation rounds.  (The inverse, used on the layer's output where 1e-3 is asked for,
// takes the output as two bf16 planes hi + lo and the three largest cross terms.)
//
// The token axis is the contraction axis, and tokens are the slow axis in memory.  Nothing is
// transposed: the activation tile [256 tokens x 64 channels] lands in shared memory by TMA exactly
// as it lies in HBM (rows = tokens, 128-byte swizzle) and is consumed as an "MN-major" B operand
// (transpose bit of the instruction descriptor); C's terms are K-major A operands streamed from L2.
//
//   D[u, ch] (TMEM lane = frequency u, column = channel) = sum_s sum_t Cs[s][u][t] * B_plane(s)[t][ch]
//
// A thread of the epilogue therefore owns one transformed token: its absolute maximum over the
// tile's channels is thread-local.  Since a token's scale needs ALL channels and a tile has 128,
// the forward transform runs twice: launch 1 only takes the row maxima (atomicMax into a table),
// launch 2 recomputes the product and quantizes with the final scales.  That costs the tensor
// work twice but moves no fp32 intermediate through HBM.
//
// Structure (as the integer GEMM): persistent CTAs, warp 0 = TMA producer, warp 1 = TMEM owner and
// MMA issuer, warps 2-5 = epilogue; two accumulator buffers so the epilogue overlaps the next tile.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

enum DctTcMode { DCT_TC_MAX = 0, DCT_TC_QUANT = 1, DCT_TC_INVERSE = 2 };

struct DctTcParams {
  int nblk;              // transform blocks of 256 tokens
  int cols;              // channels (K forward, N inverse)
  int k_hi;              // 8-bit rows per block
  float qmax_hi, qmax_lo;
  unsigned* rowmax;      // [nblk * 256] bit patterns of per-row maxima
  int8_t* a8;            // [nblk * 256, cols] codes (DCT_TC_QUANT)
  float* x_scale;        // [nblk * 256]
  void* y;               // [nblk * 256, cols] output of the inverse, float or bf16
  int y_bf16;
  const float* bias;     // [cols] or nullptr (inverse)
  int nterms;            // products accumulated per tile: 3 for the DCT; the Walsh-Hadamard matrix (+-1/16) is one
                         // exact bf16 term, so 1 forward and 2 (hi and lo plane) for its inverse
};

constexpr int DCT_N = 256;                 // block length
constexpr int DCT_THREADS = 192;
constexpr int DCT_A_STAGES = 3;
constexpr int DCT_A_BYTES = 256 * 128;     // [256 rows x 64 bf16]
constexpr int DCT_ATOM_BYTES = 256 * 128;  // [256 tokens x 64 channels bf16]
constexpr long long DCT_WAIT_LIMIT = 4000000000LL;

// Instruction descriptor for kind::f16: bf16 A (K-major) and B (MN-major), fp32 accumulation.
__host__ __device__ constexpr uint32_t make_bf16_idesc_bmn(int m, int n) {
  return (1u << 4)                           // D format: f32
         | (1u << 7)                         // A format: bf16
         | (1u << 10)                        // B format: bf16
         | (1u << 16)                        // B is MN-major (channels contiguous)
         | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Shared-memory descriptor of an MN-major operand tile stored as rows (= K index) of 128 bytes
// (64 bf16 along MN) with the 128-byte swizzle, 8-row groups 1024 bytes apart; a wider operand is
// several such [256 x 64] atoms, DCT_ATOM_BYTES apart (the descriptor's MN-direction stride).
__device__ __forceinline__ uint64_t make_mnmajor_sw128_desc(uint32_t smem_addr_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr_bytes >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>(DCT_ATOM_BYTES >> 4) << 16;  // stride between 64-wide atoms along MN
  d |= static_cast<uint64_t>(1024 >> 4) << 32;            // stride between 8-row groups along K
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;                    // SWIZZLE_128B
  return d;
}

template <int NATOM, int NPLANE>
struct DctSmem {
  static constexpr int B_BYTES = NPLANE * NATOM * DCT_ATOM_BYTES;       // one tile's B operand
  static constexpr int A_OFFSET = 2 * B_BYTES;
  static constexpr int BAR_OFFSET = A_OFFSET + DCT_A_STAGES * DCT_A_BYTES;
  // afull[3], aempty[3], bfull[2], bempty[2], tfull[2], tempty[2], then tmem base + abort word
  static constexpr int NUM_BARS = 2 * DCT_A_STAGES + 8;
  static constexpr int TOTAL = BAR_OFFSET + NUM_BARS * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
  static constexpr int ACC_COLS = 2 * NATOM * 64;                        // two halves of 128 frequencies
};

// term -> (which split of the matrix, which plane of B)
template <int MODE>
__device__ __forceinline__ void dct_term(int term, int nterms, int& split, int& plane) {
  if (MODE == DCT_TC_INVERSE) {
    // three terms: C1 hi, C2 hi, C1 lo;  two terms (single-term matrix): C1 hi, C1 lo
    split = (nterms == 3 && term == 1) ? 1 : 0;
    plane = (term == nterms - 1) ? 1 : 0;
  } else {
    split = term;
    plane = 0;
  }
}

template <int MODE, int NATOM, int NPLANE>
__global__ void __launch_bounds__(DCT_THREADS, 1)
    k_dct_tc(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b0,
             const __grid_constant__ CUtensorMap tmap_b1, DctTcParams p) {
  using SM = DctSmem<NATOM, NPLANE>;
  extern __shared__ uint8_t dct_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dct_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* afull = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFFSET);
  uint64_t* aempty = afull + DCT_A_STAGES;
  uint64_t* bfull = aempty + DCT_A_STAGES;
  uint64_t* bempty = bfull + 2;
  uint64_t* tfull = bempty + 2;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile uint32_t* abort_word = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int nstrips = p.cols / (NATOM * 64);
  const int num_tiles = p.nblk * nstrips;

  if (threadIdx.x == 0) {
    for (int s = 0; s < DCT_A_STAGES; ++s) {
      ptx::mbar_init(&afull[s], 1);
      ptx::mbar_init(&aempty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&bfull[b], 1);
      ptx::mbar_init(&bempty[b], 1);
      ptx::mbar_init(&tfull[b], 1);
      ptx::mbar_init(&tempty[b], 128);
    }
    *abort_word = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b0);
    ptx::prefetch_tensormap(&tmap_b1);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::grid_dependency_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      int st = 0;
      uint32_t aphase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int blk = tile / nstrips, strip = tile - blk * nstrips;
        const int bb = it & 1;
        const uint32_t bphase = (it >> 1) & 1u;
        if (!ptx::mbar_wait_bounded(&bempty[bb], bphase ^ 1u, abort_word, DCT_WAIT_LIMIT)) { ok = false; break; }
        uint8_t* bdst = smem + bb * SM::B_BYTES;
        ptx::mbar_arrive_expect_tx(&bfull[bb], SM::B_BYTES);
#pragma unroll
        for (int pl = 0; pl < NPLANE; ++pl)
#pragma unroll
          for (int a = 0; a < NATOM; ++a)
            ptx::tma_load_2d(bdst + (pl * NATOM + a) * DCT_ATOM_BYTES, pl == 0 ? &tmap_b0 : &tmap_b1, &bfull[bb],
                             (strip * NATOM + a) * 64, blk * DCT_N);
        for (int term = 0; term < p.nterms && ok; ++term) {
          int split, plane;
          dct_term<MODE>(term, p.nterms, split, plane);
          for (int tb = 0; tb < 4; ++tb) {
            if (!ptx::mbar_wait_bounded(&aempty[st], aphase ^ 1u, abort_word, DCT_WAIT_LIMIT)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&afull[st], DCT_A_BYTES);
            ptx::tma_load_2d(smem + SM::A_OFFSET + st * DCT_A_BYTES, &tmap_a, &afull[st], tb * 64, split * DCT_N);
            if (++st == DCT_A_STAGES) { st = 0; aphase ^= 1u; }
          }
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
        const long long t0 = clock64();   // let copies in flight land before the shared memory goes away
        while (clock64() - t0 < 4000000LL) {
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
      // one MMA spans all NATOM 64-channel atoms of the tile (the descriptor's MN stride = one atom)
      constexpr uint32_t idesc = make_bf16_idesc_bmn(128, 64 * NATOM);
      int st = 0;
      uint32_t aphase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int bb = it & 1;
        const uint32_t ph = (it >> 1) & 1u;
        if (!ptx::mbar_wait_bounded(&bfull[bb], ph, abort_word, DCT_WAIT_LIMIT) ||
            !ptx::mbar_wait_bounded(&tempty[bb], ph ^ 1u, abort_word, DCT_WAIT_LIMIT)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t bbase = ptx::smem_u32(smem + bb * SM::B_BYTES);
        const uint32_t dbase = tmem_base + static_cast<uint32_t>(bb * SM::ACC_COLS);
        for (int term = 0; term < p.nterms && ok; ++term) {
          int split, plane;
          dct_term<MODE>(term, p.nterms, split, plane);
          for (int tb = 0; tb < 4; ++tb) {
            if (!ptx::mbar_wait_bounded(&afull[st], aphase, abort_word, DCT_WAIT_LIMIT)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t abase = ptx::smem_u32(smem + SM::A_OFFSET + st * DCT_A_BYTES);
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const uint64_t adesc = ptx::make_kmajor_sw128_desc(abase + h * (128 * 128) + k * 32);
                const uint64_t bdesc = make_mnmajor_sw128_desc(bbase + plane * NATOM * DCT_ATOM_BYTES + (tb * 64 + k * 16) * 128);
                mma_bf16_ss(dbase + h * (NATOM * 64), adesc, bdesc, idesc, (term | tb | k) != 0 ? 1u : 0u);
              }
            ptx::tc_commit(&aempty[st]);
            if (++st == DCT_A_STAGES) { st = 0; aphase ^= 1u; }
          }
        }
        if (ok) {
          ptx::tc_commit(&tfull[bb]);
          ptx::tc_commit(&bempty[bb]);
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;              // TMEM lanes 32 * (warp % 4) ...
    const int rloc = quarter * 32 + lane;      // frequency inside a half
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int blk = tile / nstrips, strip = tile - blk * nstrips;
      const int bb = it & 1;
      const uint32_t ph = (it >> 1) & 1u;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(&tfull[bb], ph, abort_word, DCT_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      const int col0 = strip * NATOM * 64;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int u = h * 128 + rloc;
        const long row = (long)blk * DCT_N + u;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                               static_cast<uint32_t>(bb * SM::ACC_COLS + h * NATOM * 64);
        float scale = 1.f, inv = 1.f;
        if (MODE == DCT_TC_QUANT) {
          const float amax = __uint_as_float(__ldcg(p.rowmax + row));
          const float qmax = (u < p.k_hi) ? p.qmax_hi : p.qmax_lo;
          scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
          inv = __fdiv_rn(1.0f, scale);
          if (strip == 0) p.x_scale[row] = scale;
        }
        float m = 0.f;
#pragma unroll
        for (int chunk = 0; chunk < NATOM * 2; ++chunk) {
          uint32_t r[32];
          ptx::tmem_ld_32x32b_x32(taddr + chunk * 32, r);
          ptx::tmem_ld_wait();
          if (MODE == DCT_TC_MAX) {
#pragma unroll
            for (int j = 0; j < 32; ++j) m = fmaxf(m, fabsf(__uint_as_float(r[j])));
          } else if (MODE == DCT_TC_QUANT) {
            uint32_t w[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              uint32_t b[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float t = __uint_as_float(r[4 * g + e]);
                const float q0 = t * inv;
                const float q = fmaf(fmaf(-q0, scale, t), inv, q0);   // t / scale, Newton-corrected
                b[e] = __float_as_uint(q + 12582912.0f);               // round to nearest even
              }
              w[g] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
            }
            uint4* dst = reinterpret_cast<uint4*>(p.a8 + row * p.cols + col0 + chunk * 32);
            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            const float* bias = p.bias ? p.bias + col0 + chunk * 32 : nullptr;
            if (p.y_bf16) {
              uint32_t w[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const float v0 = __uint_as_float(r[2 * j]) + (bias ? __ldg(bias + 2 * j) : 0.f);
                const float v1 = __uint_as_float(r[2 * j + 1]) + (bias ? __ldg(bias + 2 * j + 1) : 0.f);
                const __nv_bfloat162 pk = __floats2bfloat162_rn(v0, v1);
                w[j] = *reinterpret_cast<const uint32_t*>(&pk);
              }
              uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.y) + row * p.cols + col0 + chunk * 32);
#pragma unroll
              for (int j = 0; j < 4; ++j) dst[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            } else {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.y) + row * p.cols + col0 + chunk * 32);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                dst[j] = make_float4(__uint_as_float(r[4 * j]) + (bias ? __ldg(bias + 4 * j) : 0.f),
                                     __uint_as_float(r[4 * j + 1]) + (bias ? __ldg(bias + 4 * j + 1) : 0.f),
                                     __uint_as_float(r[4 * j + 2]) + (bias ? __ldg(bias + 4 * j + 2) : 0.f),
                                     __uint_as_float(r[4 * j + 3]) + (bias ? __ldg(bias + 4 * j + 3) : 0.f));
            }
          }
        }
        if (MODE == DCT_TC_MAX) atomicMax(p.rowmax + row, __float_as_uint(m));
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[bb]);
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// The three bf16 terms of the orthonormal 256-point DCT-II matrix, as A operands:
//   out[(s * 256 + r) * 256 + k] = term s of  C[r][k]  (forward: rows = frequencies)
//                                  or of      C[k][r]  (transpose = inverse: rows = tokens)
// wht != 0: the sequency-ordered Walsh-Hadamard matrix instead (entries +-1/16: term 1 is exact, the others 0).
__global__ void __launch_bounds__(256) k_dct_split_matrix(int transpose, int wht, __nv_bfloat16* __restrict__ out) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= DCT_N * DCT_N) return;
  const int r = idx / DCT_N, k = idx - r * DCT_N;
  const int u = transpose ? k : r, t = transpose ? r : k;
  double c;
  if (wht) {
    c = wht_sign(u, t, 8) * 0.0625;
  } else {
    const long a = ((long)(2 * t + 1) * u) % (4L * DCT_N);
    const double cu = (u == 0) ? 0.70710678118654752440 : 1.0;
    c = cu * sqrt(2.0 / DCT_N) * cospi(static_cast<double>(a) / (2.0 * DCT_N));
  }
#pragma unroll
  for (int s = 0; s < 3; ++s) {
    const __nv_bfloat16 h = __double2bfloat16(c);
    out[(size_t)s * DCT_N * DCT_N + idx] = h;
    c -= static_cast<double>(__bfloat162float(h));
  }
}

}  // namespace stamp
