// Fused Haar transform + per-token mixed-precision quantizer for bf16 activations, one pass over X in HBM
// (Algorithm 1: the sequence transform of the activations and their per-token quantizer; Sec. "Efficient Energy
// Concentration").
//
// Why this shape.  The quantizer needs, per transformed token, the maximum over ALL channels before it can
// code any of them, while a Haar coefficient needs a run of tokens of ONE channel.  On the CUDA cores alone the
// pass spends about 12 instructions per element (unpack, butterflies, shuffles for the row maxima, tables) and
// has to park every coefficient in registers while the maxima are exchanged: it ends up bound by instruction
// issue at well under half of the HBM bandwidth.  Here the two things the SM has besides its CUDA cores carry
// that load:
//   * the tensor cores apply up to seven Haar levels to a tile of 128 tokens x 128 channels as ONE product
//     D = H X, where H (128 x 128, entries 0 / +1 / -1: the un-normalised Haar analysis matrix) is exact in
//     bf16 and lives in tensor memory (64 columns: the product reads it as a tensor-memory operand, which leaves
//     the whole shared memory to the activation tiles), X is bf16 as it lies in HBM (TMA, consumed as an MN-major
//     operand: nothing is transposed), and the accumulation is fp32.  The 2^(-j/2) factors are applied afterwards
//     exactly as the butterfly kernel does;
//   * the activation tile stays in shared memory (32 KB of bf16) while the row maxima travel, and the product
//     is simply issued again when they are back -- 4 us of tensor time per GB of activations, on a pipe that has
//     nothing else to do in this pass -- so that no warp parks a coefficient in registers across the exchange
//     and the ring of seven tiles, not the register file, sets how many tiles can be waiting.  Tensor memory
//     (lane = transformed token, column = channel) holds H and the three accumulators in flight.
// An epilogue thread owns ONE transformed token of the tile: its maximum over the tile's channels is a
// thread-local reduction, and later its scale, bit width and destination row are per-thread constants.  What
// is left for the CUDA cores is about 5 instructions per element.
//
// Row maxima across the feature axis.  A tile covers 128 channels; the K / 128 tiles of a 128-token row block
// are consecutive work items, taken at about the same time by neighbouring CTAs of the persistent grid.
//   job P1(item): product -> four warps of their own (one per quarter of the accumulator's lanes) reduce |D| per
//                 lane over the tile's 128 columns and leave the 128 maxima in shared memory; a publisher warp
//                 combines them into the row block's table in global memory (atomicMax) and, once they are
//                 delivered, counts the tile in (two publishers alternate);
//   job P2(item): HTC_LAG items later the MMA thread waits (bounded) until the row block's count is complete,
//                 issues the product again into the accumulator of one of two sets of quantizing warps, and
//                 these read the final maxima, derive scale, bit width and destination of their row, quantize
//                 and store the codes.
// The warps that take the maxima do nothing else, so a tile's maxima leave the SM a few hundred clocks after its
// first product and never queue behind a quantizing pass.  A CTA only ever waits for P1 jobs of items that
// precede or accompany its own in the global item order, and a P1 job needs nothing but a ring stage and an
// accumulator freed by jobs further back, so the waits cannot form a cycle as long as every CTA of the grid is
// resident (one CTA per SM, grid <= number of SMs) and a row block has no more tiles than the grid has CTAs.
//
// Levels above the seventh continue on the un-normalised 128-token sums (1/128 of the data, fp32) in the
// butterfly kernel (k_haar_cq), which also serves fp32 activations and shapes this kernel does not take.
#pragma once
#include "common.cuh"
#include "k_haar_cq.cuh"
#include "ptx.cuh"
#include <type_traits>

namespace stamp {

struct HtcParams {
  int K;             // channels, a multiple of 128
  int n;             // tokens per transform block, a multiple of 128
  int n_shift;       // log2 n when n is a power of two, else -1
  int lv;            // Haar levels applied here, 1..7 (2^lv <= n)
  int last;          // 1: lv is the transform's depth, the approximation rows are quantized here
                     // 0: (lv == 7) the 128-token sums go to aout, un-normalised, for the next launch
  int k_hi;          // 8-bit rows per transform block
  float qmax_hi, qmax_lo;
  long ntiles;       // row blocks of 128 tokens: M / 128
  int nchunks;       // tiles per row block: K / 128
  unsigned* rowmax;  // [M] zero on entry: bit patterns of the per-row maxima, indexed row block * 128 + lane
  unsigned* cnt;     // [M / 128] zero on entry: tiles of a row block whose maxima have been sent
  float* aout;       // [M / 128, K]
  int8_t* a8;        // HTC_OUT_A8 / HTC_OUT_TILED: [M, K] one code per int8 (GEMM operand)
  int8_t* q_hi;      // HTC_OUT_PUBLIC: packed public outputs
  uint8_t* q_lo;
  float* x_scale;    // [M] logical order (A8, PUBLIC)
  float* T_out;      // HTC_OUT_T: [M, K] transformed values, fp32 (debug export)
  float* sx_epi;     // HTC_OUT_TILED: [M] scale * 2^(-j/2) of every tile row, indexed like a8
  // fold != 0: the levels above the seventh are finished by this kernel's tail (logical-order outputs only), in
  // strips of 128 channels (1) or 64 channels (2)
  int fold;
  int levels;        // depth of the whole transform (fold)
  int nseq;          // transform blocks: M / n (fold)
  unsigned* done;    // [1] zero on entry: CTAs whose 128-token sums are written
  unsigned* rowmax2; // [M / 128] zero on entry: maxima of the coarse rows, block * (n / 128) + logical row
  unsigned* cnt2;    // [nseq] zero on entry: strips of a block whose coarse maxima have been sent
  const uint8_t* pf_base;   // optional region to pull towards L2 (the layer's weight codes), pf_bytes % 16 == 0
  long pf_bytes;
};

enum HtcOut { HTC_OUT_A8 = 0, HTC_OUT_PUBLIC = 1, HTC_OUT_T = 2, HTC_OUT_TILED = 3 };

// warps: 0 TMA producer, 1 MMA issuer, 2-3 publishers, then HTC_QSETS sets of eight quantizing warps, then 4 maxima warps
constexpr int HTC_QSETS = 2;
constexpr int HTC_MAXW0 = 4 + 8 * HTC_QSETS;          // first maxima warp
constexpr int HTC_THREADS = (HTC_MAXW0 + 4) * 32;
constexpr int HTC_STAGES = 7;                         // shared-memory ring of activation tiles
constexpr int HTC_H_COL = 128 * (1 + HTC_QSETS);      // H as a tensor-memory operand: 64 columns after the accumulators
constexpr int HTC_LAG = 4;                 // items between the two products of a tile (< HTC_STAGES)
constexpr int HTC_NBUF = 4;                // 128-column accumulators in tensor memory: one for P1 jobs, one per quantizing set
constexpr int HTC_TILE_BYTES = 128 * 128 * 2;   // [128 tokens x 128 channels] bf16 = two 64-channel atoms
constexpr int HTC_ATOM_BYTES = 128 * 128;       // [128 tokens x 64 channels] bf16
constexpr int HTC_BAR_OFFSET = HTC_STAGES * HTC_TILE_BYTES;
constexpr int HTC_NUM_BARS = 2 * HTC_STAGES + 2 * HTC_NBUF + 4;   // ring, accumulators (full / empty), pfull[2], pempty[2]
constexpr int HTC_SLOT_OFFSET = HTC_BAR_OFFSET + HTC_NUM_BARS * 8 + 16;   // [2 sets][128 lanes] maxima on their way out
constexpr int HTC_DYN_BYTES = HTC_SLOT_OFFSET + 2 * 128 * 4 + 1024;
constexpr uint32_t HTC_NIB_BIAS = 0x3F400000u;     // sum over i < 8 of 0x4B400000 << 4 i, modulo 2^32 (see the 4-bit packing)
constexpr long long HTC_WAIT_LIMIT = 4000000000LL;   // SM clocks (~2 s) before a wait gives up

// bf16 A (K-major) x bf16 B (MN-major) -> fp32, M = 128, N = 128
__host__ __device__ constexpr uint32_t htc_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(128 >> 3) << 17) |
         (static_cast<uint32_t>(128 >> 4) << 24);
}

// D (+)= A B with A read from tensor memory (lane = row of A, two bf16 per 32-bit column: 16 tokens = 8 columns)
__device__ __forceinline__ void htc_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(htc_idesc()), "r"(accumulate)
      : "memory");
}

// MN-major operand: rows (= K index = token) of 128 bytes (64 channels), 128-byte swizzle, 8-row groups 1024
// bytes apart; the second 64-channel atom lies HTC_ATOM_BYTES further.
__device__ __forceinline__ uint64_t htc_bdesc(uint32_t smem_addr_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr_bytes >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>(HTC_ATOM_BYTES >> 4) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Lane r of a tile holds, for lv levels: the approximation values a_lv[r] for r < 128 >> lv, else the detail
// d_j[r - (128 >> j)] of the level j with 128 >> j <= r < 128 >> (j - 1)  (band order [a | d_lv | ... | d_1]).
__device__ __forceinline__ void htc_lane_row(int lv, int r, int& j, int& idx, bool& approx) {
  if (r < (128 >> lv)) {
    j = lv;
    idx = r;
    approx = true;
  } else {
    j = 7 - (31 - __clz(r));
    idx = r - (128 >> j);
    approx = false;
  }
}

// Clears the row-maximum table and the tile counts before k_haar_tc.  A kernel rather than a memset, so that both
// launches can be programmatic dependents: this one's launch overlaps the tail of whatever ran before (it waits for
// that to complete before it writes), and k_haar_tc sets up its barriers, tensor memory and H while this one runs.
__global__ void __launch_bounds__(256) k_htc_clear(uint4* __restrict__ words16, long n16) {
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (long)gridDim.x * blockDim.x)
    words16[i] = make_uint4(0u, 0u, 0u, 0u);
}

template <int OUT>
__global__ void __launch_bounds__(HTC_THREADS, 1) k_haar_tc(const __grid_constant__ CUtensorMap tmap_x, const HtcParams p) {
  extern __shared__ uint8_t htc_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(htc_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* b_sm = smem;                              // ring of activation tiles
  uint64_t* sfull = reinterpret_cast<uint64_t*>(smem + HTC_BAR_OFFSET);
  uint64_t* sempty = sfull + HTC_STAGES;
  uint64_t* tfull = sempty + HTC_STAGES;
  uint64_t* tempty = tfull + HTC_NBUF;
  uint64_t* pfull = tempty + HTC_NBUF;
  uint64_t* pempty = pfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pempty + 2);
  volatile uint32_t* abort_word = tmem_slot + 1;
  unsigned* pslot = reinterpret_cast<unsigned*>(smem + HTC_SLOT_OFFSET);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // item numbers fit 32 bits (checked by the host): the per-tile index arithmetic below is 32-bit on purpose
  const unsigned nitems = static_cast<unsigned>(p.ntiles) * static_cast<unsigned>(p.nchunks);
  const int n_local = nitems > blockIdx.x ? static_cast<int>((nitems - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;   // this CTA's items
  const unsigned nchunks = static_cast<unsigned>(p.nchunks);

  if (threadIdx.x == 0) {
    for (int s = 0; s < HTC_STAGES; ++s) {
      ptx::mbar_init(&sfull[s], 1);
      ptx::mbar_init(&sempty[s], 1);
    }
    for (int b = 0; b < HTC_NBUF; ++b) {
      ptx::mbar_init(&tfull[b], 1);
      ptx::mbar_init(&tempty[b], b == 0 ? 4 * 32 : 8 * 32);   // the four maxima warps / the eight warps of a quantizing set
    }
    for (int q = 0; q < 2; ++q) {
      ptx::mbar_init(&pfull[q], 4 * 32);
      ptx::mbar_init(&pempty[q], 32);
    }
    *abort_word = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // H into tensor memory: thread = row r of H (its lane), column c = tokens 2 c (low half) and 2 c + 1 (high half)
  if (warp >= 4 && warp < 8) {
    const int r = (warp & 3) * 32 + lane;
    int j, idx;
    bool approx;
    htc_lane_row(p.lv, r, j, idx, approx);
    const int first = idx << j, mid = first + (1 << j) / 2, end = first + (1 << j);
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + HTC_H_COL;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t w[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        uint32_t pair = 0;
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          const int t = 2 * (16 * g + c) + s2;
          uint32_t v = 0;
          if (t >= first && t < end) v = (approx || t < mid) ? 0x3F80u : 0xBF80u;   // +1.0 / -1.0 in bf16
          pair |= v << (16 * s2);
        }
        w[c] = pair;
      }
      ptx::tmem_st_32x32b_x16(taddr + 16 * g, w);
    }
    ptx::tmem_st_wait();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 0 && p.pf_bytes > 0) {   // fire-and-forget hints, 8 KB each
    constexpr long PF_CHUNK = 8192;
    const long nchunk = (p.pf_bytes + PF_CHUNK - 1) / PF_CHUNK;
    for (long c = (long)blockIdx.x * 32 + lane; c < nchunk; c += (long)gridDim.x * 32) {
      const long off = c * PF_CHUNK;
      const long left = p.pf_bytes - off;
      ptx::prefetch_l2_bulk(p.pf_base + off, static_cast<uint32_t>(left < PF_CHUNK ? left : PF_CHUNK));
    }
  }
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();   // the next kernel may set itself up on SMs as they fall free; it still waits for this grid to finish

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      for (unsigned item = blockIdx.x; item < nitems; item += gridDim.x) {
        const unsigned rb = item / nchunks;
        const int c = static_cast<int>(item - rb * nchunks);
        if (!ptx::mbar_wait_bounded_sleepy(&sempty[stage], phase ^ 1u, abort_word, HTC_WAIT_LIMIT)) {
          ok = false;
          break;
        }
        uint8_t* dst = b_sm + stage * HTC_TILE_BYTES;
        ptx::mbar_arrive_expect_tx(&sfull[stage], HTC_TILE_BYTES);
        ptx::tma_load_2d(dst, &tmap_x, &sfull[stage], c * 128, static_cast<int>(rb * 128u));
        ptx::tma_load_2d(dst + HTC_ATOM_BYTES, &tmap_x, &sfull[stage], c * 128 + 64, static_cast<int>(rb * 128u));
        armed |= 1u << stage;
        armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
        if (++stage == HTC_STAGES) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
        for (int s = 0; s < HTC_STAGES; ++s)   // let copies in flight land before the shared memory goes away
          if (armed & (1u << s)) {
            const long long t0 = clock64();
            while (!ptx::mbar_try_wait(&sfull[s], (armed_parity >> s) & 1u) && clock64() - t0 < 2000000LL) {
            }
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // Static order: P1 of item t, then P2 of item t - HTC_LAG.  Accumulator 0 for a P1 job, 1 + i % HTC_QSETS for
    // the P2 job of item i (the quantizing set i % HTC_QSETS drains it).
    if (ptx::elect_one()) {
      bool ok = true;
      // D = H X of the tile in ring stage `stage` into accumulator `buf`, whose `use`-th filling this is; the
      // second product of a tile also hands the stage back to the producer
      auto product = [&](int stage, int buf, int use, bool release_stage) -> bool {
        if (!ptx::mbar_wait_bounded_sleepy(&tempty[buf], static_cast<uint32_t>((use & 1) ^ 1), abort_word, HTC_WAIT_LIMIT)) return false;
        ptx::tc_fence_after();
        const uint32_t bbase = ptx::smem_u32(b_sm + stage * HTC_TILE_BYTES);
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * 128);
#pragma unroll
        for (int k = 0; k < 8; ++k) {   // 16 tokens per instruction
          const uint64_t bdesc = htc_bdesc(bbase + k * 16 * 128);
          htc_mma_ts(tmem_d, tmem_base + HTC_H_COL + 8 * k, bdesc, k != 0 ? 1u : 0u);   // 16 tokens = 8 columns of H
        }
        if (release_stage) ptx::tc_commit(&sempty[stage]);
        ptx::tc_commit(&tfull[buf]);
        return true;
      };
      for (int t = 0; t < n_local + HTC_LAG && ok; ++t) {
        if (t < n_local) {   // P1 of item t
          const int stage = t % HTC_STAGES;
          if (!ptx::mbar_wait_bounded_sleepy(&sfull[stage], static_cast<uint32_t>((t / HTC_STAGES) & 1), abort_word, HTC_WAIT_LIMIT) ||
              !product(stage, 0, t, false)) {
            ok = false;
            break;
          }
        }
        if (t >= HTC_LAG) {  // P2 of item t - HTC_LAG: its row block's maxima must be complete
          const int i = t - HTC_LAG;
          const unsigned rb = (blockIdx.x + static_cast<unsigned>(i) * gridDim.x) / nchunks;
          const long long t0 = clock64();
          unsigned spins = 0;
          while (ld_acquire_gpu(p.cnt + rb) < nchunks) {
            if ((++spins & 15u) == 0u && (*abort_word != 0u || clock64() - t0 > HTC_WAIT_LIMIT)) {
              ok = false;
              break;
            }
            __nanosleep(20);
          }
          if (!ok || !product(i % HTC_STAGES, 1 + i % HTC_QSETS, i / HTC_QSETS, true)) {
            ok = false;
            break;
          }
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------------ publisher warps (items of one parity each)
    // Takes a tile's 128 lane maxima out of shared memory, sends them to the row block's table and, once they
    // are delivered, counts the tile in.
    const int set = warp - 2;
    bool ok = true;
    for (int i = set; i < n_local; i += 2) {
      const unsigned rb = (blockIdx.x + static_cast<unsigned>(i) * gridDim.x) / nchunks;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&pfull[set], static_cast<uint32_t>((i >> 1) & 1), abort_word, HTC_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      unsigned m[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) m[q] = pslot[set * 128 + q * 32 + lane];
      ptx::mbar_arrive(&pempty[set]);      // the slot may be written again
#pragma unroll
      for (int q = 0; q < 4; ++q) atomicMax(p.rowmax + (size_t)rb * 128 + q * 32 + lane, m[q]);
      // Counting the tile in is a release at GPU scope: whoever reads the complete count with an acquire load also
      // sees the maxima (the other lanes' atomics are ordered before lane 0's release by the warp barrier).  The
      // release costs less than a full fence between the atomics and a relaxed count (164 against 168 us on
      // 32768 x 8192 tokens x channels).
      __syncwarp();
      if (lane == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.cnt + rb) : "memory");
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  } else if (warp >= HTC_MAXW0) {
    // ------------------------------------------------------------------ maxima warps: one per quarter of the lanes
    // P1 of every item: |D| of this thread's lane over the tile's 128 columns, left in the slot of the item's
    // parity for the publisher.  The accumulator is released as soon as its values are in registers.
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    bool ok = true;
    for (int i = 0; i < n_local; ++i) {
      const int slot = i & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&tfull[0], static_cast<uint32_t>(i & 1), abort_word, HTC_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      uint32_t v[2][16];
      float m0 = 0.f, m1 = 0.f;
      ptx::tmem_ld_32x32b_x16(taddr, v[0]);
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        ptx::tmem_ld_wait();
        if (ch < 7) ptx::tmem_ld_32x32b_x16(taddr + 16 * (ch + 1), v[(ch + 1) & 1]);
        const uint32_t(&x)[16] = v[ch & 1];
#pragma unroll
        for (int q = 0; q < 16; q += 2) {
          m0 = fmaxf(m0, fabsf(__uint_as_float(x[q])));
          m1 = fmaxf(m1, fabsf(__uint_as_float(x[q + 1])));
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[0]);
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&pempty[slot], static_cast<uint32_t>(((i >> 1) & 1) ^ 1), abort_word, HTC_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      pslot[slot * 128 + r] = __float_as_uint(fmaxf(m0, m1));
      ptx::mbar_arrive(&pfull[slot]);
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  } else {
    // ------------------------------------------------------------------ quantizing warps
    // Two sets of eight warps take the CTA's items in turn; inside a set a warp owns the 32 lanes of its
    // quarter (warp % 4) and 64 of the tile's 128 columns, a thread ONE transformed token: scale, bit width and
    // destination row are per-thread scalars, and a thread's 64 codes are 32 or 64 contiguous bytes of its row.
    const int e = warp - 4;
    const int set = e >> 3;
    const int quarter = warp & 3;
    const int half = (e >> 2) & 1;
    const int r = quarter * 32 + lane;
    int j, idx;
    bool approx;
    htc_lane_row(p.lv, r, j, idx, approx);
    const bool raw = approx && !p.last;        // the 128-token sum: handed on un-normalised
    const bool odd = (j & 1) != 0;
    const bool warp_has_odd = __any_sync(0xffffffffu, odd);   // false: no lane of the warp needs the 1/sqrt 2 factor
    const float pw = __int_as_float((127 - (j >> 1)) << 23);      // 2^(-(j >> 1))
    const float2 nhi = odd ? make_float2(CQ_RSQRT2_HI, CQ_RSQRT2_HI) : make_float2(1.f, 1.f);
    const float2 nlo = odd ? make_float2(CQ_RSQRT2_LO, CQ_RSQRT2_LO) : make_float2(0.f, 0.f);
    const unsigned K = static_cast<unsigned>(p.K);
    const unsigned n = static_cast<unsigned>(p.n);
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>((1 + set) * 128 + half * 64);
    bool ok = true;
    // (row block, tile inside it) of the set's items, advanced without a division per item
    const unsigned item0 = blockIdx.x + static_cast<unsigned>(set) * gridDim.x;
    unsigned rb = item0 / nchunks;
    unsigned cu = item0 - rb * nchunks;
    const unsigned step_rb = (HTC_QSETS * gridDim.x) / nchunks, step_c = HTC_QSETS * gridDim.x - step_rb * nchunks;

    for (int i = set; i < n_local && ok; i += HTC_QSETS, rb += step_rb, cu += step_c) {
      if (cu >= nchunks) {
        cu -= nchunks;
        ++rb;
      }
      // where this lane's row goes (the tile's tokens are [128 rb, 128 rb + 128)); rows and row pitches fit 32 bits
      const unsigned tok0 = rb * 128u;
      const unsigned blk = p.n_shift >= 0 ? tok0 >> p.n_shift : tok0 / n;
      const unsigned off = tok0 - blk * n;
      const unsigned ib = (off >> j) + idx;                         // index inside the block at level j
      const unsigned i_in_blk = approx ? ib : (n >> j) + ib;        // logical row inside the block
      const bool hi = i_in_blk < static_cast<unsigned>(p.k_hi);
      const float qmax = hi ? p.qmax_hi : p.qmax_lo;
      const unsigned row = blk * n + i_in_blk;
      const unsigned col0 = cu * 128u + half * 64u;
      uint8_t* dst = nullptr;       // this lane's 64 channels of its row
      bool four_bit = false;
      size_t scale_at = 0;          // where this lane reports its scale (one lane of the row block's first tile)
      float* scale_to = p.x_scale;
      if (raw) {
        dst = reinterpret_cast<uint8_t*>(p.aout) + ((size_t)rb * K + col0) * 4;
      } else if (OUT == HTC_OUT_T) {
        dst = reinterpret_cast<uint8_t*>(p.T_out) + ((size_t)row * K + col0) * 4;
      } else if (OUT == HTC_OUT_PUBLIC) {
        if (hi) {
          dst = reinterpret_cast<uint8_t*>(p.q_hi) + (size_t)(blk * p.k_hi + i_in_blk) * K + col0;
        } else {
          dst = p.q_lo + (size_t)(blk * (n - p.k_hi) + (i_in_blk - p.k_hi)) * (K >> 1) + (col0 >> 1);
          four_bit = true;
        }
        scale_at = row;
      } else if (OUT == HTC_OUT_A8) {
        dst = reinterpret_cast<uint8_t*>(p.a8) + (size_t)row * K + col0;
        scale_at = row;
      } else {
        // tile order of the GEMM's fused inverse (see k_haar_cq.cuh): 256-token tiles
        const unsigned tile = (blk * n + (ib << j)) >> 8;
        const int i_loc = static_cast<int>(ib & ((256u >> j) - 1u));
        const int tcol = approx ? 32 * i_loc : cq_tile_col_detail(j, i_loc);
        const unsigned prow = tile * 256u + tcol;
        dst = reinterpret_cast<uint8_t*>(p.a8) + (size_t)prow * K + col0;
        scale_at = prow;
        scale_to = p.sx_epi;
      }
      // a warp whose 32 rows all take 4-bit codes (the common case) packs nibbles only
      const bool all_four = __all_sync(0xffffffffu, four_bit && !raw);
      // the MMA thread issued this product after it saw the row block's count complete: the table is final
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&tfull[1 + set], static_cast<uint32_t>((i / HTC_QSETS) & 1), abort_word, HTC_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      uint32_t v[2][16];
      ptx::tmem_ld_32x32b_x16(taddr, v[0]);
      const float u = __uint_as_float(ld_relaxed_gpu(p.rowmax + (size_t)rb * 128 + r));
      const float amax = odd ? fmaf(u, CQ_RSQRT2_HI, u * CQ_RSQRT2_LO) : u;      // in units of 2^(-(j >> 1))
      const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
      const float inv = __fdiv_rn(1.0f, scale);
      const float true_scale = (amax > 0.f) ? scale * pw : 1.0f;
      const float2 inv2 = make_float2(inv, inv), ns2 = make_float2(-scale, -scale);
      // Rounding by adding 1.5 * 2^23: the sum's low mantissa bits are the two's complement code.  A 4-bit row adds 8
      // more, so that its low nibble is the code + 8 in [1, 15] and nothing above it changes: eight such words
      // combine into eight nibbles with shifts and adds alone, and one XOR takes the 8 out of every nibble again.
      const float magic = four_bit ? CQ_MAGIC + 8.0f : CQ_MAGIC;
      const float2 magic2 = make_float2(magic, magic);
      if (cu == 0 && half == 0 && !raw && OUT != HTC_OUT_T)
        scale_to[scale_at] = (OUT == HTC_OUT_TILED) ? true_scale * (odd ? pw * CQ_RSQRT2_HI : pw) : true_scale;

      // One chunk of 16 columns: x -> 16 codes (or values).  Codes collect in `pend` until they fill a 32-byte
      // sector of the row (64 four-bit codes: the whole pass; 32 eight-bit codes: two chunks), which then leaves
      // in one store: a warp's store touches 32 different rows, so the fewer pieces per row the better.
      // MIXED: the warp's rows differ in kind (raw sum, 8-bit, 4-bit).  Every lane then runs the same
      // instructions -- both packings, selected per lane, and predicated stores -- instead of the kinds taking
      // turns through the whole chunk.
      uint32_t pend[8];
      auto chunk = [&](const uint32_t(&x)[16], auto ch_tag, auto norm_tag, auto mixed_tag) {
        constexpr int ch = decltype(ch_tag)::value;
        constexpr bool NORM = decltype(norm_tag)::value;
        constexpr bool MIXED = decltype(mixed_tag)::value;
        if (MIXED && raw) {
          ptx::st_global_v8(dst + ch * 64, x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
          ptx::st_global_v8(dst + ch * 64 + 32, x[8], x[9], x[10], x[11], x[12], x[13], x[14], x[15]);
        }
        uint32_t bits[16];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float2 raw2 = make_float2(__uint_as_float(x[2 * g]), __uint_as_float(x[2 * g + 1]));
          // 2^(-j/2) = c * 2^(-(j >> 1)): only c touches the data, head + tail so the product is rounded once
          const float2 t = NORM ? __ffma2_rn(raw2, nhi, __fmul2_rn(raw2, nlo)) : raw2;
          if (OUT == HTC_OUT_T) {
            bits[2 * g] = __float_as_uint(t.x * pw);
            bits[2 * g + 1] = __float_as_uint(t.y * pw);
          } else {
            const float2 q0 = __fmul2_rn(t, inv2);
            const float2 rem = __ffma2_rn(q0, ns2, t);
            const float2 q = __fadd2_rn(__ffma2_rn(rem, inv2, q0), magic2);
            bits[2 * g] = __float_as_uint(q.x);
            bits[2 * g + 1] = __float_as_uint(q.y);
          }
        }
        if (OUT == HTC_OUT_T) {
          if (!raw) {
            ptx::st_global_v8(dst + ch * 64, bits[0], bits[1], bits[2], bits[3], bits[4], bits[5], bits[6], bits[7]);
            ptx::st_global_v8(dst + ch * 64 + 32, bits[8], bits[9], bits[10], bits[11], bits[12], bits[13], bits[14], bits[15]);
          }
          return;
        }
        // 4-bit: word = sum_i (0x4B400000 | u_i) << 4 i  (mod 2^32), u_i the code + 8; the constant part of the sum
        // is HTC_NIB_BIAS; low nibble = even channel.  Two interleaved chains (even / odd nibbles).
        uint32_t w4[2];
        if (OUT == HTC_OUT_PUBLIC) {
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            uint32_t ev = bits[8 * h2 + 6], od = bits[8 * h2 + 7];
#pragma unroll
            for (int k = 2; k >= 0; --k) {
              ev = (ev << 8) + bits[8 * h2 + 2 * k];
              od = (od << 8) + bits[8 * h2 + 2 * k + 1];
            }
            w4[h2] = ((od << 4) + ev - HTC_NIB_BIAS) ^ 0x88888888u;
          }
        }
        if (OUT == HTC_OUT_PUBLIC && !MIXED) {
          pend[2 * ch] = w4[0];
          pend[2 * ch + 1] = w4[1];
          if (ch == 3) ptx::st_global_v8(dst, pend[0], pend[1], pend[2], pend[3], pend[4], pend[5], pend[6], pend[7]);
          return;
        }
        // 8-bit: the low byte of each word is the two's complement code
        uint32_t w8[4];
#pragma unroll
        for (int g = 0; g < 4; ++g)
          w8[g] = __byte_perm(__byte_perm(bits[4 * g], bits[4 * g + 1], 0x0040), __byte_perm(bits[4 * g + 2], bits[4 * g + 3], 0x0040), 0x5410);
        if (OUT != HTC_OUT_PUBLIC) {   // GEMM operand: every row one code per byte
          if (ch & 1) {
            if (!raw) ptx::st_global_v8(dst + 32 * (ch >> 1), pend[0], pend[1], pend[2], pend[3], w8[0], w8[1], w8[2], w8[3]);
          } else {
#pragma unroll
            for (int g = 0; g < 4; ++g) pend[g] = w8[g];
          }
          return;
        }
        // public format, mixed warp: an 8-bit lane fills pend[0..3], then stores with this chunk's words at odd
        // chunks; a 4-bit lane fills pend[2 ch], pend[2 ch + 1] and stores after the last chunk
        if (ch & 1) {
          if (!raw && !four_bit) ptx::st_global_v8(dst + 32 * (ch >> 1), pend[0], pend[1], pend[2], pend[3], w8[0], w8[1], w8[2], w8[3]);
          pend[2 * ch] = w4[0];
          pend[2 * ch + 1] = w4[1];
        } else {
          if (ch == 0) {
#pragma unroll
            for (int g = 0; g < 4; ++g) pend[g] = four_bit ? (g < 2 ? w4[g] : 0u) : w8[g];
          } else {   // ch == 2: a 4-bit lane keeps pend[0..3] (chunks 0, 1) and adds pend[4..5]; an 8-bit lane restarts
            pend[4] = w4[0];
            pend[5] = w4[1];
#pragma unroll
            for (int g = 0; g < 4; ++g) pend[g] = four_bit ? pend[g] : w8[g];
          }
        }
        if (ch == 3 && !raw && four_bit) ptx::st_global_v8(dst, pend[0], pend[1], pend[2], pend[3], pend[4], pend[5], pend[6], pend[7]);
      };
      const bool mixed = (OUT == HTC_OUT_PUBLIC) ? !all_four : __any_sync(0xffffffffu, raw);
      auto step = [&](auto ch_tag) {
        constexpr int ch = decltype(ch_tag)::value;
        ptx::tmem_ld_wait();
        if (ch < 3) {
          ptx::tmem_ld_32x32b_x16(taddr + 16 * (ch + 1), v[(ch + 1) & 1]);
        } else {
          ptx::tc_fence_before();
          ptx::mbar_arrive(&tempty[1 + set]);   // every value of the accumulator is in registers: it may be refilled
        }
        if (mixed)
          chunk(v[ch & 1], ch_tag, std::true_type{}, std::true_type{});
        else if (warp_has_odd)
          chunk(v[ch & 1], ch_tag, std::true_type{}, std::false_type{});
        else
          chunk(v[ch & 1], ch_tag, std::false_type{}, std::false_type{});
      };
      step(std::integral_constant<int, 0>{});
      step(std::integral_constant<int, 1>{});
      step(std::integral_constant<int, 2>{});
      step(std::integral_constant<int, 3>{});
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  }

  // ------------------------------------------------------------------ tail: the levels above the seventh
  // The 128-token sums of a block (n / 128 rows x K, fp32, 1 / 128 of the data) are what the deeper levels work on.
  // When they fit the shared memory that the ring no longer needs, the CTAs finish the transform themselves
  // instead of leaving it to one or two more launches: a CTA takes (block, 128-channel strip) items, loads the
  // strip's sums, runs the remaining levels in place (after level l the sums sit at rows that are multiples of
  // 2^(l+1), the details of that level at the odd multiples of 2^l: every pair writes back to the two rows it
  // read), exchanges the maxima of the coarse rows exactly as above (table, release count, bounded acquire
  // wait) and quantizes them with the arithmetic of the quantizing warps.
  if (p.fold) {
    __syncthreads();   // every role is through: this CTA's sums are written
    float* S = reinterpret_cast<float*>(b_sm);
    volatile uint32_t* tail_ok = abort_word + 1;
    const int R = p.n >> 7, lr = p.levels - 7;
    // strips of 128 channels, or of 64 when that gives more CTAs something to do (sh = log2 of float4 per strip row)
    const int sh = p.fold == 2 ? 4 : 5, sw4 = 1 << sh;
    const unsigned nstrips = static_cast<unsigned>(p.K >> (sh + 2));
    if (threadIdx.x == 0) {
      asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.done) : "memory");
      bool ok = (*abort_word == 0u);
      const long long t0 = clock64();
      unsigned spins = 0;
      while (ok && ld_acquire_gpu(p.done) < gridDim.x) {
        if ((++spins & 15u) == 0u && clock64() - t0 > HTC_WAIT_LIMIT) ok = false;
        __nanosleep(100);
      }
      if (!ok) raise_device_status(STAMP_ERR_TIMEOUT);
      *tail_ok = ok ? 1u : 0u;
    }
    __syncthreads();
    bool ok = (*tail_ok != 0u);
    const unsigned ntail = static_cast<unsigned>(p.nseq) * nstrips;
    const int K = p.K;
    for (unsigned it = blockIdx.x; it < ntail && ok; it += gridDim.x) {
      const unsigned blk = it / nstrips;
      const unsigned c = it - blk * nstrips;
      // (1) the strip's sums: R rows x 4 sw4 channels
      for (int e0 = threadIdx.x; e0 < (R << sh); e0 += 4 * HTC_THREADS) {   // four loads in flight per thread
        float4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int e = e0 + k * HTC_THREADS;
          if (e < (R << sh))   // other CTAs wrote the sums: read past L1
            v[k] = __ldcg(reinterpret_cast<const float4*>(p.aout + ((size_t)blk * R + (e >> sh)) * K + ((c << sh) + (e & (sw4 - 1))) * 4u));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int e = e0 + k * HTC_THREADS;
          if (e < (R << sh)) reinterpret_cast<float4*>(S)[e] = v[k];
        }
      }
      __syncthreads();
      // (2) remaining levels on un-normalised sums, in place
      for (int l = 0; l < lr; ++l) {
        const int npairs = R >> (l + 1);
        for (int e = threadIdx.x; e < (npairs << sh); e += HTC_THREADS) {   // four channels at a time
          const int i = e >> sh, q = e & (sw4 - 1);
          float4* a = reinterpret_cast<float4*>(S) + ((i << (l + 1)) << sh) + q;
          float4* b = a + (sw4 << l);
          const float4 x0 = *a, x1 = *b;
          *a = make_float4(x0.x + x1.x, x0.y + x1.y, x0.z + x1.z, x0.w + x1.w);
          *b = make_float4(x0.x - x1.x, x0.y - x1.y, x0.z - x1.z, x0.w - x1.w);
        }
        __syncthreads();
      }
      // (3) maxima of the strip's rows (un-normalised, as in the main loop), one warp per row
      // (a warp takes one row of 128 channels or two rows of 64: R is even)
      const int rpw = 32 >> sh, sub = lane >> sh, ln = lane & (sw4 - 1);
      const unsigned submask = sh == 5 ? 0xffffffffu : (0xffffu << (16 * sub));
      for (int row0 = warp * rpw; row0 < R; row0 += (HTC_THREADS / 32) * rpw) {
        const int row = row0 + sub;
        const float4 v = reinterpret_cast<const float4*>(S)[(row << sh) + ln];
        const float m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
        const unsigned mm = __reduce_max_sync(submask, __float_as_uint(m));
        if (ln == 0) atomicMax(p.rowmax2 + (size_t)blk * R + row, mm);   // indexed by the row in S
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.cnt2 + blk) : "memory");
        const long long t0 = clock64();
        unsigned spins = 0;
        bool got = true;
        while (ld_acquire_gpu(p.cnt2 + blk) < nstrips) {
          if ((++spins & 15u) == 0u && clock64() - t0 > HTC_WAIT_LIMIT) {
            got = false;
            break;
          }
          __nanosleep(100);
        }
        if (!got) raise_device_status(STAMP_ERR_TIMEOUT);
        *tail_ok = got ? 1u : 0u;
      }
      __syncthreads();
      ok = (*tail_ok != 0u);
      if (!ok) break;
      // the block's final maxima, once, behind the strip (one load per row here instead of one round trip per row below)
      // every row's level, destination, scale and reciprocal, one thread per row (the two divisions of all rows run
      // side by side here instead of one after the other in the loop below)
      float4* srow = reinterpret_cast<float4*>(S) + ((size_t)R << sh);   // {scale, 1 / scale, scale as stored, level | hi << 8}
      for (int row = threadIdx.x; row < R; row += HTC_THREADS) {
        int j, lrow;
        if ((row & ((1 << lr) - 1)) == 0) {
          j = p.levels;
          lrow = row >> lr;
        } else {
          const int tz = __ffs(row) - 1;
          j = 8 + tz;
          lrow = (p.n >> j) + (row >> (tz + 1));
        }
        const bool hi = lrow < p.k_hi;
        const float qmax = hi ? p.qmax_hi : p.qmax_lo;
        const float u = __uint_as_float(ld_relaxed_gpu(p.rowmax2 + (size_t)blk * R + row));
        const float amax = (j & 1) ? fmaf(u, CQ_RSQRT2_HI, u * CQ_RSQRT2_LO) : u;
        const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
        const float pw = __int_as_float((127 - (j >> 1)) << 23);      // 2^(-(j >> 1))
        srow[row] = make_float4(scale, __fdiv_rn(1.0f, scale), (amax > 0.f) ? scale * pw : 1.0f,
                                __int_as_float(j | (hi ? 256 : 0) | (lrow << 9)));
      }
      __syncthreads();
      // (4) quantize, one warp per row, a lane four channels
      for (int row0 = warp * rpw; row0 < R; row0 += (HTC_THREADS / 32) * rpw) {
        const int row = row0 + sub;
        const float4 sr = srow[row];
        const float scale = sr.x, inv = sr.y, true_scale = sr.z;
        const int tag = __float_as_int(sr.w);
        const int j = tag & 255, lrow = tag >> 9;
        const bool hi = (tag & 256) != 0, odd = (j & 1) != 0;
        const float pw = __int_as_float((127 - (j >> 1)) << 23);      // 2^(-(j >> 1))
        const float4 v = reinterpret_cast<const float4*>(S)[(row << sh) + ln];
        const float raw4[4] = {v.x, v.y, v.z, v.w};
        const size_t grow = (size_t)blk * p.n + lrow;     // logical row of the whole problem
        const unsigned col = ((c << sh) + ln) * 4u;
        if (OUT == HTC_OUT_T) {
          float o[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) o[k] = (odd ? fmaf(raw4[k], CQ_RSQRT2_HI, raw4[k] * CQ_RSQRT2_LO) : raw4[k]) * pw;
          *reinterpret_cast<float4*>(p.T_out + grow * K + col) = make_float4(o[0], o[1], o[2], o[3]);
          continue;
        }
        uint32_t code[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float t = odd ? fmaf(raw4[k], CQ_RSQRT2_HI, raw4[k] * CQ_RSQRT2_LO) : raw4[k];
          const float q0 = t * inv;
          const float rem = fmaf(q0, -scale, t);
          code[k] = __float_as_uint(fmaf(rem, inv, q0) + CQ_MAGIC);   // low byte: the two's complement code
        }
        if (OUT == HTC_OUT_PUBLIC && !hi) {
          const uint32_t b0 = (code[0] & 0xFu) | ((code[1] & 0xFu) << 4), b1 = (code[2] & 0xFu) | ((code[3] & 0xFu) << 4);
          *reinterpret_cast<uint16_t*>(p.q_lo + ((size_t)blk * (p.n - p.k_hi) + (lrow - p.k_hi)) * (size_t)(K >> 1) + (col >> 1)) =
              static_cast<uint16_t>(b0 | (b1 << 8));
        } else {
          const uint32_t w = (code[0] & 0xFFu) | ((code[1] & 0xFFu) << 8) | ((code[2] & 0xFFu) << 16) | (code[3] << 24);
          int8_t* base8 = (OUT == HTC_OUT_PUBLIC) ? p.q_hi + ((size_t)blk * p.k_hi + lrow) * (size_t)K : p.a8 + grow * (size_t)K;
          *reinterpret_cast<uint32_t*>(base8 + col) = w;
        }
        if (c == 0 && ln == 0) p.x_scale[grow] = true_scale;
      }
      __syncthreads();   // S is loaded again for the CTA's next item
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace stamp
