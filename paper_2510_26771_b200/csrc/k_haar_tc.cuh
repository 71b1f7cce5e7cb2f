// Fused Haar transform + per-token mixed-precision quantizer for bf16 activations, one pass over X in HBM
// (Algorithm lines "X <- L X" and "x_i <- Q(x_i; b_i)"; Sec. "Efficient Energy Concentration").
//
// Why this shape.  The quantizer needs, per transformed token, the maximum over ALL channels before it can
// code any of them, while a Haar coefficient needs a run of tokens of ONE channel.  On the CUDA cores alone the
// pass spends about 12 instructions per element (unpack, butterflies, shuffles for the row maxima, tables) and
// has to park every coefficient in registers while the maxima are exchanged: it ends up bound by instruction
// issue at well under half of the HBM bandwidth.  Here the two things the SM has besides its CUDA cores carry
// that load:
//   * the tensor cores apply up to seven Haar levels to a tile of 128 tokens x 128 channels as ONE product
//     D = H X, where H (128 x 128, entries 0 / +1 / -1: the un-normalised Haar analysis matrix) is exact in
//     bf16, X is bf16 as it lies in HBM (TMA, consumed as an MN-major operand: nothing is transposed), and the
//     accumulation is fp32.  The 2^(-j/2) factors are applied afterwards exactly as the butterfly kernel does;
//   * the activation tile stays in shared memory (32 KB of bf16) while the row maxima travel, and the product
//     is simply issued again when they are back -- 4 us of tensor time per GB of activations, on a pipe that has
//     nothing else to do in this pass -- so that no warp parks a coefficient in registers across the exchange
//     and the ring of six tiles, not the register file, sets how many tiles can be waiting.  Tensor memory
//     (lane = transformed token, column = channel) only holds the four accumulators in flight.
// An epilogue thread owns ONE transformed token of the tile: its maximum over the tile's channels is a
// thread-local reduction, and later its scale, bit width and destination row are per-thread constants.  What
// is left for the CUDA cores is about 5 instructions per element.
//
// Row maxima across the feature axis.  A tile covers 128 channels; the K / 128 tiles of a 128-token row block
// are consecutive work items, taken at about the same time by neighbouring CTAs of the persistent grid.
//   job P1(item): product -> the epilogue warps reduce |D| per lane over the tile's columns and combine the
//                 result into the row block's table in global memory (atomicMax), then count themselves in;
//   job P2(item): HTC_LAG items later the MMA thread waits (bounded) until the row block's count is complete,
//                 issues the product again, and the epilogue warps read the final maxima, derive scale, bit
//                 width and destination of their row, quantize the accumulator and store the codes.
// Sending the maxima and counting the tile in is the job of two publisher warps: the fence between the two
// waits about a microsecond for the atomics to be delivered, which an epilogue warp cannot afford.  A CTA only ever waits for P1 jobs of items that
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

namespace stamp {

struct HtcParams {
  int K;             // channels, a multiple of 128
  int n;             // tokens per transform block (power of two)
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
  const uint8_t* pf_base;   // optional region to pull towards L2 (the layer's weight codes), pf_bytes % 16 == 0
  long pf_bytes;
};

enum HtcOut { HTC_OUT_A8 = 0, HTC_OUT_PUBLIC = 1, HTC_OUT_T = 2, HTC_OUT_TILED = 3 };

constexpr int HTC_THREADS = 20 * 32;       // TMA warp, MMA warp, two sets of eight epilogue warps, two publisher warps
constexpr int HTC_STAGES = 6;              // shared-memory ring of activation tiles
constexpr int HTC_LAG = 4;                 // items between the two products of a tile (even: both jobs go to one warp set)
constexpr int HTC_NBUF = 4;                // 128-column accumulators in tensor memory
constexpr int HTC_TILE_BYTES = 128 * 128 * 2;   // [128 tokens x 128 channels] bf16 = two 64-channel atoms
constexpr int HTC_ATOM_BYTES = 128 * 128;       // [128 tokens x 64 channels] bf16
constexpr int HTC_A_BYTES = 128 * 128 * 2;      // H: [128 rows x 128 tokens] bf16 = two 64-token atoms
constexpr int HTC_BAR_OFFSET = HTC_A_BYTES + HTC_STAGES * HTC_TILE_BYTES;
constexpr int HTC_NUM_BARS = 2 * HTC_STAGES + 2 * HTC_NBUF + 4;   // + pfull[2], pempty[2]
constexpr int HTC_SLOT_OFFSET = HTC_BAR_OFFSET + HTC_NUM_BARS * 8 + 16;   // [2 sets][128 lanes] maxima on their way out
constexpr int HTC_DYN_BYTES = HTC_SLOT_OFFSET + 2 * 128 * 4 + 1024;
constexpr long long HTC_WAIT_LIMIT = 4000000000LL;   // SM clocks (~2 s) before a wait gives up

// bf16 A (K-major) x bf16 B (MN-major) -> fp32, M = 128, N = 128
__host__ __device__ constexpr uint32_t htc_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(128 >> 3) << 17) |
         (static_cast<uint32_t>(128 >> 4) << 24);
}

__device__ __forceinline__ void htc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(htc_idesc()), "r"(accumulate)
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

template <int OUT>
__global__ void __launch_bounds__(HTC_THREADS, 1) k_haar_tc(const __grid_constant__ CUtensorMap tmap_x, const HtcParams p) {
  extern __shared__ uint8_t htc_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(htc_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_sm = smem;                              // H
  uint8_t* b_sm = smem + HTC_A_BYTES;                // ring of activation tiles
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
  const long nitems = p.ntiles * p.nchunks;
  const long n_local = nitems > blockIdx.x ? (nitems - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;   // this CTA's items

  // ---- the analysis matrix, written straight into the K-major 128-byte-swizzled operand layout:
  // element (row r, token t) of atom t / 64 sits in 16-byte chunk ((t % 64) / 8) ^ (r % 8) of row r
  for (int e = threadIdx.x; e < 128 * 16; e += HTC_THREADS) {
    const int r = e >> 4, c16 = e & 15;              // row, 8-token group
    int j, idx;
    bool approx;
    htc_lane_row(p.lv, r, j, idx, approx);
    const int first = idx << j, mid = first + (1 << j) / 2, end = first + (1 << j);
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      uint32_t pair = 0;
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        const int t = c16 * 8 + 2 * h + s;
        uint32_t v = 0;
        if (t >= first && t < end) v = (approx || t < mid) ? 0x3F80u : 0xBF80u;   // +1.0 / -1.0 in bf16
        pair |= v << (16 * s);
      }
      w[h] = pair;
    }
    const int atom = c16 >> 3, chunk = (c16 & 7) ^ (r & 7);
    *reinterpret_cast<uint4*>(a_sm + atom * HTC_ATOM_BYTES + r * 128 + chunk * 16) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  if (threadIdx.x < 256) pslot[threadIdx.x] = 0u;
  if (threadIdx.x == 0) {
    for (int s = 0; s < HTC_STAGES; ++s) {
      ptx::mbar_init(&sfull[s], 1);
      ptx::mbar_init(&sempty[s], 1);
    }
    for (int b = 0; b < HTC_NBUF; ++b) {
      ptx::mbar_init(&tfull[b], 1);
      ptx::mbar_init(&tempty[b], 8 * 32);   // the eight warps of the set that drains the accumulator
    }
    for (int q = 0; q < 2; ++q) {
      ptx::mbar_init(&pfull[q], 8 * 32);
      ptx::mbar_init(&pempty[q], 32);
    }
    *abort_word = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_x);
  }
  ptx::fence_proxy_async_smem();   // H was written with ordinary stores; the tensor cores read it through the async proxy
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
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

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      for (long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long rb = item / p.nchunks;
        const int c = static_cast<int>(item - rb * p.nchunks);
        if (!ptx::mbar_wait_bounded_sleepy(&sempty[stage], phase ^ 1u, abort_word, HTC_WAIT_LIMIT)) {
          ok = false;
          break;
        }
        uint8_t* dst = b_sm + stage * HTC_TILE_BYTES;
        ptx::mbar_arrive_expect_tx(&sfull[stage], HTC_TILE_BYTES);
        ptx::tma_load_2d(dst, &tmap_x, &sfull[stage], c * 128, static_cast<int>(rb * 128));
        ptx::tma_load_2d(dst + HTC_ATOM_BYTES, &tmap_x, &sfull[stage], c * 128 + 64, static_cast<int>(rb * 128));
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
    if (ptx::elect_one()) {
      bool ok = true;
      const uint32_t abase = ptx::smem_u32(a_sm);
      const unsigned target = static_cast<unsigned>(p.nchunks);
      long job = 0;
      // D = H X of the tile in ring stage `stage` into the accumulator of job `job`; the last product of a tile
      // also hands the stage back to the producer
      auto product = [&](int stage, bool release_stage) -> bool {
        const int buf = static_cast<int>(job & (HTC_NBUF - 1));
        if (!ptx::mbar_wait_bounded_sleepy(&tempty[buf], static_cast<uint32_t>(((job / HTC_NBUF) & 1) ^ 1), abort_word, HTC_WAIT_LIMIT))
          return false;
        ptx::tc_fence_after();
        const uint32_t bbase = ptx::smem_u32(b_sm + stage * HTC_TILE_BYTES);
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * 128);
#pragma unroll
        for (int k = 0; k < 8; ++k) {   // 16 tokens per instruction
          const uint64_t adesc = ptx::make_kmajor_sw128_desc(abase + (k >> 2) * HTC_ATOM_BYTES + (k & 3) * 32);
          const uint64_t bdesc = htc_bdesc(bbase + k * 16 * 128);
          htc_mma(tmem_d, adesc, bdesc, k != 0 ? 1u : 0u);
        }
        if (release_stage) ptx::tc_commit(&sempty[stage]);
        ptx::tc_commit(&tfull[buf]);
        ++job;
        return true;
      };
      for (long t = 0; t < n_local + HTC_LAG && ok; ++t) {
        if (t < n_local) {   // P1 of item t
          const int stage = static_cast<int>(t % HTC_STAGES);
          if (!ptx::mbar_wait_bounded_sleepy(&sfull[stage], static_cast<uint32_t>((t / HTC_STAGES) & 1), abort_word, HTC_WAIT_LIMIT) ||
              !product(stage, false)) {
            ok = false;
            break;
          }
        }
        if (t >= HTC_LAG) {  // P2 of item t - HTC_LAG: its row block's maxima must be complete
          const long i = t - HTC_LAG;
          const long rb = (blockIdx.x + i * gridDim.x) / p.nchunks;
          const long long t0 = clock64();
          unsigned spins = 0;
          while (ld_acquire_gpu(p.cnt + rb) < target) {
            if ((++spins & 15u) == 0u && (*abort_word != 0u || clock64() - t0 > HTC_WAIT_LIMIT)) {
              ok = false;
              break;
            }
            __nanosleep(20);
          }
          if (!ok || !product(static_cast<int>(i % HTC_STAGES), true)) {
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
  } else if (warp >= 18) {
    // ------------------------------------------------------------------ publisher warps (one per epilogue set)
    // Takes the lane maxima a set has gathered for a tile out of shared memory, sends them to the row block's
    // table and, once they are delivered (the fence), counts the tile in.  The wait for the delivery -- about a
    // microsecond under load -- is all this warp does, so it stalls nobody.
    const int set = warp - 18;
    bool ok = true;
    long k = 0;
    for (long i = set; i < n_local; i += 2, ++k) {
      const long rb = (blockIdx.x + i * gridDim.x) / p.nchunks;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&pfull[set], static_cast<uint32_t>(k & 1), abort_word, HTC_WAIT_LIMIT))) {
        ok = false;
        break;
      }
      unsigned m[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        m[q] = pslot[set * 128 + q * 32 + lane];
        pslot[set * 128 + q * 32 + lane] = 0u;
      }
      ptx::mbar_arrive(&pempty[set]);      // the slot is clear again
#pragma unroll
      for (int q = 0; q < 4; ++q) atomicMax(p.rowmax + rb * 128 + q * 32 + lane, m[q]);
      __threadfence();
      __syncwarp();
      if (lane == 0) atomicAdd(p.cnt + rb, 1u);
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    // Two sets of eight warps take the CTA's items alternately (both jobs of an item go to the same set); inside
    // a set a warp owns the 32 lanes of its quarter (warp % 4) and 64 of the tile's 128 columns.  A warp's jobs
    // alternate: P1 of item i (lane maxima of its columns, handed to the set's publisher warp), then P2 of item
    // i - HTC_LAG (scale, codes, stores) -- each waits for the accumulator the MMA thread fills for it.
    const int e = warp - 2;
    const int set = e >> 3;
    const int quarter = warp & 3;
    const int half = (e >> 2) & 1;
    const int r = quarter * 32 + lane;
    int j, idx;
    bool approx;
    htc_lane_row(p.lv, r, j, idx, approx);
    const bool raw = approx && !p.last;        // the 128-token sum: handed on un-normalised
    const bool odd = (j & 1) != 0;
    const float pw = __int_as_float((127 - (j >> 1)) << 23);      // 2^(-(j >> 1))
    const float2 nhi = odd ? make_float2(CQ_RSQRT2_HI, CQ_RSQRT2_HI) : make_float2(1.f, 1.f);
    const float2 nlo = odd ? make_float2(CQ_RSQRT2_LO, CQ_RSQRT2_LO) : make_float2(0.f, 0.f);
    const int K = p.K;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(half * 64);
    bool ok = true;

    // job index of the two products of local item i in the MMA thread's issue order
    auto job_p1 = [&](long i) -> long { return i + (i > HTC_LAG ? i - HTC_LAG : 0); };
    auto job_p2 = [&](long i) -> long { return i + HTC_LAG < n_local ? 2 * i + HTC_LAG + 1 : n_local + i; };
    auto wait_acc = [&](long jb) -> bool {
      const int buf = static_cast<int>(jb & (HTC_NBUF - 1));
      const bool got = __all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&tfull[buf], static_cast<uint32_t>((jb / HTC_NBUF) & 1),
                                                                      abort_word, HTC_WAIT_LIMIT));
      ptx::tc_fence_after();
      return got;
    };

    // P2 of local item i
    auto pass2 = [&](long i) -> bool {
      const long item = blockIdx.x + i * gridDim.x;
      const long rb = item / p.nchunks;
      const int c = static_cast<int>(item - rb * p.nchunks);
      const long jb = job_p2(i);
      const int buf = static_cast<int>(jb & (HTC_NBUF - 1));
      // where this lane's row goes (all per-thread scalars; the tile's tokens are [128 rb, 128 rb + 128))
      const long tok0 = rb * 128;
      const long blk = tok0 / p.n;
      const int off = static_cast<int>(tok0 - blk * p.n);
      const int ib = (off >> j) + idx;                          // index inside the block at level j
      const int i_in_blk = approx ? ib : (p.n >> j) + ib;        // logical row inside the block
      const bool hi = i_in_blk < p.k_hi;
      const float qmax = hi ? p.qmax_hi : p.qmax_lo;
      // the MMA thread issued this product after it saw the row block's count complete: the table is final
      if (!wait_acc(jb)) return false;
      const float u = __uint_as_float(ld_relaxed_gpu(p.rowmax + rb * 128 + r));
      const float amax = odd ? fmaf(u, CQ_RSQRT2_HI, u * CQ_RSQRT2_LO) : u;      // in units of 2^(-(j >> 1))
      const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
      const float inv = __fdiv_rn(1.0f, scale);
      const float true_scale = (amax > 0.f) ? scale * pw : 1.0f;
      const float2 inv2 = make_float2(inv, inv), ns2 = make_float2(-scale, -scale);
      const long row = blk * p.n + i_in_blk;
      const int col0 = c * 128 + half * 64;
      uint8_t* dst = nullptr;       // this lane's 64 channels of its row
      bool four_bit = false;
      if (raw) {
        dst = reinterpret_cast<uint8_t*>(p.aout + rb * (long)K + col0);
      } else if (OUT == HTC_OUT_T) {
        dst = reinterpret_cast<uint8_t*>(p.T_out + row * (long)K + col0);
      } else if (OUT == HTC_OUT_PUBLIC) {
        if (hi) {
          dst = reinterpret_cast<uint8_t*>(p.q_hi + (blk * p.k_hi + i_in_blk) * (long)K + col0);
        } else {
          dst = p.q_lo + (blk * (p.n - p.k_hi) + (i_in_blk - p.k_hi)) * (long)(K >> 1) + (col0 >> 1);
          four_bit = true;
        }
        if (c == 0 && half == 0) p.x_scale[row] = true_scale;
      } else if (OUT == HTC_OUT_A8) {
        dst = reinterpret_cast<uint8_t*>(p.a8 + row * (long)K + col0);
        if (c == 0 && half == 0) p.x_scale[row] = true_scale;
      } else {
        // tile order of the GEMM's fused inverse (see k_haar_cq.cuh): 256-token tiles
        const long tile = (blk * p.n + ((long)ib << j)) >> 8;
        const int i_loc = ib & ((256 >> j) - 1);
        const int tcol = approx ? 32 * i_loc : cq_tile_col_detail(j, i_loc);
        const long prow = tile * 256 + tcol;
        dst = reinterpret_cast<uint8_t*>(p.a8 + prow * (long)K + col0);
        if (c == 0 && half == 0) p.sx_epi[prow] = true_scale * (odd ? pw * CQ_RSQRT2_HI : pw);
      }
      const uint32_t taddr = lane_base + static_cast<uint32_t>(buf * 128);
      uint32_t v[2][32];
      ptx::tmem_ld_32x32b_x32(taddr, v[0]);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        ptx::tmem_ld_wait();
        if (ch == 0) ptx::tmem_ld_32x32b_x32(taddr + 32, v[1]);
        const uint32_t(&x)[32] = v[ch];
        if (raw) {
          float4* o = reinterpret_cast<float4*>(dst) + ch * 8;
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            o[q4] = make_float4(__uint_as_float(x[4 * q4]), __uint_as_float(x[4 * q4 + 1]), __uint_as_float(x[4 * q4 + 2]),
                                __uint_as_float(x[4 * q4 + 3]));
          continue;
        }
        uint32_t w[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          uint32_t bits[4];
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const float2 raw2 = make_float2(__uint_as_float(x[4 * g + 2 * h2]), __uint_as_float(x[4 * g + 2 * h2 + 1]));
            // 2^(-j/2) = c * 2^(-(j >> 1)): only c touches the data, head + tail so the product is rounded once
            const float2 t = __ffma2_rn(raw2, nhi, __fmul2_rn(raw2, nlo));
            if (OUT == HTC_OUT_T) {
              bits[2 * h2] = __float_as_uint(t.x * pw);
              bits[2 * h2 + 1] = __float_as_uint(t.y * pw);
            } else {
              const float2 q0 = __fmul2_rn(t, inv2);
              const float2 rem = __ffma2_rn(q0, ns2, t);
              const float2 q = __fadd2_rn(__ffma2_rn(rem, inv2, q0), make_float2(CQ_MAGIC, CQ_MAGIC));
              bits[2 * h2] = __float_as_uint(q.x);
              bits[2 * h2 + 1] = __float_as_uint(q.y);
            }
          }
          if (OUT == HTC_OUT_T) {
            reinterpret_cast<uint4*>(dst)[ch * 8 + g] = make_uint4(bits[0], bits[1], bits[2], bits[3]);
          } else {
            // the low byte of each word is the two's complement code
            w[g] = __byte_perm(__byte_perm(bits[0], bits[1], 0x0040), __byte_perm(bits[2], bits[3], 0x0040), 0x5410);
          }
        }
        if (OUT == HTC_OUT_T) continue;
        if (four_bit) {
          uint32_t n4[4];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const uint32_t na = w[2 * g] & 0x0F0F0F0Fu, nb = w[2 * g + 1] & 0x0F0F0F0Fu;
            const uint32_t ta = (na | (na >> 4)) & 0x00FF00FFu, tb = (nb | (nb >> 4)) & 0x00FF00FFu;   // bytes 0, 2
            n4[g] = __byte_perm(ta, tb, 0x6420);
          }
          reinterpret_cast<uint4*>(dst)[ch] = make_uint4(n4[0], n4[1], n4[2], n4[3]);
        } else {
          reinterpret_cast<uint4*>(dst)[2 * ch] = make_uint4(w[0], w[1], w[2], w[3]);
          reinterpret_cast<uint4*>(dst)[2 * ch + 1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[buf]);
      return true;
    };

    long i = set;
    for (; i < n_local && ok; i += 2) {
      const long item = blockIdx.x + i * gridDim.x;
      const long rb = item / p.nchunks;
      // ---- P1: maxima of this warp's 64 columns
      const long jb = job_p1(i);
      const int buf = static_cast<int>(jb & (HTC_NBUF - 1));
      if (!wait_acc(jb)) {
        ok = false;
        break;
      }
      {
        const uint32_t taddr = lane_base + static_cast<uint32_t>(buf * 128);
        uint32_t v[2][32];
        ptx::tmem_ld_32x32b_x32(taddr, v[0]);
        ptx::tmem_ld_32x32b_x32(taddr + 32, v[1]);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        ptx::mbar_arrive(&tempty[buf]);     // the values are in registers: the accumulator may be refilled
        float m0 = 0.f, m1 = 0.f;
#pragma unroll
        for (int q4 = 0; q4 < 32; ++q4) {
          m0 = fmaxf(m0, fabsf(__uint_as_float(v[0][q4])));
          m1 = fmaxf(m1, fabsf(__uint_as_float(v[1][q4])));
        }
        // hand the maxima to the set's publisher warp (its slot is clear once it has taken the previous tile's)
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&pempty[set], static_cast<uint32_t>(((i >> 1) & 1) ^ 1), abort_word,
                                                            HTC_WAIT_LIMIT))) {
          ok = false;
          break;
        }
        atomicMax(&pslot[set * 128 + r], __float_as_uint(fmaxf(m0, m1)));
        ptx::mbar_arrive(&pfull[set]);
      }
      // ---- P2 of the item HTC_LAG back
      if (i >= HTC_LAG && !pass2(i - HTC_LAG)) ok = false;
    }
    // the last HTC_LAG items of the CTA: their second products come after its last first product
    for (long i2 = i - HTC_LAG; i2 < n_local && ok; i2 += 2)
      if (i2 >= 0 && !pass2(i2)) ok = false;
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

}  // namespace stamp
