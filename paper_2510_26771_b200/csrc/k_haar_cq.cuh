// Fused Haar transform + per-token mixed-precision quantizer (Algorithm 1, "STaMP
// linear layer": its sequence transform and its per-token quantizer): one pass over the activation in HBM, up to four Haar levels per launch.
//
// The two axes pull in different directions: a transformed token's scale needs the maximum over
// ALL K channels of its row, while a Haar coefficient of level l needs 2^l consecutive tokens of
// ONE channel.  Here a thread owns four adjacent channels of a group of G = 2^P consecutive tokens
// and keeps all G coefficients of its channels in registers; a CTA owns a strip of channels; a
// thread-block cluster of C CTAs covers the whole feature axis (C = 1 up to 2048 channels).  The
// only thing the CTAs of a cluster exchange is the G per-row maxima of their strips: each CTA
// posts them into a mailbox in every peer's shared memory with asynchronous remote stores whose
// arrival is counted on an mbarrier of the receiving CTA (st.async, distributed shared memory), so
// there is no cluster-wide barrier and no fence on the sending side in the loop.  Every detail row of the P levels is then quantized from registers and stored; the
// group's un-normalised sum row (1/G of the data, fp32) is the input of the next launch, which
// runs the same kernel on fp32 rows, until the last launch also quantizes the approximation rows.
//
// Clusters are persistent: each walks over token groups with a stride of the number of clusters.
// bf16 activations are staged through a shared-memory ring filled by bulk asynchronous copies
// (one per token row of the strip) issued NS - 1 groups ahead, so HBM reads stay in flight while
// a group is being reduced, exchanged and stored; fp32 rows (the small later launches) are read
// with plain coalesced 128-bit loads.
//
// Arithmetic.  Butterflies run on un-normalised sums with packed fp32x2 operations.  A level-j
// coefficient is the un-normalised value times 2^(-j/2) = c * 2^(-(j >> 1)) with c = 1 (j even) or
// 1/sqrt 2 (j odd).  Only c is applied to the data (head + tail FMA, so the product is rounded
// once); the exact power of two is carried by the scale instead: with t' = fl(v c) and
// s' = fl(absmax' / qmax), t / s and t' / s' are the same fp32 quotient and the stored scale is
// s' * 2^(-(j >> 1)).  t' / s' is evaluated as reciprocal + one Newton step, and rounded to the
// nearest integer (ties to even) by adding 1.5 * 2^23.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

struct CqParams {
  const void* in;   // [nseq, Lin, K] bf16 / fp32 activations, or fp32 un-normalised sums over 2^lvl0 tokens
  float* aout;      // [nseq, Lin >> P, K] un-normalised sums over 2^(lvl0+P) tokens; nullptr in the last launch
  int K;            // channels
  int Kc;           // channels per CTA strip (= 4 * blockDim.x)
  int Lin;          // input rows per transform block in this launch
  int n;            // tokens per transform block
  int lvl0;         // Haar levels already applied to the input rows
  int k_hi;         // 8-bit rows per transform block
  float qmax_hi, qmax_lo;
  long ngroups;     // nseq * (Lin >> P)
  int nstages;      // depth of the shared-memory ring (bf16 input only)
  int8_t* a8;       // [M, K] one code per int8 (GEMM operand)      -- CQ_OUT_A8
  int8_t* q_hi;     // public packed outputs                         -- CQ_OUT_PUBLIC
  uint8_t* q_lo;
  float* x_scale;   // [M]
  float* T_out;     // [M, K] transformed values (debug export)      -- CQ_OUT_T
  // CQ_OUT_TILED: a8 rows in the order the GEMM's fused inverse epilogue consumes them
  long a8_top_row;  // codes of the rows of levels > 8 (logical order inside a block) go to rows a8_top_row + i of a8
  float* sx_top;    // [M / 256]    their scales
  float* sx_epi;    // [M]          scale * 2^(-j/2) of every tile row, indexed like a8
  // Optional: a region (the layer's weight codes) to pull towards L2 while this launch and the small
  // launches after it leave HBM idle; the kernels that follow read it from there.  pf_bytes % 16 == 0.
  const uint8_t* pf_base;
  long pf_bytes;
};

constexpr float CQ_MAGIC = 12582912.0f;            // 1.5 * 2^23
constexpr long long CQ_WAIT_LIMIT = 2000000000LL;  // SM clocks before a wait on a copy gives up
constexpr float CQ_RSQRT2_HI = 0.707106769084930419921875f;  // fp32(1/sqrt 2)
constexpr float CQ_RSQRT2_LO = 1.2101617101e-8f;             // 1/sqrt 2 - fp32(1/sqrt 2)

// What a launch writes besides the scales: the GEMM's int8 operand, the public packed codes, or
// the fp32 transformed values (debug export).
enum CqOut { CQ_OUT_A8 = 0, CQ_OUT_PUBLIC = 1, CQ_OUT_T = 2, CQ_OUT_TILED = 3 };

// Row order of the tiled operand (CQ_OUT_TILED).  The GEMM's token tile t covers the 256 original
// tokens [256 t, 256 t + 256) and must own every coefficient their reconstruction needs from
// levels 1..D, D = min(levels, 8) >= 5 (rows of levels > 8 go to a small separate table).  Inside a tile, column 32 c + r (r = 1..31) holds the r-th value,
// in [d_5 | d_4 (2) | d_3 (4) | d_2 (8) | d_1 (16)] order, of the 32-token chunk c; column 32 q holds
// the q-th of the tile's eight coarse values in band order [a_D | d_D | ... | d_6].  An epilogue
// thread thus finds, per chunk, the 31 details in the order its in-register synthesis wants them,
// with the chunk's level-5 sum (rebuilt from the eight coarse values) in slot 0.
// Returns the column inside the tile; `i` is the coefficient's index inside its 256-token tile.
__device__ __forceinline__ int cq_tile_col_detail(int j, int i_loc) {
  if (j <= 5) {
    const int sh = 5 - j;
    return 32 * (i_loc >> sh) + (1 << sh) + (i_loc & ((1 << sh) - 1));
  }
  return 32 * ((256 >> j) + i_loc);
}

__device__ __forceinline__ float2 cq_f2(float a) { return make_float2(a, a); }

// The butterflies run in place: a pair (x[2i], x[2i+1]) of stride-s neighbours becomes (sum, difference)
// where it stands, and the next level pairs the sums (stride 2s).  The coefficient that the output
// order [a | d_P | d_(P-1) (2) | ... | d_1 (G/2)] calls row r therefore sits in register:
__host__ __device__ constexpr int cq_reg_of_row(int P, int r) {
  if (r == 0) return 0;
  int k = 0;
  while ((2 << k) <= r) ++k;          // r in [2^k, 2^(k+1)): detail of local level l = P - k
  const int l = P - k, i = r - (1 << k);
  return (2 * i + 1) << (l - 1);
}

// Shared memory: [ring: nstages x G x Kc x sizeof(TIn)] [full barriers: 8 x u64] [mailbox barriers: 2 x u64]
//   [maxima: 2 x 16 u32] [mailbox: 2 x 8 CTAs x 16 u32]
//   [per row: {1/s', 1/s', -s', -s'} 16 B] [per row: {logical row, row in q_hi / q_lo | 8-bit flag,
//   2^(-(j>>1)) bits, 0} 16 B]
template <int P, typename TIn>
__host__ __device__ constexpr size_t cq_slab_bytes(int Kc) { return (size_t)(1 << P) * Kc * sizeof(TIn); }
constexpr size_t CQ_TAIL_BYTES = 8 * 8 + 64 + 2 * 16 * 4 + 2 * 8 * 16 * 4 + 16 * 16 + 16 * 16;

// LODD = lvl0 & 1: with it the parity of every row's level, hence whether it needs the 1/sqrt 2
// factor, is known at compile time.
template <int P, typename TIn, int OUT, int LODD>
__global__ void __launch_bounds__(512, 1) k_haar_cq(const CqParams p) {
  constexpr int G = 1 << P;
  constexpr bool STAGED = (sizeof(TIn) == 2);
  static_assert(P <= 4, "a thread holds 16 rows of four channels at most");
  extern __shared__ __align__(128) uint8_t cq_smem[];
  const size_t slab = STAGED ? cq_slab_bytes<P, TIn>(p.Kc) : 0;
  uint8_t* tail = cq_smem + (STAGED ? slab * p.nstages : 0);
  uint64_t* full = reinterpret_cast<uint64_t*>(tail);
  uint64_t* mb = reinterpret_cast<uint64_t*>(tail + 64);           // [2] one per mailbox buffer
  unsigned* mymax = reinterpret_cast<unsigned*>(tail + 128);       // [2][16]
  unsigned* mailbox = reinterpret_cast<unsigned*>(tail + 256);     // [2][8][16]
  float4* tabB = reinterpret_cast<float4*>(tail + 1280);           // [16]
  int4* tabC = reinterpret_cast<int4*>(tail + 1536);               // [16]
  __shared__ uint32_t abort_word;

  const int tid = threadIdx.x;
  const int lane = tid & 31;
  unsigned csize, rank;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
  rank = ptx::cluster_ctarank();
  const long cid = blockIdx.x / csize, ncl = gridDim.x / csize;
  const int K = p.K;
  const int cbase = static_cast<int>(rank) * p.Kc;
  const int cvalid = max(0, min(p.Kc, K - cbase));   // channels of this strip (0: the strip is empty)
  const uint32_t row_bytes = static_cast<uint32_t>(cvalid) * sizeof(TIn);
  const int gps = p.Lin >> P;                         // groups per transform block: a power of two
  const int gps_shift = 31 - __clz(gps);              // (64-bit divisions in the loop would cost more than a row)
  const bool last = (p.aout == nullptr);
  const int NS = p.nstages;
  const bool valid = 4 * tid < cvalid;                // this thread's four channels exist
  // threads past the end of a ragged strip redo its last quad: same maxima, nothing stored
  const int qe = valid ? tid : max(cvalid / 4 - 1, 0);
  const int c0 = cbase + 4 * tid;

  if (tid < 32) mymax[tid] = 0u;
  if (tid == 0) {
    abort_word = 0;
    if (STAGED)
      for (int s = 0; s < NS; ++s) ptx::mbar_init(&full[s], 1);
    ptx::mbar_init(&mb[0], 1);
    ptx::mbar_init(&mb[1], 1);
    ptx::fence_mbar_init();
  }
  // every CTA of the cluster has initialised its barriers before anyone posts to them
  ptx::cluster_sync();
  if (p.pf_bytes > 0 && tid >= 480) {   // the last warp: fire-and-forget hints, 8 KB each
    constexpr long PF_CHUNK = 8192;
    const long nchunk = (p.pf_bytes + PF_CHUNK - 1) / PF_CHUNK;
    for (long c = (long)blockIdx.x * 32 + lane; c < nchunk; c += (long)gridDim.x * 32) {
      const long off = c * PF_CHUNK;
      const long left = p.pf_bytes - off;
      ptx::prefetch_l2_bulk(p.pf_base + off, static_cast<uint32_t>(left < PF_CHUNK ? left : PF_CHUNK));
    }
  }
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();   // the next kernel may set itself up on SMs as they fall free; it still waits for this grid to finish   // the input rows may come from the previous launch

  // warp 0 brings one group's rows of this strip into a ring stage: lane r copies token row r
  auto issue_load = [&](long grp, int stage) {
    if (!STAGED || cvalid == 0 || tid >= 32) return;
    const long sq = grp >> gps_shift;
    const long g = grp & (gps - 1);
    const uint8_t* src = static_cast<const uint8_t*>(p.in) + (((sq * p.Lin + g * G) * (long)K + cbase) * (long)sizeof(TIn));
    uint8_t* dst = cq_smem + stage * slab;
    if (lane == 0) ptx::mbar_arrive_expect_tx(&full[stage], row_bytes * G);
    __syncwarp();
    if (lane < G) ptx::bulk_load(dst + (size_t)lane * row_bytes, src + (size_t)lane * K * sizeof(TIn), row_bytes, &full[stage]);
  };

  if (STAGED)
    for (int s = 0; s < NS - 1; ++s) {
      const long grp = cid + s * ncl;
      if (grp < p.ngroups) issue_load(grp, s);
    }

  bool ok = true;
  int it = 0;
  int stage = 0;           // ring stage of this group and the parity of its barrier phase, kept
  uint32_t ring_phase = 0; // incrementally: a division per iteration costs more than a row's arithmetic
  for (long grp = cid; grp < p.ngroups; grp += ncl, ++it) {
    const int b = static_cast<int>(it & 1);
    if (STAGED && ok) {
      // the stage read in the previous iteration is free: every thread passed a barrier since
      const long nxt = grp + (long)(NS - 1) * ncl;
      if (nxt < p.ngroups) issue_load(nxt, stage == 0 ? NS - 1 : stage - 1);
    }
    // this group's mailbox buffer expects G maxima from each CTA of the cluster (its previous use,
    // two groups ago, was completed and read before this thread passed that group's barrier)
    if (tid == 0) ptx::mbar_arrive_expect_tx(&mb[b], csize * G * 4u);
    if (STAGED && cvalid > 0 && ok) {
      // every thread waits for the copies itself (that also makes the data visible to it); a
      // thread that gives up tells the others through the abort word their waits poll
      if (!ptx::mbar_wait_bounded(&full[stage], ring_phase, &abort_word, CQ_WAIT_LIMIT)) {
        ok = false;
        abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
    const long sq = grp >> gps_shift;
    const int g = static_cast<int>(grp & (gps - 1));

    // ---- load G tokens x 4 channels, butterflies in registers (un-normalised)
    float2 v[2][G];
    if (ok && cvalid > 0) {
      if (STAGED) {
        const uint8_t* s8 = cq_smem + stage * slab + 8 * qe;
#pragma unroll
        for (int r = 0; r < G; ++r) {
          const uint2 w = *reinterpret_cast<const uint2*>(s8 + r * row_bytes);
          // bf16 -> fp32 by byte permutation (keeps the shifts off the FMA pipe)
          v[0][r] = make_float2(__uint_as_float(__byte_perm(w.x, 0u, 0x1044)), __uint_as_float(__byte_perm(w.x, 0u, 0x3244)));
          v[1][r] = make_float2(__uint_as_float(__byte_perm(w.y, 0u, 0x1044)), __uint_as_float(__byte_perm(w.y, 0u, 0x3244)));
        }
      } else {
        const float* src = static_cast<const float*>(p.in) + ((sq * p.Lin + (long)g * G) * (long)K + cbase + 4 * qe);
#pragma unroll
        for (int r = 0; r < G; ++r) {
          const float4 w = *reinterpret_cast<const float4*>(src + (long)r * K);
          v[0][r] = make_float2(w.x, w.y);
          v[1][r] = make_float2(w.z, w.w);
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < G; ++r) v[0][r] = v[1][r] = cq_f2(0.f);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
      for (int st = 1; st < G; st <<= 1) {
#pragma unroll
        for (int i = 0; i < G; i += 2 * st) {
          const float2 a = v[h][i], b2 = v[h][i + st];
          v[h][i] = __fadd2_rn(a, b2);
          v[h][i + st] = ptx::fsub2_rn(a, b2);
        }
      }
    }
    // row r of [a | d_P | d_(P-1) (2) | ... | d_1 (G/2)] is now v[h][cq_reg_of_row(P, r)]

    // ---- per-row maxima of this strip.  G values per lane are reduced over the warp by a transposing
    // butterfly: at each stage half of the rows go to the partner lane (xor of one lane bit), so the
    // work halves every stage; lane L ends up with the warp-wide maximum of row (L >> 1) & (G - 1).
    {
      float m[G];
#pragma unroll
      for (int r = 0; r < G; ++r) {
        const int ri = cq_reg_of_row(P, r);
        m[r] = fmaxf(fmaxf(fabsf(v[0][ri].x), fabsf(v[0][ri].y)), fmaxf(fabsf(v[1][ri].x), fabsf(v[1][ri].y)));
      }
#pragma unroll
      for (int n = G; n >= 2; n >>= 1) {
        const bool upper = (lane & n) != 0;
#pragma unroll
        for (int r = 0; r < n / 2; ++r) {
          const float send = upper ? m[r] : m[r + n / 2];
          const float keepv = upper ? m[r + n / 2] : m[r];
          m[r] = fmaxf(keepv, __shfl_xor_sync(0xffffffffu, send, n));
        }
      }
      // the lane bits no stage used: bit 0 and the bits above log2 G
      m[0] = fmaxf(m[0], __shfl_xor_sync(0xffffffffu, m[0], 1));
#pragma unroll
      for (int bit = 2 * G; bit < 32; bit <<= 1)
        if (bit >= 2) m[0] = fmaxf(m[0], __shfl_xor_sync(0xffffffffu, m[0], bit));
      if (lane < 2 * G && (lane & 1) == 0) atomicMax(&mymax[b * 16 + (lane >> 1)], __float_as_uint(m[0]));
    }
    __syncthreads();
    if (tid < G) {
      // post this strip's maxima to every CTA of the cluster (this one included) and clear them
      const unsigned mine = mymax[b * 16 + tid];
      mymax[b * 16 + tid] = 0u;
      const uint32_t slot = ptx::smem_u32(&mailbox[(b * 8 + rank) * 16 + tid]);
      const uint32_t bar = ptx::smem_u32(&mb[b]);
      for (unsigned q = 0; q < csize; ++q) ptx::st_async_u32(ptx::mapa(slot, q), mine, ptx::mapa(bar, q));
    }
    if (!last && valid && ok)
      *reinterpret_cast<float4*>(p.aout + (grp * (long)K + c0)) =
          make_float4(v[0][0].x, v[0][0].y, v[1][0].x, v[1][0].y);

    // ---- row tables: maxima over the cluster, scales, output rows
    if (tid < G) {
      if (!ptx::mbar_wait_bounded_cluster(&mb[b], static_cast<uint32_t>((it >> 1) & 1), &abort_word, CQ_WAIT_LIMIT)) {
        ok = false;
        abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
    if (tid < G && (tid > 0 || last)) {
      const int r = tid;
      unsigned um = 0;
      for (unsigned q = 0; q < csize; ++q) um = max(um, mailbox[(b * 8 + q) * 16 + r]);
      int k = 0;                       // r in [2^k, 2^(k+1)): detail row of local level P - k
      while ((2 << k) <= r) ++k;
      const int l = (r == 0) ? P : P - k;
      const int j = p.lvl0 + l;
      const int i_in_blk = (r == 0) ? g : (p.n >> j) + (g << k) + (r - (1 << k));
      const float u = __uint_as_float(um);
      const float amax = (j & 1) ? fmaf(u, CQ_RSQRT2_HI, u * CQ_RSQRT2_LO) : u;   // in units of 2^(-(j >> 1))
      const bool hi = i_in_blk < p.k_hi;
      const float qmax = hi ? p.qmax_hi : p.qmax_lo;
      const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
      const float inv = __fdiv_rn(1.0f, scale);
      const float pw = __int_as_float((127 - (j >> 1)) << 23);                     // 2^(-(j >> 1))
      const long row = sq * p.n + i_in_blk;
      const long pub = hi ? sq * p.k_hi + i_in_blk : sq * (p.n - p.k_hi) + (i_in_blk - p.k_hi);
      tabB[r] = make_float4(inv, inv, -scale, -scale);
      const float true_scale = (amax > 0.f) ? scale * pw : 1.0f;
      if (OUT == CQ_OUT_TILED) {
        // where the row lives in the tiled operand (or in the small table of rows above the tiles)
        const bool top = j > 8;
        long prow;
        if (top) {
          const long trow = sq * (p.n >> 8) + i_in_blk;   // the first n / 256 logical rows of a block are exactly those
          if (rank == 0 && ok) p.sx_top[trow] = true_scale;
          prow = p.a8_top_row + trow;
        } else {
          const int idx = (r == 0) ? g : (g << k) + (r - (1 << k));   // index inside the block at level j
          const long tile = (sq * p.n + ((long)idx << j)) >> 8;
          const int i_loc = idx & ((256 >> j) - 1);
          const int col = (r == 0) ? 32 * i_loc : cq_tile_col_detail(j, i_loc);
          prow = tile * 256 + col;
          const float nrm = (j & 1) ? pw * CQ_RSQRT2_HI : pw;        // 2^(-j/2)
          if (rank == 0 && ok) p.sx_epi[prow] = true_scale * nrm;
        }
        tabC[r] = make_int4(static_cast<int>(prow), 0, __float_as_int(pw), top ? 1 : 0);
      } else {
        tabC[r] = make_int4(static_cast<int>(row), static_cast<int>(pub) | (hi ? static_cast<int>(0x80000000u) : 0),
                            __float_as_int(pw), 0);
        if (rank == 0 && ok) p.x_scale[row] = true_scale;
      }
    }
    __syncthreads();

    // ---- normalise, quantize and store from registers
    if (valid && ok) {
      // per-thread bases; a row's address is base + row * pitch
      int8_t* const a8c = p.a8 + c0;
      int8_t* const qhc = p.q_hi + c0;
      uint8_t* const qlc = p.q_lo + (c0 >> 1);
      uint8_t* const Tc = reinterpret_cast<uint8_t*>(p.T_out + c0);
#pragma unroll
      for (int r = 0; r < G; ++r) {
        if (r == 0 && !last) continue;
        // local level of row r: P for the sum row, P - floor(log2 r) for a detail row
        int lg = 0;
#pragma unroll
        for (int s = 1; s < 5; ++s) lg += (r >> s) ? 1 : 0;
        const int l = (r == 0) ? P : P - lg;
        const bool odd = ((LODD + l) & 1) != 0;
        const int ri = cq_reg_of_row(P, r);
        const int4 Cc = tabC[r];
        float2 t[2];
#pragma unroll
        for (int h = 0; h < 2; ++h)
          t[h] = odd ? __ffma2_rn(v[h][ri], cq_f2(CQ_RSQRT2_HI), __fmul2_rn(v[h][ri], cq_f2(CQ_RSQRT2_LO))) : v[h][ri];
        if (OUT == CQ_OUT_T) {
          const float pw = __int_as_float(Cc.z);
          *reinterpret_cast<float4*>(ptx::ptr_mad_wide(Tc, Cc.x, 4 * K)) =
              make_float4(t[0].x * pw, t[0].y * pw, t[1].x * pw, t[1].y * pw);
          continue;
        }
        const float4 Bv = tabB[r];
        const float2 inv2 = make_float2(Bv.x, Bv.y), ns2 = make_float2(Bv.z, Bv.w);
        uint32_t bits[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float2 q0 = __fmul2_rn(t[h], inv2);
          const float2 rem = __ffma2_rn(q0, ns2, t[h]);
          const float2 q = __fadd2_rn(__ffma2_rn(rem, inv2, q0), cq_f2(CQ_MAGIC));
          bits[2 * h] = __float_as_uint(q.x);
          bits[2 * h + 1] = __float_as_uint(q.y);
        }
        // the low byte of each word is the two's complement code
        const uint32_t four = __byte_perm(__byte_perm(bits[0], bits[1], 0x0040), __byte_perm(bits[2], bits[3], 0x0040), 0x5410);
        if (OUT == CQ_OUT_TILED) {
          *reinterpret_cast<uint32_t*>(ptx::ptr_mad_wide(a8c, Cc.x, K)) = four;
        } else if (OUT == CQ_OUT_A8) {
          *reinterpret_cast<uint32_t*>(ptx::ptr_mad_wide(a8c, Cc.x, K)) = four;
        } else if (Cc.y < 0) {
          *reinterpret_cast<uint32_t*>(ptx::ptr_mad_wide(qhc, Cc.y & 0x7FFFFFFF, K)) = four;
        } else {
          const uint32_t nib = (four & 0x0F0F0F0Fu);
          const uint32_t two = (nib | (nib >> 4)) & 0x00FF00FFu;   // bytes 0 and 2 hold two codes each
          *reinterpret_cast<uint16_t*>(ptx::ptr_mad_wide(qlc, Cc.y, K >> 1)) =
              static_cast<uint16_t>(__byte_perm(two, 0u, 0x4420));
        }
      }
    }
    // the row tables and the ring stage are reused in the next iteration: its barriers order that
    if (++stage == NS) {
      stage = 0;
      ring_phase ^= 1u;
    }
  }
  if (STAGED && !ok) {
    // copies issued ahead were never consumed: give them time to land before the shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {
    }
  }
  // leave together: no CTA's shared memory goes away while a peer's posts could still be in flight
  ptx::cluster_sync();
}

}  // namespace stamp
