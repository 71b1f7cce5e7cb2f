// Integer GEMM of the STaMP linear layer on the 5th-generation tensor cores (the product step of
// Algorithm 1 evaluated on the integer codes, followed by the de-quantization of Sec. 2.1).
//
//   acc[tok, ch] = sum_k a8[tok, k] * w8[ch, k]            int8 x int8 -> int32
//
// Operand roles are swapped with respect to the usual activation-major GEMM: the weight tile
// (128 output channels) is the MMA "A" operand and the token tile (BN tokens) is the MMA "B"
// operand, so an accumulator lives in TMEM with lane = output channel and column = token.
// An epilogue thread therefore owns one output channel and reads runs of consecutive tokens
// into registers -- the axis along which the inverse sequence transform acts -- while a warp's
// 32 lanes cover 32 consecutive channels of one token, i.e. one coalesced 128-byte store.
//
// Structure: persistent CTAs (one per SM), warp-specialised.
//   warp 0     TMA producer: 128-byte-swizzled K-major tiles of both operands into a
//              STAGES-deep shared-memory ring (one mbarrier pair per stage)
//   warp 1     allocates TMEM; one elected thread issues tcgen05.mma kind::i8 (128 x BN x 32
//              per instruction, four per 128-byte K block) into one of two accumulators
//   warps 2-9  epilogue: tcgen05.ld the finished accumulator (the other one is being filled),
//              de-quantize with per-token x per-channel scales, store.  A warp reaches only the 32
//              TMEM lanes of its quarter (warp % 4), so two warps share a quarter and each drains
//              half of the accumulator's columns
// Every mbarrier wait is bounded; when one expires the CTA raises the device status word,
// drains its outstanding copies, frees TMEM and returns.
//
// PAIR = true: the same kernel on CTA pairs (tcgen05 cta_group::2, clusters of two).  A pair owns a tile of 256
// channels x 256 tokens: either CTA stages ITS 128 channels and ITS 128 tokens of every K block (32 KB per
// stage instead of 48), the even-ranked CTA issues one M256 x N256 x K32 instruction for both, and either
// CTA's epilogue drains the 128 accumulator lanes that land in its own tensor memory.  With half of the token
// operand coming from the neighbour, a CTA moves 16 KB through its shared memory per instruction instead of
// 24 KB, which is what kept the single-CTA main loop below the tensor rate.  The odd-ranked CTA's copies are
// counted on the even-ranked CTA's barrier; stage and accumulator hand-backs reach both CTAs with one
// multicast commit; the epilogue threads of both CTAs release an accumulator on the issuing CTA's barrier.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

enum GemmEpilogue { EPI_DEQUANT_F32 = 0, EPI_RAW_I32 = 1, EPI_HAAR_F32 = 2, EPI_HAAR_BF16 = 3, EPI_DEQUANT_BF16X2 = 4,
                    EPI_DEQUANT_ZP_F32 = 5, EPI_HAAR2D_F32 = 6, EPI_HAAR2D_BF16 = 7 };

struct GemmParams {
  int n_out;               // output channels (MMA M extent)
  int m_tok;               // tokens (MMA N extent)
  int k;                   // reduction length, multiple of 128
  const float* x_scale;    // [m_tok]
  const float* w_scale;    // [n_out], or nullptr for 1
  void* out;               // [m_tok, n_out] float (EPI_DEQUANT_F32) or int32 (EPI_RAW_I32); EPI_DEQUANT_BF16X2:
                           // two bf16 planes [2][m_tok, n_out], value = hi + lo (operand of the DCT inverse)
  int group;               // channel tiles per raster band
  // EPI_HAAR_*: the token operand is in the tiled row order of the transform+quantize kernel, x_scale
  // holds scale * 2^(-j/2) per tile row, and the epilogue applies the inverse Haar transform of the
  // tile's 256 tokens (the inverse-transform step of Algorithm 1), w_scale and the bias before storing Y.
  int depth;               // Haar levels closed inside a tile, 5..8
  const float* a8v;        // [m_tok / 256, n_out] level-8 approximation of every tile when the transform
                           // has more than 8 levels (orthonormal scaling), else nullptr
  const float* bias;       // [n_out] or nullptr
  // EPI_DEQUANT_ZP_F32: zero-point codes (Sec. 2.1, first equation):  out = (acc - x_zero[tok] * w_sum[ch])
  // * x_scale[tok] * w_scale[ch], the bracket in 64-bit integers
  const int* x_zero;       // [m_tok] zero point of every token's stored codes
  const int* w_sum;        // [n_out] sum over k of the weight codes of a channel
  // (x_zero / w_sum may also be given to EPI_HAAR2D_*: the same term is then taken out before the synthesis.)
  // EPI_HAAR2D_*: the token operand is in the patch order of the 2-D Haar quantize kernel (64 consecutive rows
  // = the coefficients of one 8 x 8 patch of the token grid in synthesis order), x_scale holds scale * 2^-l, and
  // the epilogue applies the three-level inverse 2-D Haar transform of the tile's four patches, w_scale and the
  // bias before storing Y at the patches' raster positions.
  int grid_w;              // width of the token grid of a transform block
  int n_block;             // tokens per transform block (grid_w x height)
};

constexpr int GEMM_BM = 128;           // output channels per tile
constexpr int GEMM_BK = 128;           // int8 per K block = one 128-byte swizzle row
constexpr int GEMM_EPI_THREADS = 256;   // two epilogue warps per TMEM lane quarter, each draining half the columns
constexpr int GEMM_THREADS = 64 + GEMM_EPI_THREADS;
constexpr long long GEMM_WAIT_LIMIT = 4000000000LL;  // SM clocks (~2 s) before a wait gives up

template <int BN, int STAGES, bool PAIR = false>
struct GemmSmem {
  static constexpr int W_BYTES = GEMM_BM * GEMM_BK;
  static constexpr int X_BYTES = (PAIR ? BN / 2 : BN) * GEMM_BK;   // a CTA of a pair stages half of the token tile
  static constexpr int STAGE_BYTES = W_BYTES + X_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  // full[STAGES], empty[STAGES], tfull[2], tempty[2], then tmem base + abort word
  static constexpr int NUM_BARS = 2 * STAGES + 4;
  static constexpr int SX_OFFSET = BAR_OFFSET + NUM_BARS * 8 + 16;  // token scales of the tile being drained
  static constexpr int ZP_OFFSET = SX_OFFSET + 2 * BN * 4;  // token zero points, same arrangement
  static constexpr int TOTAL = ZP_OFFSET + 2 * BN * 4;   // one buffer per accumulator
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for 1024-byte alignment of the ring
};

__device__ __forceinline__ void tile_coords(int tile, int ch_tiles, int tok_tiles, int group, int& ch_t, int& tok_t) {
  // bands of `group` channel tiles; inside a band, channel tiles vary fastest so that CTAs
  // running at the same time share token tiles and the band's weight tiles stay in L2
  const int per_band = group * tok_tiles;
  const int band = tile / per_band;
  const int rem = tile - band * per_band;
  const int first = band * group;
  const int height = min(group, ch_tiles - first);
  tok_t = rem / height;
  ch_t = first + (rem - tok_t * height);
}

template <int BN, int STAGES, int EPI, bool PAIR = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
    k_gemm_i8(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, GemmParams p) {
  using SM = GemmSmem<BN, STAGES, PAIR>;
  static_assert(!PAIR || BN == 256, "a pair works on 256-token tiles");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + SM::BAR_OFFSET);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile uint32_t* abort_word = tmem_slot + 1;
  float* sx_stage = reinterpret_cast<float*>(smem + SM::SX_OFFSET);
  int* zp_stage = reinterpret_cast<int*>(smem + SM::ZP_OFFSET);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // PAIR: a work item is a pair tile of 2 x 128 channels; this CTA takes channel tile 2 ch_t + rank of it
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
  constexpr int CH_PER_TILE = PAIR ? 2 * GEMM_BM : GEMM_BM;
  const int ch_tiles = (p.n_out + CH_PER_TILE - 1) / CH_PER_TILE;
  const int tok_tiles = (p.m_tok + BN - 1) / BN;
  const int num_tiles = ch_tiles * tok_tiles;
  const int num_kb = p.k / GEMM_BK;
  const int tile0 = PAIR ? blockIdx.x >> 1 : blockIdx.x;
  const int tile_step = PAIR ? gridDim.x >> 1 : gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tfull[a], 1);
      ptx::mbar_init(&tempty[a], PAIR ? 2 * GEMM_EPI_THREADS : GEMM_EPI_THREADS);
    }
    *abort_word = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_w);
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      ptx::tmem_alloc_pair(tmem_slot, 2 * BN);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(tmem_slot, 2 * BN);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  // both CTAs of a pair have initialised their barriers before either signals the other's
  if constexpr (PAIR) ptx::cluster_sync();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::grid_dependency_wait();   // operands and scales come from the kernels launched before

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      for (int tile = tile0; tile < num_tiles && ok; tile += tile_step) {
        int ch_t, tok_t;
        tile_coords(tile, ch_tiles, tok_tiles, p.group, ch_t, tok_t);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait_bounded(&empty[stage], phase ^ 1u, abort_word, GEMM_WAIT_LIMIT)) {
            ok = false;
            break;
          }
          uint8_t* ws = smem + stage * SM::STAGE_BYTES;
          if constexpr (PAIR) {
            // this CTA's 128 channels and 128 tokens; all four copies of the pair are counted on the even CTA's barrier
            const uint32_t bar0 = ptx::mapa(ptx::smem_u32(&full[stage]), 0u);
            if (rank == 0) ptx::mbar_arrive_expect_tx(&full[stage], 2 * SM::STAGE_BYTES);
            ptx::tma_load_2d_pair(ws, &tmap_w, bar0, kb * GEMM_BK, (2 * ch_t + static_cast<int>(rank)) * GEMM_BM);
            ptx::tma_load_2d_pair(ws + SM::W_BYTES, &tmap_x, bar0, kb * GEMM_BK, tok_t * BN + static_cast<int>(rank) * (BN / 2));
          } else {
          ptx::mbar_arrive_expect_tx(&full[stage], SM::STAGE_BYTES);
          ptx::tma_load_2d(ws, &tmap_w, &full[stage], kb * GEMM_BK, ch_t * GEMM_BM);
          ptx::tma_load_2d(ws + SM::W_BYTES, &tmap_x, &full[stage], kb * GEMM_BK, tok_t * BN);
          }
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
        // let the copies already in flight land before the CTA gives its shared memory back
        for (int s = 0; s < STAGES; ++s)
          if (armed & (1u << s)) {
            const long long t0 = clock64();
            // (the odd CTA of a pair has no barrier of its own to watch: it just gives its copies the time)
            while ((rank != 0 || !ptx::mbar_try_wait(&full[s], (armed_parity >> s) & 1u)) && clock64() - t0 < 2000000LL) {
            }
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (PAIR: the even-ranked CTA's, for both)
    if (rank == 0 && ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::make_i8_idesc(PAIR ? 2 * GEMM_BM : GEMM_BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = tile0; tile < num_tiles && ok; tile += tile_step, ++it) {
        const int a = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1u;
        if (!ptx::mbar_wait_bounded(&tempty[a], acc_phase ^ 1u, abort_word, GEMM_WAIT_LIMIT)) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(a * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait_bounded(&full[stage], phase, abort_word, GEMM_WAIT_LIMIT)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t wa = ptx::smem_u32(smem + stage * SM::STAGE_BYTES);
          const uint32_t xa = wa + SM::W_BYTES;
#pragma unroll
          for (int k = 0; k < GEMM_BK / 32; ++k) {
            const uint64_t adesc = ptx::make_kmajor_sw128_desc(wa + k * 32);
            const uint64_t bdesc = ptx::make_kmajor_sw128_desc(xa + k * 32);
            if constexpr (PAIR)
              ptx::mma_i8_ss_pair(tmem_d, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
            else
              ptx::mma_i8_ss(tmem_d, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if constexpr (PAIR) ptx::tc_commit_pair(&empty[stage], 3); else ptx::tc_commit(&empty[stage]);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) {                           // accumulator complete (in both CTAs of a pair)
          if constexpr (PAIR) ptx::tc_commit_pair(&tfull[a], 3); else ptx::tc_commit(&tfull[a]);
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;  // TMEM lanes this warp may touch: 32 * (warp % 4) ...
    const int row = quarter * 32 + lane;
    const int half = (warp - 2) >> 2;     // which half of the accumulator's columns this warp drains
    const int ep_tid = threadIdx.x - 64;  // 0..255
    int it = 0;
    bool ok = true;
    const uint32_t tempty_bar0 = PAIR ? ptx::mapa(ptx::smem_u32(&tempty[0]), 0u) : 0u;   // the issuing CTA's barriers
    for (int tile = tile0; tile < num_tiles && ok; tile += tile_step, ++it) {
      int ch_t, tok_t;
      tile_coords(tile, ch_tiles, tok_tiles, p.group, ch_t, tok_t);
      if constexpr (PAIR) ch_t = 2 * ch_t + static_cast<int>(rank);
      const int a = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1u;
      const int ch = ch_t * GEMM_BM + row;
      const int tok0 = tok_t * BN;
      const bool ch_ok = ch < p.n_out;
      const bool full_tile = (tok0 + BN <= p.m_tok);
      float* sxs = sx_stage + a * BN;
      float sw = 0.f;
      int* zps = zp_stage + a * BN;
      // zero-point codes: always in the de-quantize epilogue made for them, on request in the 2-D Haar ones
      const bool with_zp = (EPI == EPI_DEQUANT_ZP_F32) ||
                           ((EPI == EPI_HAAR2D_F32 || EPI == EPI_HAAR2D_BF16) && p.x_zero != nullptr);
      float my_sx = 0.f;
      int my_zp = 0, wsum = 0;
      if (EPI != EPI_RAW_I32) {
        if (ch_ok) sw = p.w_scale ? __ldg(p.w_scale + ch) : 1.0f;
        // fetch this tile's token scales while the accumulator is still being filled
        if (ep_tid < BN && tok0 + ep_tid < p.m_tok) {
          my_sx = __ldg(p.x_scale + tok0 + ep_tid);
          if (with_zp) my_zp = __ldg(p.x_zero + tok0 + ep_tid);
        }
        if (with_zp && ch_ok) wsum = __ldg(p.w_sum + ch);
      }
      // The eight epilogue warps continue or stop TOGETHER: a warp whose wait ran out raises the abort
      // word, and everybody reads it behind the named barrier below -- no warp is left waiting at that
      // barrier for one that already gave up.  (The TMEM loads are warp-collective as well.)
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(&tfull[a], acc_phase, abort_word, GEMM_WAIT_LIMIT)))
        *abort_word = 1;
      ptx::tc_fence_after();
      if (EPI != EPI_RAW_I32) {
        // every epilogue thread has finished the previous tile that used accumulator `a` (all of
        // them arrived on tempty[a] before tfull[a] could complete again), so its staging buffer is free
        if (ep_tid < BN) {
          sxs[ep_tid] = my_sx;
          if (with_zp) zps[ep_tid] = my_zp;
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(GEMM_EPI_THREADS) : "memory");
      if (*abort_word != 0u) {
        ok = false;
        break;
      }
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(a * BN);
      if constexpr (EPI == EPI_HAAR2D_F32 || EPI == EPI_HAAR2D_BF16) {
        static_assert(BN == 256, "four 8 x 8 patches per tile");
        float bch = 0.f;
        if (ch_ok && p.bias) bch = __ldg(p.bias + ch);
        const int pw = p.grid_w >> 3;        // patches per grid row
        const int ppb = p.n_block >> 6;      // patches per transform block
#pragma unroll 1
        for (int pp = 0; pp < 2; ++pp) {     // this warp's two patches
          const int pcol = (half * 2 + pp) * 64;
          uint32_t r0[32], r1[32];
          ptx::tmem_ld_32x32b_x32(taddr + pcol, r0);
          ptx::tmem_ld_32x32b_x32(taddr + pcol + 32, r1);
          ptx::tmem_ld_wait();
          const float* sxp = sxs + pcol;
          const int* zpp = zps + pcol;
          // column idx of the patch: 0 = LL_3, then per level l (3, 2, 1) the cells' (LH, HL, HH) triples from
          // column 4^(3-l) on; the scales carry 2^-l, so the synthesis is additions only
          auto val = [&](int idx) -> float {
            const uint32_t u = idx < 32 ? r0[idx & 31] : r1[idx & 31];
            if (with_zp)   // (acc - zc * sum_k w) in 64-bit integers, as in EPI_DEQUANT_ZP_F32
              return __ll2float_rn(static_cast<long long>(static_cast<int>(u)) -
                                   static_cast<long long>(zpp[idx]) * wsum) * sxp[idx];
            return static_cast<float>(static_cast<int>(u)) * sxp[idx];
          };
          float v[8][8];
          v[0][0] = val(0);
#pragma unroll
          for (int l = 3; l >= 1; --l) {
            const int st = 1 << (l - 1);
            const int base = 1 << (2 * (3 - l));
#pragma unroll
            for (int y = 0; y < 8; y += 2 * st)
#pragma unroll
              for (int x = 0; x < 8; x += 2 * st) {
                const int idx = base + 3 * ((y >> l) * (8 >> l) + (x >> l));
                const float ll = v[y][x], lh = val(idx), hl = val(idx + 1), hh = val(idx + 2);
                const float s0 = ll + lh, s1 = ll - lh, s2 = hl + hh, s3 = hl - hh;
                v[y][x] = s0 + s2;
                v[y][x + st] = s1 + s3;
                v[y + st][x] = s0 - s2;
                v[y + st][x + st] = s1 - s3;
              }
          }
          if (ch_ok) {
            const int pt = tok_t * 4 + half * 2 + pp;
            const int blk = pt / ppb;
            const int pi = pt - blk * ppb;
            const int py = pi / pw, px = pi - py * pw;
            const long o = ((long)blk * p.n_block + (long)(py * 8) * p.grid_w + px * 8) * p.n_out + ch;
#pragma unroll
            for (int y = 0; y < 8; ++y)
#pragma unroll
              for (int x = 0; x < 8; ++x) {
                const long oo = o + ((long)y * p.grid_w + x) * p.n_out;
                if constexpr (EPI == EPI_HAAR2D_F32)
                  static_cast<float*>(p.out)[oo] = fmaf(v[y][x], sw, bch);
                else
                  static_cast<__nv_bfloat16*>(p.out)[oo] = __float2bfloat16_rn(fmaf(v[y][x], sw, bch));
              }
          }
        }
      } else if constexpr (EPI == EPI_HAAR_F32 || EPI == EPI_HAAR_BF16) {
        static_assert(BN == 256, "the fused inverse works on 256-token tiles");
        // ---- the tile's eight coarse values (column 32 q), synthesised down to the level-5 sums
        float hd[8];
        {
          uint32_t h[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) ptx::tmem_ld_32x32b_x1(taddr + 32 * q, h[q]);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 8; ++q) hd[q] = static_cast<float>(static_cast<int>(h[q])) * sxs[32 * q];
        }
        float bch = 0.f;
        if (ch_ok) {
          if (p.a8v) hd[0] = __ldg(p.a8v + (long)tok_t * p.n_out + ch) * 0.0625f;   // 2^(-8/2)
          if (p.bias) bch = __ldg(p.bias + ch);
        }
        float a5[8];
        {
          float c2[4];
          if (p.depth == 8) {
            const float u0 = hd[0] + hd[1], u1 = hd[0] - hd[1];
            c2[0] = u0 + hd[2]; c2[1] = u0 - hd[2]; c2[2] = u1 + hd[3]; c2[3] = u1 - hd[3];
          } else if (p.depth == 7) {
            c2[0] = hd[0] + hd[2]; c2[1] = hd[0] - hd[2]; c2[2] = hd[1] + hd[3]; c2[3] = hd[1] - hd[3];
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) c2[i] = hd[i];
          }
          if (p.depth >= 6) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              a5[2 * i] = c2[i] + hd[4 + i];
              a5[2 * i + 1] = c2[i] - hd[4 + i];
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) a5[i] = hd[i];
          }
        }
        // ---- this warp's four chunks of 32 tokens: slot 0 <- level-5 sum, 31 details, five synthesis levels
        const int c0 = half * 4;
        uint32_t r[2][32];
        ptx::tmem_ld_32x32b_x32(taddr + c0 * 32, r[0]);
#pragma unroll
        for (int ci = 0; ci < 4; ++ci) {
          const int chunk = c0 + ci;
          ptx::tmem_ld_wait();
          if (ci + 1 < 4) ptx::tmem_ld_32x32b_x32(taddr + (chunk + 1) * 32, r[(ci + 1) & 1]);
          const uint32_t(&rc)[32] = r[ci & 1];
          float y[32];
          y[0] = half ? a5[4 + ci] : a5[ci];
#pragma unroll
          for (int len = 1; len < 32; len <<= 1) {
#pragma unroll
            for (int i = len - 1; i >= 0; --i) {
              const float d = static_cast<float>(static_cast<int>(rc[len + i])) * sxs[chunk * 32 + len + i];
              const float t = y[i];
              y[2 * i] = t + d;
              y[2 * i + 1] = t - d;
            }
          }
          if (ch_ok) {
            const long o = (long)(tok0 + chunk * 32) * p.n_out + ch;
            if constexpr (EPI == EPI_HAAR_F32) {
              float* out = static_cast<float*>(p.out) + o;
#pragma unroll
              for (int j = 0; j < 32; ++j) out[(long)j * p.n_out] = fmaf(y[j], sw, bch);
            } else {
              __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out) + o;
#pragma unroll
              for (int j = 0; j < 32; ++j) out[(long)j * p.n_out] = __float2bfloat16_rn(fmaf(y[j], sw, bch));
            }
          }
        }
      } else {
      constexpr int NCH = BN / 64;   // chunks of 32 tokens per warp
      const int c0 = half * NCH;
      uint32_t r[2][32];
      ptx::tmem_ld_32x32b_x32(taddr + c0 * 32, r[0]);
#pragma unroll
      for (int ci = 0; ci < NCH; ++ci) {
        const int chunk = c0 + ci;
        ptx::tmem_ld_wait();
        if (ci + 1 < NCH) ptx::tmem_ld_32x32b_x32(taddr + (chunk + 1) * 32, r[(ci + 1) & 1]);
        const uint32_t(&rc)[32] = r[ci & 1];
        const int tbase = tok0 + chunk * 32;
        if (EPI == EPI_DEQUANT_F32) {
          float* out = static_cast<float*>(p.out) + (long)tbase * p.n_out + ch;
          if (full_tile && ch_ok) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              out[(long)j * p.n_out] = static_cast<float>(static_cast<int>(rc[j])) * sxs[chunk * 32 + j] * sw;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (tbase + j < p.m_tok && ch_ok)
                out[(long)j * p.n_out] = static_cast<float>(static_cast<int>(rc[j])) * sxs[chunk * 32 + j] * sw;
          }
        } else if (EPI == EPI_DEQUANT_ZP_F32) {
          float* out = static_cast<float*>(p.out) + (long)tbase * p.n_out + ch;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (tbase + j < p.m_tok && ch_ok) {
              const long long v = static_cast<long long>(static_cast<int>(rc[j])) -
                                  static_cast<long long>(zps[chunk * 32 + j]) * wsum;
              out[(long)j * p.n_out] = __ll2float_rn(v) * sxs[chunk * 32 + j] * sw;
            }
        } else if (EPI == EPI_DEQUANT_BF16X2) {
          __nv_bfloat16* hi = static_cast<__nv_bfloat16*>(p.out) + (long)tbase * p.n_out + ch;
          __nv_bfloat16* lo = hi + (long)p.m_tok * p.n_out;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (tbase + j < p.m_tok && ch_ok) {
              const float v = static_cast<float>(static_cast<int>(rc[j])) * sxs[chunk * 32 + j] * sw;
              const __nv_bfloat16 h = __float2bfloat16_rn(v);
              hi[(long)j * p.n_out] = h;
              lo[(long)j * p.n_out] = __float2bfloat16_rn(v - __bfloat162float(h));
            }
        } else {
          int* out = static_cast<int*>(p.out) + (long)tbase * p.n_out + ch;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (tbase + j < p.m_tok && ch_ok) out[(long)j * p.n_out] = static_cast<int>(rc[j]);
        }
      }
      }
      ptx::tc_fence_before();
      if constexpr (PAIR) ptx::mbar_arrive_cluster(tempty_bar0 + static_cast<uint32_t>(a) * 8u); else ptx::mbar_arrive(&tempty[a]);
    }
    if (!ok) {
      *abort_word = 1;
      raise_device_status(STAMP_ERR_TIMEOUT);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  // neither CTA of a pair lets go of its shared and tensor memory while the other may still signal into it
  if constexpr (PAIR) ptx::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after();
    if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, 2 * BN); else ptx::tmem_dealloc(tmem_base, 2 * BN);
  }
}

}  // namespace stamp
