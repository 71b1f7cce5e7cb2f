// Integer GEMM with per-block ("group") scales along the feature axis on the tensor cores (the LVM table's W4A4
// setting with blocks of 64 features; App. "Experimental details / LVMs"; the product step of Algorithm 1 with
//     Yt[m, n] = sum_g ( sum_{k in g} q[m, k] wq[n, k] ) * sx[m, g] * sw[n, g] ).
// The integer partial sum of every group has to be scaled on its own, so the accumulator cannot run over all of K:
// the MMA thread accumulates ONE group (group / 32 instructions of kind::i8, 128 channels x 128 tokens) into one of
// four tensor-memory accumulators and commits it; the epilogue warps drain that accumulator, scale it by
// sx[token, g] * sw[channel, g] and add it to fp32 sums they keep in registers (32 per thread) while the next group
// fills the next accumulator.  The drain is the longer of the two (4 CUDA-core instructions per product of a
// 64-feature group against 1 / 64 of a tensor instruction), so this kernel runs at a fraction of the int8 rate by
// construction -- and an order of magnitude above the CUDA-core dp4a product it replaces (k_grouped.cuh, kept for
// the shapes this kernel does not take).
// Operand roles as in k_gemm.cuh: weights are the MMA A operand (128 channels = TMEM lanes), tokens the B operand
// (128 columns): an epilogue thread owns one channel and 32 tokens, a warp's store covers 32 consecutive channels.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

struct GgtParams {
  int n_out;             // N output channels
  int m_tok;             // M tokens
  int k;                 // K features, a multiple of 128
  int group;             // features per scale: 64 * 2^i, at most 4096
  const float* x_scale;  // [m_tok, k / group]
  const float* w_scale;  // [n_out, k / group]
  float* out;            // [m_tok, n_out]
};

constexpr int GGT_BM = 128, GGT_BN = 128, GGT_BK = 128, GGT_STAGES = 4;
constexpr int GGT_NACC = 4;            // TMEM accumulators (all 512 columns): groups in flight between MMA and drain
constexpr int GGT_EPI_THREADS = 512;   // sixteen epilogue warps: four per quarter of the TMEM lanes, 32 columns each
constexpr int GGT_THREADS = 64 + GGT_EPI_THREADS;
constexpr int GGT_MAX_GROUPS = 128;   // token scales of a tile staged in shared memory: [groups][128 tokens]
constexpr int GGT_STAGE_BYTES = (GGT_BM + GGT_BN) * GGT_BK;
constexpr int GGT_BAR_OFFSET = GGT_STAGES * GGT_STAGE_BYTES;
constexpr int GGT_NUM_BARS = 2 * GGT_STAGES + 2 * GGT_NACC;   // full, empty, gfull, gempty
constexpr int GGT_SX_OFFSET = GGT_BAR_OFFSET + GGT_NUM_BARS * 8 + 16;
constexpr int GGT_DYN_BYTES = GGT_SX_OFFSET + GGT_MAX_GROUPS * GGT_BN * 4 + 1024;
constexpr long long GGT_WAIT_LIMIT = 4000000000LL;

__global__ void __launch_bounds__(GGT_THREADS, 1)
    k_gemm_grouped_tc(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, GgtParams p) {
  extern __shared__ uint8_t ggt_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ggt_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + GGT_BAR_OFFSET);
  uint64_t* empty = full + GGT_STAGES;
  uint64_t* gfull = empty + GGT_STAGES;
  uint64_t* gempty = gfull + GGT_NACC;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gempty + GGT_NACC);
  volatile uint32_t* abort_word = tmem_slot + 1;
  float* sxs = reinterpret_cast<float*>(smem + GGT_SX_OFFSET);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int ch_tiles = (p.n_out + GGT_BM - 1) / GGT_BM;
  const int tok_tiles = (p.m_tok + GGT_BN - 1) / GGT_BN;
  const int num_tiles = ch_tiles * tok_tiles;
  const int num_kb = p.k / GGT_BK;
  const int ng = p.k / p.group;
  const int mma_per_group = p.group / 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < GGT_STAGES; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < GGT_NACC; ++a) {
      ptx::mbar_init(&gfull[a], 1);
      ptx::mbar_init(&gempty[a], GGT_EPI_THREADS / 32);   // one arrival per epilogue warp
    }
    *abort_word = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_w);
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, GGT_NACC * GGT_BN);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int tok_t = tile / ch_tiles, ch_t = tile - tok_t * ch_tiles;   // channel tiles fastest: CTAs share token tiles
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait_bounded_sleepy(&empty[stage], phase ^ 1u, abort_word, GGT_WAIT_LIMIT)) {
            ok = false;
            break;
          }
          uint8_t* ws = smem + stage * GGT_STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(&full[stage], GGT_STAGE_BYTES);
          ptx::tma_load_2d(ws, &tmap_w, &full[stage], kb * GGT_BK, ch_t * GGT_BM);
          ptx::tma_load_2d(ws + GGT_BM * GGT_BK, &tmap_x, &full[stage], kb * GGT_BK, tok_t * GGT_BN);
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == GGT_STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
        for (int s = 0; s < GGT_STAGES; ++s)   // let the copies in flight land before the shared memory goes away
          if (armed & (1u << s)) {
            const long long t0 = clock64();
            while (!ptx::mbar_try_wait(&full[s], (armed_parity >> s) & 1u) && clock64() - t0 < 2000000LL) {
            }
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: one accumulator per group
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::make_i8_idesc(GGT_BM, GGT_BN);
      int stage = 0;
      uint32_t phase = 0;
      unsigned gcount = 0;   // groups issued so far: accumulator gcount % GGT_NACC, its (gcount / GGT_NACC)-th filling
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int in_group = 0;    // instructions issued into the current group
        for (int kb = 0; kb < num_kb && ok; ++kb) {
          if (!ptx::mbar_wait_bounded_sleepy(&full[stage], phase, abort_word, GGT_WAIT_LIMIT)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t wa = ptx::smem_u32(smem + stage * GGT_STAGE_BYTES);
          const uint32_t xa = wa + GGT_BM * GGT_BK;
          for (int k = 0; k < GGT_BK / 32; ++k) {
            const int a = static_cast<int>(gcount % GGT_NACC);
            if (in_group == 0) {   // a new group: its accumulator must have been drained
              if (!ptx::mbar_wait_bounded_sleepy(&gempty[a], ((gcount / GGT_NACC) & 1u) ^ 1u, abort_word, GGT_WAIT_LIMIT)) {
                ok = false;
                break;
              }
              ptx::tc_fence_after();
            }
            const uint64_t adesc = ptx::make_kmajor_sw128_desc(wa + k * 32);
            const uint64_t bdesc = ptx::make_kmajor_sw128_desc(xa + k * 32);
            ptx::mma_i8_ss(tmem_base + static_cast<uint32_t>(a * GGT_BN), adesc, bdesc, idesc, in_group != 0 ? 1u : 0u);
            if (++in_group == mma_per_group) {
              ptx::tc_commit(&gfull[a]);
              in_group = 0;
              ++gcount;
            }
          }
          if (ok) ptx::tc_commit(&empty[stage]);
          if (++stage == GGT_STAGES) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        *abort_word = 1;
        raise_device_status(STAMP_ERR_TIMEOUT);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int colq = (warp - 2) >> 2;     // which 32 of the accumulator's 128 columns this warp drains
    const int ep_tid = threadIdx.x - 64;
    unsigned gcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int tok_t = tile / ch_tiles, ch_t = tile - tok_t * ch_tiles;
      const int ch = ch_t * GGT_BM + row;
      const int tok0 = tok_t * GGT_BN;
      const bool ch_ok = ch < p.n_out;
      // The tile's token scales, [group][token]; every epilogue thread is through with the previous tile's first.
      // All eight warps pass both barriers of every tile whatever happened before: a warp whose wait ran out
      // raises the abort word, the others read it behind the second barrier, and from then on everybody only
      // walks through the remaining tiles -- nobody is left waiting at a barrier for a warp that gave up.
      asm volatile("bar.sync 1, %0;" ::"n"(GGT_EPI_THREADS) : "memory");
      if (ok)
        for (int e = ep_tid; e < GGT_BN * ng; e += GGT_EPI_THREADS) {
          const int g = e >> 7, tok = e & (GGT_BN - 1);   // consecutive threads: consecutive tokens of one group
          sxs[e] = (tok0 + tok < p.m_tok) ? __ldg(p.x_scale + (size_t)(tok0 + tok) * ng + g) : 0.f;
        }
      asm volatile("bar.sync 1, %0;" ::"n"(GGT_EPI_THREADS) : "memory");
      if (*abort_word != 0u) ok = false;
      if (!ok) continue;
      float2 acc[16];   // column pairs, as the packed fp32 instructions take them
#pragma unroll
      for (int c = 0; c < 16; ++c) acc[c] = make_float2(0.f, 0.f);
      const float* swp = p.w_scale + (size_t)(ch_ok ? ch : 0) * ng;
      float sw_next = ch_ok ? __ldg(swp) : 0.f;
      for (int g = 0; g < ng; ++g, ++gcount) {
        const int a = static_cast<int>(gcount % GGT_NACC);
        const float sw = sw_next;
        if (g + 1 < ng) sw_next = ch_ok ? __ldg(swp + g + 1) : 0.f;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded_sleepy(&gfull[a], (gcount / GGT_NACC) & 1u, abort_word, GGT_WAIT_LIMIT))) {
          ok = false;
          *abort_word = 1;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(a * GGT_BN + colq * 32);
        // two chunks of 16 columns, the next chunk's load in flight while this one is scaled: int32 -> float, then,
        // two columns at a time on packed fp32 instructions, one multiply for the scale pair and one fused
        // multiply-add per product.
        const float4* sxg = reinterpret_cast<const float4*>(sxs + g * GGT_BN + colq * 32);
        const float2 sw2 = make_float2(sw, sw);
        uint32_t r[2][16];
        ptx::tmem_ld_32x32b_x16(taddr, r[0]);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          ptx::tmem_ld_wait();
          if (q < 1) {
            ptx::tmem_ld_32x32b_x16(taddr + 16 * (q + 1), r[(q + 1) & 1]);
          } else {
            // the partial sums are in registers (the wait above is warp-wide): the accumulator may take a new group;
            // one arrival per warp
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&gempty[a]);
          }
          const uint32_t(&x)[16] = r[q & 1];
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const float4 s4 = sxg[4 * q + v];
            const int c2 = 8 * q + 2 * v;
            const float2 f01 = make_float2(static_cast<float>(static_cast<int>(x[4 * v])), static_cast<float>(static_cast<int>(x[4 * v + 1])));
            const float2 f23 = make_float2(static_cast<float>(static_cast<int>(x[4 * v + 2])), static_cast<float>(static_cast<int>(x[4 * v + 3])));
            acc[c2] = __ffma2_rn(f01, __fmul2_rn(make_float2(s4.x, s4.y), sw2), acc[c2]);
            acc[c2 + 1] = __ffma2_rn(f23, __fmul2_rn(make_float2(s4.z, s4.w), sw2), acc[c2 + 1]);
          }
        }
      }
      if (ok && ch_ok) {
        float* out = p.out + (size_t)(tok0 + colq * 32) * p.n_out + ch;
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (tok0 + colq * 32 + c < p.m_tok) out[(size_t)c * p.n_out] = (c & 1) ? acc[c >> 1].y : acc[c >> 1].x;
      }
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
    ptx::tmem_dealloc(tmem_base, GGT_NACC * GGT_BN);
  }
}

}  // namespace stamp
