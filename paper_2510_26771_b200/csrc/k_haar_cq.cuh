// Fused Haar transform + per-token mixed-precision quantizer (Algorithm lines "X <- L X" and
// "x_i <- Q(x_i; b_i)"): one pass over the activation in HBM, up to five Haar levels per launch.
//
// The two axes pull in different directions: a transformed token's scale needs the maximum over
// ALL K channels of its row, while a Haar coefficient of level l needs 2^l consecutive tokens of
// ONE channel.  Here a thread owns two adjacent channels of a group of G = 2^P consecutive tokens
// and keeps all G coefficients of both channels in registers; a CTA owns a strip of channels; a
// thread-block cluster of C CTAs covers the whole feature axis.  The only thing the CTAs of a
// cluster exchange is the G per-row maxima of their strips, read from each other's shared memory
// (distributed shared memory, plain ld.shared::cluster) after one cluster barrier.  Every detail
// row of the P levels is then quantized from registers and stored; the group's un-normalised sum
// row (1/G of the data, fp32) is the input of the next launch, which runs the same kernel on
// fp32 rows, until the last launch also quantizes the approximation rows.
//
// Clusters are persistent: each walks over token groups with a stride of the number of clusters.
// bf16 activations are staged through a shared-memory ring filled by bulk asynchronous copies
// (one per token row of the strip) issued NS - 1 groups ahead, so HBM reads stay in flight while
// a group is being reduced, exchanged and stored; fp32 rows (the small later launches) are read
// with plain coalesced loads.
//
// Arithmetic: butterflies on un-normalised sums with packed fp32x2 operations, one multiplication
// by 2^(-j/2) per coefficient (head + tail FMA), scale = absmax / qmax by IEEE division, t / scale
// by reciprocal + one Newton step, round-to-nearest-even by the 1.5 * 2^23 trick.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

struct CqParams {
  const void* in;   // [nseq, Lin, K] bf16 / fp32 activations, or fp32 un-normalised sums over 2^lvl0 tokens
  float* aout;      // [nseq, Lin >> P, K] un-normalised sums over 2^(lvl0+P) tokens; nullptr in the last launch
  int K;            // channels
  int Kc;           // channels per CTA strip (= 2 * NCH * blockDim.x)
  int Lin;          // input rows per transform block in this launch
  int n;            // tokens per transform block
  int lvl0;         // Haar levels already applied to the input rows
  int k_hi;         // 8-bit rows per transform block
  float qmax_hi, qmax_lo;
  long ngroups;     // nseq * (Lin >> P)
  int nstages;      // depth of the shared-memory ring (bf16 input only)
  int8_t* a8;       // [M, K] one code per int8 (GEMM operand) or nullptr
  int8_t* q_hi;     // public outputs or nullptr
  uint8_t* q_lo;
  float* x_scale;   // [M]
  float* T_out;     // [M, K] transformed values (debug export) or nullptr
};

constexpr float CQ_MAGIC = 12582912.0f;          // 1.5 * 2^23
constexpr long long CQ_WAIT_LIMIT = 2000000000LL;  // SM clocks before a wait on a copy gives up

// What a launch writes besides the scales: the GEMM's int8 operand, the public packed codes, or
// the fp32 transformed values (debug export).
enum CqOut { CQ_OUT_A8 = 0, CQ_OUT_PUBLIC = 1, CQ_OUT_T = 2 };

// Row table in shared memory, rebuilt for every group; constants are stored twice so that a
// 128-bit load yields register pairs the packed fp32x2 instructions can use directly.
struct CqRowA { float nhi0, nhi1, nlo0, nlo1; };      // 2^(-j/2) as head + tail
struct CqRowB { float inv0, inv1, ns0, ns1; };        // 1 / scale and -scale
struct CqRowC { int row; int pub; };                  // logical row; row in q_hi / q_lo, bit 31 set for 8-bit rows

__device__ __forceinline__ float2 cq_f2(float a) { return make_float2(a, a); }

// Shared memory: [ring: nstages x G x Kc x sizeof(TIn)] [full barriers: 8 x u64] [maxima: 2 x 32 u32]
//                [row tables: 32 x (16 + 16 + 8) bytes]
template <int P, typename TIn>
__host__ __device__ constexpr size_t cq_slab_bytes(int Kc) { return (size_t)(1 << P) * Kc * sizeof(TIn); }
constexpr size_t CQ_TAIL_BYTES = 8 * 8 + 2 * 32 * 4 + 32 * 40;

template <int P, int NCH, typename TIn, int OUT>
__global__ void __launch_bounds__(512, 1) k_haar_cq(const CqParams p) {
  constexpr int G = 1 << P;
  constexpr bool STAGED = (sizeof(TIn) == 2);
  static_assert(G * NCH <= 32, "a thread holds at most 32 channel pairs");
  extern __shared__ __align__(128) uint8_t cq_smem[];
  const size_t slab = STAGED ? cq_slab_bytes<P, TIn>(p.Kc) : 0;
  uint8_t* tail = cq_smem + (STAGED ? slab * p.nstages : 0);
  uint64_t* full = reinterpret_cast<uint64_t*>(tail);
  unsigned* mymax = reinterpret_cast<unsigned*>(tail + 64);   // [2][32]
  float4* tabA = reinterpret_cast<float4*>(tail + 64 + 256);          // [32] CqRowA
  float4* tabB = reinterpret_cast<float4*>(tail + 64 + 256 + 512);    // [32] CqRowB
  int2* tabC = reinterpret_cast<int2*>(tail + 64 + 256 + 1024);       // [32] CqRowC
  __shared__ uint32_t abort_word;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31;
  unsigned csize, rank;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
  rank = ptx::cluster_ctarank();
  const long cid = blockIdx.x / csize, ncl = gridDim.x / csize;
  const int cbase = static_cast<int>(rank) * p.Kc;
  const int cvalid = max(0, min(p.Kc, p.K - cbase));   // channels of this strip (0: the strip is empty)
  const uint32_t row_bytes = static_cast<uint32_t>(cvalid) * sizeof(TIn);
  const int gps = p.Lin >> P;                           // groups per transform block
  const bool last = (p.aout == nullptr);
  const int NS = p.nstages;

  if (tid == 0) {
    abort_word = 0;
    if (STAGED) {
      for (int s = 0; s < NS; ++s) ptx::mbar_init(&full[s], 1);
      ptx::fence_mbar_init();
    }
  }
  __syncthreads();

  // warp 0 brings one group's rows of this strip into a ring stage: lane r copies token row r
  auto issue_load = [&](long grp, int stage) {
    if (!STAGED || cvalid == 0 || tid >= 32) return;
    const long sq = grp / gps;
    const long g = grp - sq * gps;
    const uint8_t* src = static_cast<const uint8_t*>(p.in) +
                         (((sq * p.Lin + g * G) * (long)p.K + cbase) * (long)sizeof(TIn));
    uint8_t* dst = cq_smem + stage * slab;
    if (lane == 0) ptx::mbar_arrive_expect_tx(&full[stage], row_bytes * G);
    __syncwarp();
    if (lane < G) ptx::bulk_load(dst + (size_t)lane * row_bytes, src + (size_t)lane * p.K * sizeof(TIn), row_bytes, &full[stage]);
  };

  if (STAGED)
    for (int s = 0; s < NS - 1; ++s) {
      const long grp = cid + s * ncl;
      if (grp < p.ngroups) issue_load(grp, s);
    }

  bool ok = true;
  long it = 0;
  for (long grp = cid; grp < p.ngroups; grp += ncl, ++it) {
    const int stage = static_cast<int>(it % NS);
    const int b = static_cast<int>(it & 1);
    if (STAGED && ok) {
      // the stage read in the previous iteration is free: every thread passed a barrier since
      const long nxt = grp + (long)(NS - 1) * ncl;
      if (nxt < p.ngroups) issue_load(nxt, static_cast<int>((it + NS - 1) % NS));
    }
    if (tid < 32) mymax[b * 32 + tid] = 0u;
    if (STAGED && cvalid > 0 && ok) {
      const bool got = ptx::mbar_wait_bounded(&full[stage], static_cast<uint32_t>((it / NS) & 1), &abort_word, CQ_WAIT_LIMIT);
      if (!got) abort_word = 1;
    }
    __syncthreads();
    if (ok && abort_word != 0) {
      ok = false;
      if (tid == 0) raise_device_status(STAMP_ERR_TIMEOUT);
    }

    const long sq = grp / gps;
    const int g = static_cast<int>(grp - sq * gps);

    // ---- load G tokens x NCH channel pairs, butterflies in registers (un-normalised)
    float2 v[NCH][G];
    bool valid[NCH];
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int pr = tid + j * NT;          // channel pair inside the strip
      valid[j] = ok && (2 * pr < cvalid);
#pragma unroll
      for (int r = 0; r < G; ++r) v[j][r] = cq_f2(0.f);
      if (valid[j]) {
        if (STAGED) {
          const uint32_t* s32 = reinterpret_cast<const uint32_t*>(cq_smem + stage * slab) + pr;
#pragma unroll
          for (int r = 0; r < G; ++r) {
            const uint32_t w = s32[(size_t)r * (row_bytes / 4)];
            v[j][r] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
          }
        } else {
          const float* src = static_cast<const float*>(p.in) + ((sq * p.Lin + (long)g * G) * (long)p.K + cbase + 2 * pr);
#pragma unroll
          for (int r = 0; r < G; ++r) v[j][r] = *reinterpret_cast<const float2*>(src + (long)r * p.K);
        }
      }
#pragma unroll
      for (int len = G; len > 1; len >>= 1) {
        float2 t[G];
#pragma unroll
        for (int i = 0; i < len / 2; ++i) {
          t[i] = __fadd2_rn(v[j][2 * i], v[j][2 * i + 1]);
          t[len / 2 + i] = __ffma2_rn(v[j][2 * i + 1], cq_f2(-1.0f), v[j][2 * i]);
        }
#pragma unroll
        for (int i = 0; i < len; ++i) v[j][i] = t[i];
      }
    }
    // v[j] is now [a | d_P | d_(P-1) (2) | ... | d_1 (G/2)]

    // ---- per-row maxima of this strip: lane r of every warp collects row r, one atomic per lane
    unsigned keep = 0u;
#pragma unroll
    for (int r = 0; r < G; ++r) {
      float m = 0.f;
#pragma unroll
      for (int j = 0; j < NCH; ++j) m = fmaxf(m, fmaxf(fabsf(v[j][r].x), fabsf(v[j][r].y)));
      const unsigned mm = __reduce_max_sync(0xffffffffu, __float_as_uint(m));
      keep = (lane == r) ? mm : keep;
    }
    if (lane < G) atomicMax(&mymax[b * 32 + lane], keep);
    __syncthreads();
    ptx::cluster_arrive();
    if (!last) {
#pragma unroll
      for (int j = 0; j < NCH; ++j)
        if (valid[j])
          *reinterpret_cast<float2*>(p.aout + ((sq * gps + g) * (long)p.K + cbase + 2 * (tid + j * NT))) = v[j][0];
    }
    ptx::cluster_wait();

    // ---- row tables: maxima over the cluster, scales, output rows
    if (tid < G && (tid > 0 || last)) {
      const int r = tid;
      unsigned um = 0;
      const uint32_t local = ptx::smem_u32(&mymax[b * 32 + r]);
      for (unsigned q = 0; q < csize; ++q) {
        unsigned x;
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(x) : "r"(ptx::mapa(local, q)));
        um = max(um, x);
      }
      int k = 0;                       // r in [2^k, 2^(k+1)): detail row of local level P - k
      while ((2 << k) <= r) ++k;
      const int l = (r == 0) ? P : P - k;
      const int j = p.lvl0 + l;
      const int i_in_blk = (r == 0) ? g : (p.n >> j) + (g << k) + (r - (1 << k));
      const HaarNorm h = haar_norm(j);
      const float u = __uint_as_float(um);
      const float amax = fmaf(u, h.hi, u * h.lo);
      const bool hi = i_in_blk < p.k_hi;
      const float qmax = hi ? p.qmax_hi : p.qmax_lo;
      const float scale = (amax > 0.f) ? __fdiv_rn(amax, qmax) : 1.0f;
      const float inv = __fdiv_rn(1.0f, scale);
      const long row = sq * p.n + i_in_blk;
      const long pub = hi ? sq * p.k_hi + i_in_blk : sq * (p.n - p.k_hi) + (i_in_blk - p.k_hi);
      tabA[r] = make_float4(h.hi, h.hi, h.lo, h.lo);
      tabB[r] = make_float4(inv, inv, -scale, -scale);
      tabC[r] = make_int2(static_cast<int>(row), static_cast<int>(pub) | (hi ? static_cast<int>(0x80000000u) : 0));
      if (rank == 0 && ok) p.x_scale[row] = scale;
    }
    __syncthreads();

    // ---- normalise, quantize and store from registers
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      if (!valid[j]) continue;
      const int c = cbase + 2 * (tid + j * NT);
      const int8_t* a8c = p.a8 + c;
      const int8_t* qhc = p.q_hi + c;
      const uint8_t* qlc = p.q_lo + (c >> 1);
      const float* Tc = p.T_out + c;
#pragma unroll
      for (int r = 0; r < G; ++r) {
        if (r == 0 && !last) continue;
        const float4 A = tabA[r];
        const int2 Cc = tabC[r];
        const float2 t = __ffma2_rn(v[j][r], make_float2(A.x, A.y), __fmul2_rn(v[j][r], make_float2(A.z, A.w)));
        if (OUT == CQ_OUT_T) {
          *const_cast<float2*>(reinterpret_cast<const float2*>(Tc + (long)Cc.x * p.K)) = t;
          continue;
        }
        const float4 Bv = tabB[r];
        const float2 inv2 = make_float2(Bv.x, Bv.y);
        const float2 q0 = __fmul2_rn(t, inv2);
        const float2 rem = __ffma2_rn(q0, make_float2(Bv.z, Bv.w), t);
        const float2 q = __fadd2_rn(__ffma2_rn(rem, inv2, q0), cq_f2(CQ_MAGIC));
        const uint32_t bx = __float_as_uint(q.x), by = __float_as_uint(q.y);
        if (OUT == CQ_OUT_A8) {
          *const_cast<uint16_t*>(reinterpret_cast<const uint16_t*>(a8c + (long)Cc.x * p.K)) =
              static_cast<uint16_t>(__byte_perm(bx, by, 0x0040));
        } else if (Cc.y < 0) {
          *const_cast<uint16_t*>(reinterpret_cast<const uint16_t*>(qhc + (long)(Cc.y & 0x7FFFFFFF) * p.K)) =
              static_cast<uint16_t>(__byte_perm(bx, by, 0x0040));
        } else {
          *const_cast<uint8_t*>(qlc + (long)Cc.y * (p.K >> 1)) = static_cast<uint8_t>((bx & 0xFu) | ((by << 4) & 0xF0u));
        }
      }
    }
    // the row tables and the ring stage are reused in the next iteration: its first barrier orders that
  }
  if (STAGED && !ok) {
    // copies issued ahead were never consumed: give them time to land before the shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {
    }
  }
  // nobody leaves while a peer may still read its maxima
  ptx::cluster_sync();
}

}  // namespace stamp
