// Host layer of the STaMP CUDA library: argument validation, workspace layout, tensor maps,
// kernel selection and launch.  Every extern "C" entry point of include/stamp.h is defined here.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "k_dct.cuh"
#include "k_dct_tc.cuh"
#include "k_debug.cuh"
#include "k_gemm.cuh"
#include "k_haar2d.cuh"
#include "k_generic.cuh"
#include "k_grouped.cuh"
#include "k_gemm_grouped_tc.cuh"
#include "k_haar_cq.cuh"
#include "k_haar_tc.cuh"
#include "k_peak.cuh"
#include "k_top_gemv.cuh"
#include "stamp.h"

namespace stamp {

static thread_local int t_launches = 0;
static thread_local cudaEvent_t t_gemm_ev_start = nullptr, t_gemm_ev_stop = nullptr;

#define STAMP_CHECK_LAUNCH()                                   \
  do {                                                         \
    ++t_launches;                                              \
    if (cudaGetLastError() != cudaSuccess) return STAMP_ERR_CUDA; \
  } while (0)

static inline bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
static inline int ilog2(int v) {
  int l = 0;
  while ((1 << l) < v) ++l;
  return l;
}
static inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

// ------------------------------------------------------------------------------------------
// Validation: stamp_config + sizes -> Problem
// ------------------------------------------------------------------------------------------
static int resolve(const stamp_config* cfg, int B, int L, int K, int N, bool need_n, Problem* out) {
  if (!cfg || !out) return STAMP_ERR_INVALID_ARG;
  if (B <= 0 || L <= 0 || K <= 0 || (need_n && N <= 0)) return STAMP_ERR_INVALID_ARG;
  if (cfg->transform < STAMP_T_IDENTITY || cfg->transform > STAMP_T_HAAR_SKIP1) return STAMP_ERR_INVALID_ARG;
  if (cfg->block < 0 || cfg->levels < 0 || cfg->k_hi < 0 || cfg->grid_w < 0) return STAMP_ERR_INVALID_ARG;
  if (cfg->transform != STAMP_T_HAAR2D && cfg->grid_w != 0) return STAMP_ERR_INVALID_ARG;
  if (cfg->bits_hi != 8 || cfg->bits_lo != 4 || cfg->bits_w != 4) return STAMP_ERR_UNSUPPORTED;
  if (cfg->group < 0) return STAMP_ERR_INVALID_ARG;
  if (cfg->group == 0) {
    if (cfg->act_gran != STAMP_G_PER_TOKEN || cfg->w_gran != STAMP_G_PER_CHANNEL) return STAMP_ERR_UNSUPPORTED;
  } else {
    // per-block scales: both operands, groups of 64 * 2^i features that divide K, symmetric codes
    if (cfg->act_gran != STAMP_G_GROUP || cfg->w_gran != STAMP_G_GROUP) return STAMP_ERR_INVALID_ARG;
    if (cfg->group % 64 != 0 || !is_pow2(cfg->group) || K % cfg->group != 0 || cfg->act_zero_point) return STAMP_ERR_UNSUPPORTED;
  }
  if (cfg->act_zero_point != 0 && cfg->act_zero_point != 1) return STAMP_ERR_INVALID_ARG;
  const int n = cfg->block ? cfg->block : L;
  if (!is_pow2(n) || L % n != 0) return STAMP_ERR_UNSUPPORTED;
  if (cfg->k_hi > n) return STAMP_ERR_INVALID_ARG;
  if (K % 128 != 0) return STAMP_ERR_UNSUPPORTED;
  if (need_n && N % 8 != 0) return STAMP_ERR_UNSUPPORTED;
  if ((long)B * L > (1L << 30)) return STAMP_ERR_UNSUPPORTED;
  int levels = 0;
  if (cfg->transform == STAMP_T_HAAR || cfg->transform == STAMP_T_HAAR_SKIP1) {
    if (cfg->transform == STAMP_T_HAAR_SKIP1 && n < 2) return STAMP_ERR_UNSUPPORTED;
    const int full = ilog2(n);
    levels = cfg->levels ? cfg->levels : full;
    if (levels > full) return STAMP_ERR_UNSUPPORTED;
  }
  if ((cfg->transform == STAMP_T_DCT2 || cfg->transform == STAMP_T_WHT) && n > 4096)
    return STAMP_ERR_UNSUPPORTED;  // dense n x n matrix in scratch
  if (cfg->transform == STAMP_T_HAAR2D) {
    const int w = cfg->grid_w;
    if (w <= 0 || n % w != 0) return STAMP_ERR_INVALID_ARG;
    levels = cfg->levels;
    if (levels < 1 || levels > 3 || (w & ((1 << levels) - 1)) != 0 || ((n / w) & ((1 << levels) - 1)) != 0)
      return STAMP_ERR_UNSUPPORTED;
  }
  out->B = B;
  out->L = L;
  out->K = K;
  out->N = need_n ? N : 0;
  out->transform = cfg->transform;
  out->n = n;
  out->levels = levels;
  out->k_hi = cfg->k_hi;
  out->grid_w = cfg->grid_w;
  out->act_zp = cfg->act_zero_point;
  out->group = cfg->group;
  out->nseq = B * (L / n);
  out->M = (long)B * L;
  out->qmax_hi = (1 << (cfg->bits_hi - 1)) - 1;
  out->qmax_lo = (1 << (cfg->bits_lo - 1)) - 1;
  out->qmax_w = (1 << (cfg->bits_w - 1)) - 1;
  return STAMP_OK;
}

static bool dtype_ok(int d) { return d == STAMP_F32 || d == STAMP_BF16; }

// ------------------------------------------------------------------------------------------
// Multi-pass plan for the Haar kernels: up to 5 levels per pass, finest first.
// ------------------------------------------------------------------------------------------
struct PassPlan {
  int npass;
  int p[8];
};
static PassPlan make_plan(int levels) {
  PassPlan pl{};
  int rem = levels;
  if (rem == 0) {
    pl.npass = 1;
    pl.p[0] = 0;
    return pl;
  }
  while (rem > 0) {
    const int p = rem > 5 ? 5 : rem;
    pl.p[pl.npass++] = p;
    rem -= p;
  }
  return pl;
}

// ------------------------------------------------------------------------------------------
// Workspace layout (one layout for all calls of a problem size).
// ------------------------------------------------------------------------------------------
struct Workspace {
  size_t rowmax, htc_cnt, xscale, skipa, T, ping, pong, atop, top_ping, top_pong, dctmat, a8, w8, yt, a8top, sxtop, yttop, a8v, dctsplit, xzero, wsum, total;
};
static Workspace layout(const Problem& pb) {
  Workspace w{};
  const size_t M = (size_t)pb.M;
  const size_t KN = (size_t)(pb.K > pb.N ? pb.K : pb.N);
  const PassPlan pl = make_plan(pb.levels);
  const size_t ping_rows = pl.npass > 1 ? (M >> pl.p[0]) : 0;
  const size_t pong_rows = pl.npass > 2 ? (M >> (pl.p[0] + pl.p[1])) : 0;
  size_t off = 0;
  w.rowmax = off; off += align256(M * 4);
  // (directly behind the row maxima: one memset clears both before the tensor-core transform+quantize launch)
  // tile counts [M / 128], CTA count [4 words], coarse-row maxima [M / 128], strip counts per block [nseq]
  w.htc_cnt = off; off += align256(((M >> 7) * 2 + 4 + (size_t)pb.nseq) * 4 + 16);
  w.xscale = off; off += align256(M * 4 * (size_t)(pb.group ? pb.K / pb.group : 1));
  // low-pass band after the first level of the first-token-excluded Haar transform (forward: K wide, inverse: N wide)
  w.skipa = off;  off += align256(pb.transform == STAMP_T_HAAR_SKIP1 ? (M / 2) * KN * 4 : 0);
  w.T = off;      off += align256(M * (size_t)pb.K * 4);
  w.ping = off;   off += align256(ping_rows * KN * 4);
  w.pong = off;   off += align256(pong_rows * KN * 4);
  // un-normalised sums handed from one launch of the fused transform+quantize kernel to the next
  // (at least 3 levels per launch but the last, so each buffer is 1/8 of the one before at most)
  w.atop = off;     off += align256((M >> 3) * (size_t)pb.K * 4);
  w.top_ping = off; off += align256((M >> 6) * (size_t)pb.K * 4);
  w.top_pong = off; off += align256((M >> 9) * (size_t)pb.K * 4);
  const bool dense = pb.transform == STAMP_T_DCT2 || pb.transform == STAMP_T_WHT;
  w.dctmat = off; off += align256(dense ? (size_t)pb.n * pb.n * 4 : 0);
  // the top table follows the M rows of a8 directly: the tiled route addresses it as rows M, M + 1, ...
  w.a8 = off;     off += M * (size_t)pb.K;
  w.a8top = off;  off += align256((M >> 8) * (size_t)pb.K) + 256;
  off = align256(off);
  w.w8 = off;     off += align256((size_t)pb.N * pb.K);
  w.yt = off;     off += align256(M * (size_t)pb.N * 4);
  // rows above the GEMM's 256-token tiles (Haar levels > 8): codes, scales, their GEMM output, its inverse
  w.sxtop = off;  off += align256((M >> 8) * 4 + 4);
  w.yttop = off;  off += align256((M >> 8) * (size_t)pb.N * 4);
  w.a8v = off;    off += align256((M >> 8) * (size_t)pb.N * 4);
  // bf16 terms of the DCT matrix and of its transpose (tensor-core DCT)
  w.dctsplit = off; off += align256(dense ? (size_t)2 * 3 * DCT_N * DCT_N * 2 : 0);
  // zero-point activation codes: per-token zero points and the weight row sums of the correction term
  w.xzero = off;  off += align256(pb.act_zp ? M * 4 : 0);
  w.wsum = off;   off += align256(pb.act_zp ? (size_t)pb.N * 4 : 0);
  w.total = off;
  return w;
}
static int check_ws(const Workspace& w, const void* ws, size_t ws_bytes) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < w.total) return STAMP_ERR_WORKSPACE;
  return STAMP_OK;
}

// ------------------------------------------------------------------------------------------
// Tensor maps (driver entry point fetched through the runtime; no link against libcuda).
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// int8 matrix [rows, K] row-major; box = 128 bytes of K x box_rows rows, 128-byte swizzle.
static int make_tmap_i8(const void* base, long rows, int K, int box_rows, CUtensorMap* out) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return STAMP_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0) return STAMP_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K};
  cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? STAMP_OK : STAMP_ERR_CUDA;
}

// bf16 matrix [rows, cols] row-major; box = 64 columns (128 bytes) x box_rows rows, 128-byte swizzle.
static int make_tmap_bf16(const void* base, long rows, long cols, CUtensorMap* out, int box_rows = 256) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return STAMP_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0) return STAMP_ERR_INVALID_ARG;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? STAMP_OK : STAMP_ERR_CUDA;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while the previous
// kernel of the stream drains; it calls grid_dependency_wait() before touching that kernel's output.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t lc{};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kern, KArgs(args)...);
}

// Per-device facts and settings.  A process may use the library on several GPUs: the SM count, the
// opt-in to more than 48 KB of dynamic shared memory (a per-device function attribute) and the number of
// resident clusters are therefore cached per device, under one mutex (host threads may call concurrently).
constexpr int MAX_DEVICES = 64;
static std::mutex g_dev_mu;

static int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
  return dev;
}

static int sm_count() {
  static int n_of[MAX_DEVICES] = {};
  const int dev = current_device();
  if (dev < 0) return 148;
  std::lock_guard<std::mutex> lock(g_dev_mu);
  if (n_of[dev] == 0) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    n_of[dev] = n > 0 ? n : 148;
  }
  return n_of[dev];
}

// Make sure `func` may be launched with `bytes` of dynamic shared memory on the current device.
static int ensure_dyn_smem(const void* func, size_t bytes) {
  static std::unordered_map<unsigned long long, size_t> granted;   // (device, function) -> bytes already allowed
  const int dev = current_device();
  if (dev < 0) return STAMP_ERR_CUDA;
  const unsigned long long key = (static_cast<unsigned long long>(dev) << 56) ^ reinterpret_cast<uintptr_t>(func);
  std::lock_guard<std::mutex> lock(g_dev_mu);
  size_t& have = granted[key];
  if (bytes > have) {
    if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
      cudaGetLastError();
      return STAMP_ERR_CUDA;
    }
    have = bytes;
  }
  return STAMP_OK;
}

// ------------------------------------------------------------------------------------------
// Launchers
// ------------------------------------------------------------------------------------------
template <int MODE, int NATOM, int NPLANE>
static int launch_dct_tc(const CUtensorMap& ta, const CUtensorMap& tb0, const CUtensorMap& tb1, const DctTcParams& dp,
                         cudaStream_t st) {
  using SM = DctSmem<NATOM, NPLANE>;
  auto kern = k_dct_tc<MODE, NATOM, NPLANE>;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), SM::DYN_BYTES)) return rc;
  const int tiles = dp.nblk * (dp.cols / (NATOM * 64));
  const int grid = tiles < sm_count() ? tiles : sm_count();
  if (launch_pdl(kern, dim3((unsigned)grid), dim3(DCT_THREADS), SM::DYN_BYTES, st, ta, tb0, tb1, dp) != cudaSuccess) {
    cudaGetLastError();
    return STAMP_ERR_CUDA;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

template <int BN, int STAGES, int EPI, bool PAIR = false>
static int launch_gemm_t(const CUtensorMap& tw, const CUtensorMap& tx, const GemmParams& gp, cudaStream_t st) {
  using SM = GemmSmem<BN, STAGES, PAIR>;
  auto kern = k_gemm_i8<BN, STAGES, EPI, PAIR>;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), SM::DYN_BYTES)) return rc;
  const int ch_tiles = (gp.n_out + (PAIR ? 2 : 1) * GEMM_BM - 1) / ((PAIR ? 2 : 1) * GEMM_BM);
  const int tok_tiles = (gp.m_tok + BN - 1) / BN;
  const int tiles = ch_tiles * tok_tiles;
  const int slots = PAIR ? sm_count() / 2 : sm_count();
  const int grid = (tiles < slots ? tiles : slots) * (PAIR ? 2 : 1);
  const bool timed = t_gemm_ev_start && t_gemm_ev_stop;
  if (timed) cudaEventRecord(t_gemm_ev_start, st);
  if (PAIR) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3(GEMM_THREADS);
    lc.dynamicSmemBytes = SM::DYN_BYTES;
    lc.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 2;
    cudaLaunchKernelEx(&lc, kern, tw, tx, gp);
  } else {
    launch_pdl(kern, dim3((unsigned)grid), dim3(GEMM_THREADS), SM::DYN_BYTES, st, tw, tx, gp);
  }
  if (timed) cudaEventRecord(t_gemm_ev_stop, st);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// acc/out[tok, ch] from int8 operands a8 [M, K], w8 [N, K].
static int launch_gemm(const int8_t* a8, const int8_t* w8, long M, int N, int K, const float* x_scale,
                       const float* w_scale, void* out, int epi, cudaStream_t st, const float* bias = nullptr,
                       const float* a8v = nullptr, int depth = 0, const int* x_zero = nullptr,
                       const int* w_sum = nullptr, int grid_w = 0, int n_block = 0) {
  GemmParams gp{};
  gp.n_out = N;
  gp.m_tok = (int)M;
  gp.k = K;
  gp.x_scale = x_scale;
  gp.w_scale = w_scale;
  gp.out = out;
  gp.group = 16;
  gp.bias = bias;
  gp.a8v = a8v;
  gp.depth = depth;
  gp.x_zero = x_zero;
  gp.w_sum = w_sum;
  gp.grid_w = grid_w;
  gp.n_block = n_block;
  CUtensorMap tw, tx;
  int rc = make_tmap_i8(w8, N, K, GEMM_BM, &tw);
  if (rc) return rc;
  // 256 tokens and more: CTA pairs, each CTA staging 128 tokens of the pair's 256-token tile
  const bool wide = M >= 256;
  rc = make_tmap_i8(a8, M, K, 128, &tx);
  if (rc) return rc;
  if (epi == EPI_HAAR_F32 || epi == EPI_HAAR_BF16) {
    if (!wide || M % 256 != 0 || depth < 5 || depth > 8) return STAMP_ERR_UNSUPPORTED;
    if (epi == EPI_HAAR_F32) return launch_gemm_t<256, 6, EPI_HAAR_F32, true>(tw, tx, gp, st);
    return launch_gemm_t<256, 6, EPI_HAAR_BF16, true>(tw, tx, gp, st);
  }
  if (epi == EPI_DEQUANT_BF16X2)
    return wide ? launch_gemm_t<256, 6, EPI_DEQUANT_BF16X2, true>(tw, tx, gp, st)
                : launch_gemm_t<128, 6, EPI_DEQUANT_BF16X2>(tw, tx, gp, st);
  if (epi == EPI_HAAR2D_F32 || epi == EPI_HAAR2D_BF16) {
    if (!wide || M % 256 != 0 || grid_w < 8 || grid_w % 8 != 0 || n_block % (8 * grid_w) != 0) return STAMP_ERR_UNSUPPORTED;
    if (epi == EPI_HAAR2D_F32) return launch_gemm_t<256, 6, EPI_HAAR2D_F32, true>(tw, tx, gp, st);
    return launch_gemm_t<256, 6, EPI_HAAR2D_BF16, true>(tw, tx, gp, st);
  }
  if (epi == EPI_DEQUANT_ZP_F32) {
    if (!x_zero || !w_sum) return STAMP_ERR_INVALID_ARG;
    return wide ? launch_gemm_t<256, 6, EPI_DEQUANT_ZP_F32, true>(tw, tx, gp, st)
                : launch_gemm_t<128, 6, EPI_DEQUANT_ZP_F32>(tw, tx, gp, st);
  }
  if (wide) {
    if (epi == EPI_DEQUANT_F32) return launch_gemm_t<256, 6, EPI_DEQUANT_F32, true>(tw, tx, gp, st);
    return launch_gemm_t<256, 6, EPI_RAW_I32, true>(tw, tx, gp, st);
  }
  if (epi == EPI_DEQUANT_F32) return launch_gemm_t<128, 6, EPI_DEQUANT_F32>(tw, tx, gp, st);
  return launch_gemm_t<128, 6, EPI_RAW_I32>(tw, tx, gp, st);
}

template <typename TIn>
static int launch_fwd_pass(int P, const TIn* in, int Lin, long ngroups, int K, float* T, int n, int lvl0, int norm_off,
                           float* aout, unsigned* rowmax, cudaStream_t st) {
  dim3 grid((K / 2 + 127) / 128, (unsigned)(ngroups < 32768 ? ngroups : 32768));
  switch (P) {
    case 0: k_haar_fwd_pass<0, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
    case 1: k_haar_fwd_pass<1, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
    case 2: k_haar_fwd_pass<2, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
    case 3: k_haar_fwd_pass<3, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
    case 4: k_haar_fwd_pass<4, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
    default: k_haar_fwd_pass<5, TIn><<<grid, 128, 0, st>>>(in, Lin, ngroups, K, T, n, lvl0, norm_off, aout, rowmax); break;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Multi-pass Haar analysis of `levels` levels over nseq sequences of Lin input rows.  The input
// rows are X itself (norm_off = 0) or un-normalised sums over 2^norm_off tokens.  Coefficients go
// to T, laid out as blocks of n rows in [a | d_coarse .. d_fine] order where the first level of
// this call has row-mapping level lvl0 + 1; optionally the per-row |T| maxima (pre-zeroed here).
static int run_haar_passes(const void* in, bool in_bf16, int nseq, int Lin, int K, int levels, float* T, int n,
                           int lvl0, int norm_off, unsigned* rowmax, size_t rowmax_rows, float* ping, float* pong,
                           cudaStream_t st) {
  if (rowmax && cudaMemsetAsync(rowmax, 0, rowmax_rows * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
  const PassPlan pl = make_plan(levels);
  const float* cur = nullptr;
  float* bufs[2] = {ping, pong};
  for (int i = 0; i < pl.npass; ++i) {
    const int P = pl.p[i];
    const bool last = (i == pl.npass - 1);
    float* aout = last ? nullptr : bufs[i & 1];
    const long ngroups = (long)nseq * (Lin >> P);
    int rc;
    if (i == 0 && in_bf16)
      rc = launch_fwd_pass<__nv_bfloat16>(P, static_cast<const __nv_bfloat16*>(in), Lin, ngroups, K, T, n, lvl0,
                                          norm_off, aout, rowmax, st);
    else
      rc = launch_fwd_pass<float>(P, i == 0 ? static_cast<const float*>(in) : cur, Lin, ngroups, K, T, n, lvl0,
                                  norm_off, aout, rowmax, st);
    if (rc) return rc;
    cur = aout;
    lvl0 += P;
    Lin >>= P;
  }
  return STAMP_OK;
}

// The dense n x n matrix of a block transform: DCT-II or sequency-ordered Walsh-Hadamard.
static int make_dct_matrix(int transform, int n, float* mat, cudaStream_t st) {
  if (transform == STAMP_T_WHT)
    k_wht_matrix<<<(unsigned)(((long)n * n + 255) / 256), 256, 0, st>>>(n, ilog2(n), mat);
  else
    k_dct_matrix<<<(unsigned)(((long)n * n + 255) / 256), 256, 0, st>>>(n, mat);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// T = L X (Haar, identity or blockwise DCT-II), fp32, logical order; optionally the per-row |T| maxima.
template <int LV, typename TIn, int MODE = H2D_STORE_T>
static int launch_haar2d_fwd(const Problem& pb, const TIn* X, float* T, unsigned* rowmax, cudaStream_t st,
                             const Haar2dQuant& hq = Haar2dQuant{}) {
  const long npatch = pb.M >> (2 * LV);
  dim3 grid((pb.K / 2 + 127) / 128, (unsigned)(npatch < 32768 ? npatch : 32768));
  k_haar2d_fwd<LV, TIn, MODE><<<grid, 128, 0, st>>>(X, pb.n, pb.grid_w, npatch, pb.K, T, rowmax, hq);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

template <typename TIn, int THREADS, bool ZP>
static int launch_haar2d_patch(const Haar2dPatchParams& pp, long npatch, size_t smem, cudaStream_t st) {
  auto kern = k_haar2d_patch_quant<TIn, THREADS, ZP>;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return rc;
  kern<<<(unsigned)npatch, THREADS, smem, st>>>(pp);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Fused route of the three-level 2-D Haar transform: codes and scales in patch order.  One CTA per patch when a
// patch (64 tokens x K channels) fits in shared memory; otherwise row maxima, scales, then codes in three launches.
template <typename TIn>
static int run_quantize_haar2d_patch(const Problem& pb, const TIn* X, unsigned* rowmax, float* x_scale, float* x_inv,
                                     int8_t* a8, float* sx_epi, int* zp_epi, const int8_t* w8, int* w_sum,
                                     cudaStream_t st) {
  const size_t smem = (size_t)64 * pb.K * sizeof(TIn);
  if (smem <= 224 * 1024) {
    Haar2dPatchParams pp{X, pb.n, pb.grid_w, pb.K, pb.k_hi, (float)pb.qmax_hi, (float)pb.qmax_lo, a8, sx_epi, x_scale,
                         zp_epi, nullptr, 0, nullptr, nullptr, 0};
    if (pb.act_zp && w8 && w_sum) {   // the weight row sums of the zero-point term, taken by the same launch
      pp.rs_w8 = w8;
      pp.rs_rows = pb.N;
      pp.rs_out = w_sum;
    }
    if (w8 && (size_t)pb.N * pb.K <= (size_t)24 << 20) {   // small weight matrix: have it in L2 when the GEMM starts
      pp.pf_base = reinterpret_cast<const uint8_t*>(w8);
      pp.pf_bytes = (long)pb.N * pb.K;
    }
    // a thread owns a channel pair: 576 threads when the pairs fill them exactly (1152 channels), else 512
    if (pb.act_zp) {
      if ((pb.K / 2) % 576 == 0) return launch_haar2d_patch<TIn, 576, true>(pp, pb.M >> 6, smem, st);
      return launch_haar2d_patch<TIn, 512, true>(pp, pb.M >> 6, smem, st);
    }
    if ((pb.K / 2) % 576 == 0) return launch_haar2d_patch<TIn, 576, false>(pp, pb.M >> 6, smem, st);
    return launch_haar2d_patch<TIn, 512, false>(pp, pb.M >> 6, smem, st);
  }
  if (pb.act_zp) return STAMP_ERR_UNSUPPORTED;   // the caller takes the general zero-point route
  if (cudaMemsetAsync(rowmax, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
  if (int rc = launch_haar2d_fwd<3, TIn, H2D_MAX>(pb, X, nullptr, rowmax, st)) return rc;
  k_haar2d_row_scales<<<(unsigned)((pb.M + 255) / 256), 256, 0, st>>>(rowmax, pb.M, pb.n, pb.k_hi, (float)pb.qmax_hi,
                                                                      (float)pb.qmax_lo, x_scale, x_inv);
  STAMP_CHECK_LAUNCH();
  Haar2dQuant hq{a8, sx_epi, x_scale, x_inv, (float)pb.qmax_hi, (float)pb.qmax_lo, pb.k_hi};
  return launch_haar2d_fwd<3, TIn, H2D_QUANT>(pb, X, nullptr, rowmax, st, hq);
}
template <int LV, typename TOut>
static int launch_haar2d_inv(const Problem& pb, const float* Yt, const float* bias, TOut* Y, cudaStream_t st) {
  const long npatch = pb.M >> (2 * LV);
  dim3 grid((pb.N / 2 + 127) / 128, (unsigned)(npatch < 32768 ? npatch : 32768));
  k_haar2d_inv<LV, TOut><<<grid, 128, 0, st>>>(Yt, pb.n, pb.grid_w, npatch, pb.N, bias, Y);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

static int run_transform_generic(const Problem& pb, const void* X, int x_dtype, float* T, unsigned* rowmax,
                                 float* ping, float* pong, float* mat, cudaStream_t st, float* skipa = nullptr) {
  if (pb.transform == STAMP_T_HAAR_SKIP1) {
    // first level (pairs from token 1 on, last token carried, token 0 copied), then the dyadic levels on the
    // low-pass band, whose rows sit one below their place in a plain Haar block
    if (!skipa) return STAMP_ERR_INVALID_ARG;
    if (rowmax && cudaMemsetAsync(rowmax, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
    const long npairs = pb.M / 2;
    dim3 grid((pb.K / 2 + 127) / 128, (unsigned)(npairs < 32768 ? npairs : 32768));
    const int one = pb.levels == 1;
    if (x_dtype == STAMP_BF16)
      k_skip1_fwd_level1<__nv_bfloat16><<<grid, 128, 0, st>>>(static_cast<const __nv_bfloat16*>(X), pb.n, npairs, pb.K, T, skipa,
                                                              one, rowmax);
    else
      k_skip1_fwd_level1<float><<<grid, 128, 0, st>>>(static_cast<const float*>(X), pb.n, npairs, pb.K, T, skipa, one, rowmax);
    STAMP_CHECK_LAUNCH();
    if (one) return STAMP_OK;
    return run_haar_passes(skipa, false, pb.nseq, pb.n / 2, pb.K, pb.levels - 1, T + pb.K, pb.n, 1, 0,
                           rowmax ? rowmax + 1 : nullptr, 0, ping, pong, st);
  }
  if (pb.transform == STAMP_T_HAAR2D) {
    if (rowmax && cudaMemsetAsync(rowmax, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
    const bool bf = x_dtype == STAMP_BF16;
    const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(X);
    const float* xf = static_cast<const float*>(X);
    switch (pb.levels) {
      case 1: return bf ? launch_haar2d_fwd<1>(pb, xb, T, rowmax, st) : launch_haar2d_fwd<1>(pb, xf, T, rowmax, st);
      case 2: return bf ? launch_haar2d_fwd<2>(pb, xb, T, rowmax, st) : launch_haar2d_fwd<2>(pb, xf, T, rowmax, st);
      default: return bf ? launch_haar2d_fwd<3>(pb, xb, T, rowmax, st) : launch_haar2d_fwd<3>(pb, xf, T, rowmax, st);
    }
  }
  if (pb.transform == STAMP_T_DCT2 || pb.transform == STAMP_T_WHT) {
    if (rowmax && cudaMemsetAsync(rowmax, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
    if (int rc = make_dct_matrix(pb.transform, pb.n, mat, st)) return rc;
    const dim3 grid((unsigned)(pb.nseq * ((pb.n + 63) / 64)), (unsigned)((pb.K + 63) / 64));
    if (x_dtype == STAMP_BF16)
      k_dct_apply<false, __nv_bfloat16, float><<<grid, 256, 0, st>>>(mat, pb.n, static_cast<const __nv_bfloat16*>(X),
                                                                      pb.K, T, nullptr, rowmax);
    else
      k_dct_apply<false, float, float><<<grid, 256, 0, st>>>(mat, pb.n, static_cast<const float*>(X), pb.K, T, nullptr,
                                                              rowmax);
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  return run_haar_passes(X, x_dtype == STAMP_BF16, pb.nseq, pb.n, pb.K, pb.levels, T, pb.n, 0, 0, rowmax,
                         (size_t)pb.M, ping, pong, st);
}

template <typename TOut>
static int launch_inv_pass(int P, const float* Yt, const float* ain, int n, int jlo, long ngroups, int N,
                           const float* bias, void* out, cudaStream_t st, int norm_off = 0) {
  dim3 grid((N / 2 + 127) / 128, (unsigned)(ngroups < 32768 ? ngroups : 32768));
  switch (P) {
    case 0: launch_pdl(k_haar_inv_pass<0, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
    case 1: launch_pdl(k_haar_inv_pass<1, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
    case 2: launch_pdl(k_haar_inv_pass<2, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
    case 3: launch_pdl(k_haar_inv_pass<3, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
    case 4: launch_pdl(k_haar_inv_pass<4, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
    default: launch_pdl(k_haar_inv_pass<5, TOut>, grid, dim3(128), 0, st, Yt, ain, n, jlo, ngroups, N, bias, out, norm_off); break;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Y = L^T Yt + bias (Haar or identity), coarse passes first.
static int run_inverse_generic(const Problem& pb, const float* Yt, const float* bias, void* Y, int y_dtype,
                               float* ping, float* pong, float* mat, cudaStream_t st, float* skipa = nullptr) {
  if (pb.transform == STAMP_T_HAAR_SKIP1) {
    if (!skipa) return STAMP_ERR_INVALID_ARG;
    const float* a1 = nullptr;
    if (pb.levels > 1) {   // dyadic levels l..2, coarse to fine, down to the low-pass band of level 1
      const PassPlan pl = make_plan(pb.levels - 1);
      int jlo_of[8];
      int acc = 1;
      for (int i = 0; i < pl.npass; ++i) {
        jlo_of[i] = acc;
        acc += pl.p[i];
      }
      const float* ain = nullptr;
      float* bufs[2] = {ping, pong};
      for (int i = pl.npass - 1; i >= 0; --i) {
        const int P = pl.p[i], jlo = jlo_of[i];
        const long ngroups = (long)pb.nseq * (pb.n >> (jlo + P));
        float* aout = i == 0 ? skipa : bufs[(i - 1) & 1];
        if (int rc = launch_inv_pass<float>(P, Yt + pb.N, ain, pb.n, jlo, ngroups, pb.N, nullptr, aout, st)) return rc;
        ain = aout;
      }
      a1 = skipa;
    }
    const long npairs = pb.M / 2;
    dim3 grid((pb.N / 2 + 127) / 128, (unsigned)(npairs < 32768 ? npairs : 32768));
    if (y_dtype == STAMP_BF16)
      k_skip1_inv_level1<__nv_bfloat16><<<grid, 128, 0, st>>>(Yt, a1, pb.n, npairs, pb.N, bias, static_cast<__nv_bfloat16*>(Y));
    else
      k_skip1_inv_level1<float><<<grid, 128, 0, st>>>(Yt, a1, pb.n, npairs, pb.N, bias, static_cast<float*>(Y));
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  if (pb.transform == STAMP_T_HAAR2D) {
    const bool bf = y_dtype == STAMP_BF16;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(Y);
    float* yf = static_cast<float*>(Y);
    switch (pb.levels) {
      case 1: return bf ? launch_haar2d_inv<1>(pb, Yt, bias, yb, st) : launch_haar2d_inv<1>(pb, Yt, bias, yf, st);
      case 2: return bf ? launch_haar2d_inv<2>(pb, Yt, bias, yb, st) : launch_haar2d_inv<2>(pb, Yt, bias, yf, st);
      default: return bf ? launch_haar2d_inv<3>(pb, Yt, bias, yb, st) : launch_haar2d_inv<3>(pb, Yt, bias, yf, st);
    }
  }
  if (pb.transform == STAMP_T_DCT2 || pb.transform == STAMP_T_WHT) {
    if (int rc = make_dct_matrix(pb.transform, pb.n, mat, st)) return rc;
    const dim3 grid((unsigned)(pb.nseq * ((pb.n + 63) / 64)), (unsigned)((pb.N + 63) / 64));
    if (y_dtype == STAMP_BF16)
      k_dct_apply<true, float, __nv_bfloat16><<<grid, 256, 0, st>>>(mat, pb.n, Yt, pb.N, static_cast<__nv_bfloat16*>(Y),
                                                                     bias, nullptr);
    else
      k_dct_apply<true, float, float><<<grid, 256, 0, st>>>(mat, pb.n, Yt, pb.N, static_cast<float*>(Y), bias, nullptr);
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  const PassPlan pl = make_plan(pb.levels);
  // forward pass i covered levels (sum p[0..i-1], sum p[0..i]]; run them in reverse
  int jlo_of[8];
  int acc = 0;
  for (int i = 0; i < pl.npass; ++i) {
    jlo_of[i] = acc;
    acc += pl.p[i];
  }
  const float* ain = nullptr;
  float* bufs[2] = {ping, pong};
  for (int i = pl.npass - 1; i >= 0; --i) {
    const int P = pl.p[i];
    const int jlo = jlo_of[i];
    const long ngroups = (long)pb.nseq * (pb.n >> (jlo + P));
    int rc;
    if (i == 0) {
      rc = (y_dtype == STAMP_BF16)
               ? launch_inv_pass<__nv_bfloat16>(P, Yt, ain, pb.n, jlo, ngroups, pb.N, bias, Y, st)
               : launch_inv_pass<float>(P, Yt, ain, pb.n, jlo, ngroups, pb.N, bias, Y, st);
    } else {
      // partial sums of level jlo have (M >> jlo) rows: the buffer sized for forward pass i-1's output
      float* aout = bufs[(i - 1) & 1];
      rc = launch_inv_pass<float>(P, Yt, ain, pb.n, jlo, ngroups, pb.N, nullptr, aout, st);
      if (rc) return rc;
      ain = aout;
      continue;
    }
    if (rc) return rc;
  }
  return STAMP_OK;
}

// Quantize materialised rows: T / rowmax hold the first n_src rows of every block of pb.n rows.
static int run_quant_rows(const Problem& pb, const float* T, const unsigned* rowmax, int n_src, int8_t* a8,
                          void* q_hi, void* q_lo, float* x_scale, cudaStream_t st) {
  const long rows = (long)pb.nseq * n_src;
  k_quant_rows<<<(unsigned)rows, 256, 0, st>>>(T, rowmax, pb.K, n_src, pb.n, pb.k_hi, pb.qmax_hi, pb.qmax_lo, a8,
                                               static_cast<int8_t*>(q_hi), static_cast<uint8_t*>(q_lo), x_scale);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Zero-point codes from materialised T (all rows of every block).
// (w8 / w_sum given: the same launch also takes the weight row sums, in CTAs of its own.)
static int run_quant_rows_zp(const Problem& pb, const float* T, int8_t* a8, void* q_hi, void* q_lo, float* x_scale,
                             int* x_zero, cudaStream_t st, const int8_t* w8 = nullptr, int* w_sum = nullptr) {
  const int rs_rows = (w8 && w_sum) ? pb.N : 0;
  k_quant_rows_zp<<<(unsigned)(pb.M + (rs_rows + 7) / 8), 256, 0, st>>>(T, pb.M, pb.K, pb.n, pb.k_hi, a8,
                                                                         static_cast<int8_t*>(q_hi),
                                                                         static_cast<uint8_t*>(q_lo), x_scale, x_zero, w8,
                                                                         rs_rows, w_sum);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Per-block scales: quantize materialised rows group by group; the dp4a product that scales every group.
static int run_quant_rows_grouped(const Problem& pb, const float* T, int8_t* a8, void* q_hi, void* q_lo, float* x_scale,
                                  cudaStream_t st) {
  k_quant_rows_grouped<<<(unsigned)pb.M, 256, (size_t)(pb.K / 64) * 4, st>>>(T, pb.K, pb.n, pb.k_hi, pb.qmax_hi, pb.qmax_lo,
                                                                            pb.group, a8, static_cast<int8_t*>(q_hi),
                                                                            static_cast<uint8_t*>(q_lo), x_scale);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}
static int run_gemm_grouped(const Problem& pb, const int8_t* a8, const int8_t* w8, const float* x_scale,
                            const float* w_scale, float* Yt, cudaStream_t st) {
  // tensor cores when a ring stage (128 features) holds whole groups or is part of one (groups of up to 4096
  // features) and a tile's token scales fit the shared-memory table
  if (pb.K % GGT_BK == 0 && pb.group >= 64 && pb.group <= 4096 && (pb.group == 64 || pb.group % 128 == 0) &&
      pb.K / pb.group <= GGT_MAX_GROUPS && pb.M < (1L << 31)) {
    GgtParams gp{};
    gp.n_out = pb.N;
    gp.m_tok = (int)pb.M;
    gp.k = pb.K;
    gp.group = pb.group;
    gp.x_scale = x_scale;
    gp.w_scale = w_scale;
    gp.out = Yt;
    CUtensorMap tw, tx;
    int rc = make_tmap_i8(w8, pb.N, pb.K, GGT_BM, &tw);
    if (rc) return rc;
    if ((rc = make_tmap_i8(a8, pb.M, pb.K, GGT_BN, &tx))) return rc;
    if ((rc = ensure_dyn_smem(reinterpret_cast<const void*>(k_gemm_grouped_tc), GGT_DYN_BYTES))) return rc;
    const long tiles = ((pb.N + GGT_BM - 1) / GGT_BM) * ((pb.M + GGT_BN - 1) / GGT_BN);
    const int grid = (int)std::min<long>(tiles, sm_count());
    k_gemm_grouped_tc<<<grid, GGT_THREADS, GGT_DYN_BYTES, st>>>(tw, tx, gp);
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  dim3 grid((unsigned)((pb.N + GG_TILE - 1) / GG_TILE), (unsigned)((pb.M + GG_TILE - 1) / GG_TILE));
  k_gemm_grouped<<<grid, 256, 0, st>>>(a8, w8, x_scale, w_scale, pb.M, pb.N, pb.K, pb.group, Yt);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

static int run_weight_row_sums(const int8_t* w8, int N, int K, int* w_sum, cudaStream_t st) {
  k_row_sums_i8<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(w8, N, K, w_sum);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// ------------------------------------------------------------------------------------------
// Fused Haar transform + quantizer: cluster kernel, up to five levels per launch.
// ------------------------------------------------------------------------------------------
struct CqChoice {
  int C;     // CTAs per cluster = strips along the feature axis
  int NT;    // threads per CTA (four channels each)
  int pmax;  // Haar levels per launch at most
};
// Fewest strips for which a CTA of at most 512 threads covers its strip.  False when the feature
// axis is too long for a portable cluster of 8 CTAs (more than 16384 channels).
static bool choose_cq(int K, CqChoice* c) {
  for (int C = 1; C <= 8; ++C) {
    const int quads = (K / 4 + C - 1) / C;
    const int nt = (quads + 31) / 32 * 32;
    if (nt <= 512) {
      c->C = C;
      c->NT = nt;
      c->pmax = 4;
      return true;
    }
  }
  return false;
}

static PassPlan make_plan_max(int levels, int pmax) {
  PassPlan pl{};
  int rem = levels;
  if (rem == 0) {
    pl.npass = 1;
    pl.p[0] = 0;
    return pl;
  }
  while (rem > 0) {
    const int p = rem > pmax ? pmax : rem;
    pl.p[pl.npass++] = p;
    rem -= p;
  }
  return pl;
}

template <int P, typename TIn, int OUT, int LODD>
static int launch_cq_t(CqParams cp, const CqChoice& c, cudaStream_t st) {
  auto kern = k_haar_cq<P, TIn, OUT, LODD>;
  constexpr bool STAGED = sizeof(TIn) == 2;
  size_t smem = CQ_TAIL_BYTES;
  cp.nstages = 1;
  if (STAGED) {
    const size_t slab = cq_slab_bytes<P, TIn>(cp.Kc);
    // leave room for as many CTAs per SM as the register file allows (512 threads of 128 registers)
    const size_t budget = (size_t)200 * 1024 * c.NT / 512;
    size_t ns = (budget - CQ_TAIL_BYTES) / slab;
    ns = ns > 4 ? 4 : ns;
    if (ns < 2) return STAMP_ERR_UNSUPPORTED;
    cp.nstages = (int)ns;
    smem += slab * ns;
  }
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return rc;
  cudaLaunchConfig_t lc{};
  lc.blockDim = dim3((unsigned)c.NT);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)c.C;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 2;
  // persistent clusters: as many as can be resident at once (cached per launch shape)
  static std::mutex mu;
  static std::unordered_map<unsigned long long, int> resident;
  const unsigned long long key = ((unsigned long long)(current_device() & 0xFF) << 56) | ((unsigned long long)smem << 24) |
                                 ((unsigned long long)c.NT << 8) | (unsigned)c.C;
  int ncl = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    auto itr = resident.find(key);
    if (itr != resident.end()) {
      ncl = itr->second;
    } else {
      lc.gridDim = dim3((unsigned)(c.C * sm_count()));
      if (cudaOccupancyMaxActiveClusters(&ncl, kern, &lc) != cudaSuccess || ncl <= 0) {
        cudaGetLastError();
        ncl = sm_count() / c.C;
        if (ncl < 1) ncl = 1;
      }
      resident[key] = ncl;
    }
  }
  if ((long)ncl > cp.ngroups) ncl = (int)cp.ngroups;
  lc.gridDim = dim3((unsigned)(ncl * c.C));
  if (cudaLaunchKernelEx(&lc, kern, cp) != cudaSuccess) {
    cudaGetLastError();
    return STAMP_ERR_CUDA;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

template <typename TIn, int OUT, int LODD>
static int launch_cq_p(int P, const CqParams& cp, const CqChoice& c, cudaStream_t st) {
  switch (P) {
    case 0: return launch_cq_t<0, TIn, OUT, LODD>(cp, c, st);
    case 1: return launch_cq_t<1, TIn, OUT, LODD>(cp, c, st);
    case 2: return launch_cq_t<2, TIn, OUT, LODD>(cp, c, st);
    case 3: return launch_cq_t<3, TIn, OUT, LODD>(cp, c, st);
    default: return launch_cq_t<4, TIn, OUT, LODD>(cp, c, st);
  }
}
template <int OUT>
static int launch_cq_o(int P, bool bf16_in, const CqParams& cp, const CqChoice& c, cudaStream_t st) {
  const bool lodd = (cp.lvl0 & 1) != 0;
  if (bf16_in)
    return lodd ? launch_cq_p<__nv_bfloat16, OUT, 1>(P, cp, c, st) : launch_cq_p<__nv_bfloat16, OUT, 0>(P, cp, c, st);
  return lodd ? launch_cq_p<float, OUT, 1>(P, cp, c, st) : launch_cq_p<float, OUT, 0>(P, cp, c, st);
}

// Haar (or identity) transform + quantizer through the cluster kernel: one launch per group of
// levels, each launch quantizing its own detail rows and handing fp32 sums to the next one.
// Exactly one kind of output besides the scales: a8, or (q_hi, q_lo), or T_out.
struct CqTiled {
  int8_t* a8_top;   // must be a8 + M * K
  float* sx_top;
  float* sx_epi;
  const uint8_t* pf_base = nullptr;   // weight codes to pull towards L2 during the first launch (optional)
  long pf_bytes = 0;
};
// start_lvl > 0: the first start_lvl levels have been applied already and X holds the un-normalised fp32 sums
// over 2^start_lvl tokens, [nseq, n >> start_lvl, K], in the workspace's first hand-over buffer.
static int run_quantize_cq(const Problem& pb, const CqChoice& c, const void* X, int x_dtype, int8_t* a8, void* q_hi,
                           void* q_lo, float* x_scale, float* T_out, uint8_t* base, const Workspace& wl,
                           cudaStream_t st, const CqTiled* tiled = nullptr, int start_lvl = 0) {
  const PassPlan pl = make_plan_max(pb.levels - start_lvl, c.pmax);
  float* bufs[3] = {reinterpret_cast<float*>(base + wl.atop), reinterpret_cast<float*>(base + wl.top_ping),
                    reinterpret_cast<float*>(base + wl.top_pong)};
  CqParams cp{};
  cp.K = pb.K;
  cp.Kc = 4 * c.NT;
  cp.n = pb.n;
  cp.k_hi = pb.k_hi;
  cp.qmax_hi = (float)pb.qmax_hi;
  cp.qmax_lo = (float)pb.qmax_lo;
  cp.a8 = a8;
  cp.q_hi = static_cast<int8_t*>(q_hi);
  cp.q_lo = static_cast<uint8_t*>(q_lo);
  cp.x_scale = x_scale;
  cp.T_out = T_out;
  if (tiled) {
    cp.a8_top_row = pb.M;
    cp.sx_top = tiled->sx_top;
    cp.sx_epi = tiled->sx_epi;
  }
  const void* in = X;
  int Lin = pb.n >> start_lvl, lvl0 = start_lvl;
  for (int i = 0; i < pl.npass; ++i) {
    const int P = pl.p[i];
    const bool last = (i == pl.npass - 1);
    // launch i writes into buffer min(i, 1 + (i - 1) % 2): atop, then ping / pong alternately
    // (a continuation reads atop, so its launches alternate between ping and pong from the start)
    float* aout = last ? nullptr : start_lvl ? bufs[1 + (i & 1)] : bufs[i == 0 ? 0 : 1 + ((i - 1) & 1)];
    cp.in = in;
    cp.aout = aout;
    cp.pf_base = (tiled && i == 0) ? tiled->pf_base : nullptr;
    cp.pf_bytes = (tiled && i == 0) ? tiled->pf_bytes : 0;
    cp.Lin = Lin;
    cp.lvl0 = lvl0;
    cp.ngroups = (long)pb.nseq * (Lin >> P);
    const bool bf16_in = (i == 0 && start_lvl == 0 && x_dtype == STAMP_BF16);
    const int rc = tiled ? launch_cq_o<CQ_OUT_TILED>(P, bf16_in, cp, c, st)
                   : a8  ? launch_cq_o<CQ_OUT_A8>(P, bf16_in, cp, c, st)
                      : T_out ? launch_cq_o<CQ_OUT_T>(P, bf16_in, cp, c, st)
                              : launch_cq_o<CQ_OUT_PUBLIC>(P, bf16_in, cp, c, st);
    if (rc) return rc;
    in = aout;
    Lin >>= P;
    lvl0 += P;
  }
  return STAMP_OK;
}

// ------------------------------------------------------------------------------------------
// Haar transform + quantizer for bf16 activations: up to seven levels on the tensor cores with the
// coefficients resident in tensor memory (k_haar_tc), deeper levels by the butterfly kernel on the
// 128-token sums.
// ------------------------------------------------------------------------------------------
#ifndef HTC_FOLD_ROWS
#define HTC_FOLD_ROWS 64
#endif
static bool htc_ok(const Problem& pb, int x_dtype) {
  // the kernel's per-tile index arithmetic is 32-bit: tokens and work items must fit
  return pb.transform == STAMP_T_HAAR && x_dtype == STAMP_BF16 && pb.levels >= 1 && pb.n % 128 == 0 && !pb.act_zp &&
         pb.K % 128 == 0 && pb.K / 128 <= sm_count() && pb.M < (1L << 31) && (pb.M >> 7) * (long)(pb.K / 128) < (1L << 31);
}

template <int OUT>
static int launch_htc(const CUtensorMap& tx, const HtcParams& hp, cudaStream_t st) {
  auto kern = k_haar_tc<OUT>;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), HTC_DYN_BYTES)) return rc;
  const long items = hp.ntiles * hp.nchunks;
  const int grid = items < sm_count() ? (int)items : sm_count();
  if (launch_pdl(kern, dim3((unsigned)grid), dim3(HTC_THREADS), HTC_DYN_BYTES, st, tx, hp) != cudaSuccess) {
    cudaGetLastError();
    return STAMP_ERR_CUDA;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Exactly one kind of output besides the scales, as for run_quantize_cq: a8 (tile order when `tiled`), or
// (q_hi, q_lo), or T_out.
static int run_quantize_haar(const Problem& pb, const CqChoice& c, const void* X, int x_dtype, int8_t* a8, void* q_hi,
                             void* q_lo, float* x_scale, float* T_out, uint8_t* base, const Workspace& wl,
                             cudaStream_t st, const CqTiled* tiled = nullptr) {
  if (!htc_ok(pb, x_dtype)) return run_quantize_cq(pb, c, X, x_dtype, a8, q_hi, q_lo, x_scale, T_out, base, wl, st, tiled);
  const int lv = pb.levels < 7 ? pb.levels : 7;
  HtcParams hp{};
  hp.K = pb.K;
  hp.n = pb.n;
  hp.n_shift = -1;
  for (int sh = 7; sh < 31; ++sh)
    if ((1 << sh) == pb.n) hp.n_shift = sh;
  hp.lv = lv;
  hp.last = (lv == pb.levels) ? 1 : 0;
  hp.k_hi = pb.k_hi;
  hp.qmax_hi = (float)pb.qmax_hi;
  hp.qmax_lo = (float)pb.qmax_lo;
  hp.ntiles = pb.M >> 7;
  hp.nchunks = pb.K / 128;
  hp.rowmax = reinterpret_cast<unsigned*>(base + wl.rowmax);
  hp.cnt = reinterpret_cast<unsigned*>(base + wl.htc_cnt);
  hp.aout = reinterpret_cast<float*>(base + wl.atop);
  hp.a8 = a8;
  hp.q_hi = static_cast<int8_t*>(q_hi);
  hp.q_lo = static_cast<uint8_t*>(q_lo);
  hp.x_scale = x_scale;
  hp.T_out = T_out;
  if (tiled) {
    hp.sx_epi = tiled->sx_epi;
    hp.pf_base = tiled->pf_base;
    hp.pf_bytes = tiled->pf_bytes;
  }
  // row maxima and tile counts start from zero (the two regions are adjacent)
  // The kernel's tail finishes the levels above the seventh itself when the outputs are in logical order and a
  // block has at most 64 rows of 128-token sums (blocks of up to 8192 tokens).  Measured, whole call, tail against
  // continuation launches: 31 against 35 us at 2048 tokens x 4096 channels, 54.6 against 55.5 us at 8192 x 8192;
  // with 256 rows per block (32768 tokens) one CTA per 128-channel strip is too few hands (164 against 154 us).
  const int coarse_rows = pb.n >> 7;
  hp.fold = (!tiled && !hp.last && coarse_rows <= HTC_FOLD_ROWS) ? 1 : 0;
  if (hp.fold && (long)pb.nseq * (pb.K / 64) <= sm_count()) hp.fold = 2;   // 64-channel strips: twice as many CTAs at work
  hp.levels = pb.levels;
  hp.nseq = pb.nseq;
  hp.done = hp.cnt + (pb.M >> 7);
  hp.rowmax2 = hp.done + 4;
  hp.cnt2 = hp.rowmax2 + (pb.M >> 7);
  {
    const size_t bytes = (wl.htc_cnt - wl.rowmax) + ((size_t)(pb.M >> 7) * 2 + 4 + (size_t)pb.nseq) * 4;
    const long n16 = (long)((bytes + 15) / 16);   // both regions are 256-byte aligned and padded in the workspace
    const int grid = (int)std::min<long>((n16 + 255) / 256, 64);
    if (launch_pdl(k_htc_clear, dim3((unsigned)grid), dim3(256), 0, st, reinterpret_cast<uint4*>(base + wl.rowmax), n16) !=
        cudaSuccess) {
      cudaGetLastError();
      return STAMP_ERR_CUDA;
    }
    STAMP_CHECK_LAUNCH();
  }
  CUtensorMap tx;
  int rc = make_tmap_bf16(X, pb.M, pb.K, &tx, 128);
  if (rc) return rc;
  rc = tiled ? launch_htc<HTC_OUT_TILED>(tx, hp, st)
       : a8  ? launch_htc<HTC_OUT_A8>(tx, hp, st)
        : T_out ? launch_htc<HTC_OUT_T>(tx, hp, st)
                : launch_htc<HTC_OUT_PUBLIC>(tx, hp, st);
  if (rc || hp.last || hp.fold) return rc;
  CqTiled rest;
  if (tiled) {
    rest = *tiled;
    rest.pf_base = nullptr;   // the hints went out with the first launch
    rest.pf_bytes = 0;
  }
  return run_quantize_cq(pb, c, hp.aout, STAMP_F32, a8, q_hi, q_lo, x_scale, T_out, base, wl, st, tiled ? &rest : nullptr, lv);
}

// ------------------------------------------------------------------------------------------
// Blockwise 256-point DCT-II on the tensor cores (bf16 activations).
// ------------------------------------------------------------------------------------------
static bool dct_tc_ok(const Problem& pb, int x_dtype) {
  return (pb.transform == STAMP_T_DCT2 || pb.transform == STAMP_T_WHT) && pb.n == DCT_N && x_dtype == STAMP_BF16;
}

// Transform + quantizer: row maxima in a first launch, codes (a8, logical order) and scales in a second.
static int run_quantize_dct_tc(const Problem& pb, const void* X, int8_t* a8, float* x_scale, uint8_t* base,
                               const Workspace& wl, cudaStream_t st) {
  __nv_bfloat16* split = reinterpret_cast<__nv_bfloat16*>(base + wl.dctsplit);
  unsigned* rowmax = reinterpret_cast<unsigned*>(base + wl.rowmax);
  const int wht = pb.transform == STAMP_T_WHT;
  k_dct_split_matrix<<<DCT_N * DCT_N / 256, 256, 0, st>>>(0, wht, split);
  STAMP_CHECK_LAUNCH();
  if (cudaMemsetAsync(rowmax, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
  CUtensorMap ta, tb;
  int rc = make_tmap_bf16(split, 3 * DCT_N, DCT_N, &ta);
  if (rc) return rc;
  if ((rc = make_tmap_bf16(X, pb.M, pb.K, &tb))) return rc;
  DctTcParams dp{};
  dp.nblk = pb.nseq;
  dp.cols = pb.K;
  dp.k_hi = pb.k_hi;
  dp.qmax_hi = (float)pb.qmax_hi;
  dp.qmax_lo = (float)pb.qmax_lo;
  dp.rowmax = rowmax;
  dp.a8 = a8;
  dp.x_scale = x_scale;
  dp.nterms = wht ? 1 : 3;
  if ((rc = launch_dct_tc<DCT_TC_MAX, 2, 1>(ta, tb, tb, dp, st))) return rc;
  return launch_dct_tc<DCT_TC_QUANT, 2, 1>(ta, tb, tb, dp, st);
}

// Y = C^T (hi + lo) + bias from the two bf16 planes the GEMM's epilogue wrote.  N % 64 == 0.
static int run_inverse_dct_tc(const Problem& pb, const __nv_bfloat16* planes, const float* bias, void* Y, int y_dtype,
                              uint8_t* base, const Workspace& wl, cudaStream_t st) {
  __nv_bfloat16* split = reinterpret_cast<__nv_bfloat16*>(base + wl.dctsplit) + 3 * DCT_N * DCT_N;
  const int wht = pb.transform == STAMP_T_WHT;
  k_dct_split_matrix<<<DCT_N * DCT_N / 256, 256, 0, st>>>(1, wht, split);
  STAMP_CHECK_LAUNCH();
  CUtensorMap ta, tb0, tb1;
  int rc = make_tmap_bf16(split, 3 * DCT_N, DCT_N, &ta);
  if (rc) return rc;
  if ((rc = make_tmap_bf16(planes, pb.M, pb.N, &tb0))) return rc;
  if ((rc = make_tmap_bf16(planes + (size_t)pb.M * pb.N, pb.M, pb.N, &tb1))) return rc;
  DctTcParams dp{};
  dp.nblk = pb.nseq;
  dp.cols = pb.N;
  dp.y = Y;
  dp.y_bf16 = (y_dtype == STAMP_BF16);
  dp.bias = bias;
  dp.nterms = wht ? 2 : 3;
  return launch_dct_tc<DCT_TC_INVERSE, 1, 2>(ta, tb0, tb1, dp, st);
}

// Top rows of a short sequence: codes x weights, de-quantization and the inverse of the levels above 8
// in one launch (k_top_gemv).  Returns STAMP_ERR_UNSUPPORTED when the shape is outside its range.
template <int R, bool PACKED>
static int launch_top_gemv(const int8_t* codes, const float* sx, const int8_t* w8, int K, int N, int top_levels,
                           float* a8v, cudaStream_t st) {
  auto kern = k_top_gemv<R, PACKED>;
  const size_t smem = (size_t)R * K;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return rc;
  const int per_cta = (TOPG_THREADS / 32) * TOPG_CH_PER_WARP;
  if (launch_pdl(kern, dim3((unsigned)((N + per_cta - 1) / per_cta)), dim3(TOPG_THREADS), smem, st, codes, sx, w8, K, N,
                 top_levels, a8v) != cudaSuccess) {
    cudaGetLastError();
    return STAMP_ERR_CUDA;
  }
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}
// w4: the same weights as packed 4-bit codes [N, K / 2] when the caller has them (the kernel then streams half the
// bytes), else null.
static int run_top_gemv(const Problem& pb, const int8_t* codes, const float* sx, const int8_t* w8, const uint8_t* w4,
                        float* a8v, cudaStream_t st) {
  const long R = pb.M >> 8;
  if (R > 16 || (size_t)R * pb.K > 160 * 1024 || pb.K % 32 != 0) return STAMP_ERR_UNSUPPORTED;
  const int tl = pb.levels - 8;
  // Measured (ms per layer step, int8 weights / packed weights): 2 rows: 0.0618 / 0.0587 at K = N = 8192, 0.0352 / 0.0349
  // at 2048; 8 rows: 0.0978 / 0.1095 on 4096 x 11008, 0.1383 / 0.1522 at K = N = 8192 -- with more than two rows the
  // expansion of the nibbles costs more than the bytes it saves, so the packed copy is read for up to two rows only.
  if (R > 2) w4 = nullptr;
  const int8_t* w4p = reinterpret_cast<const int8_t*>(w4);
  switch (R) {
    case 2: return w4 ? launch_top_gemv<2, true>(codes, sx, w4p, pb.K, pb.N, tl, a8v, st) : launch_top_gemv<2, false>(codes, sx, w8, pb.K, pb.N, tl, a8v, st);
    case 4: return w4 ? launch_top_gemv<4, true>(codes, sx, w4p, pb.K, pb.N, tl, a8v, st) : launch_top_gemv<4, false>(codes, sx, w8, pb.K, pb.N, tl, a8v, st);
    case 8: return w4 ? launch_top_gemv<8, true>(codes, sx, w4p, pb.K, pb.N, tl, a8v, st) : launch_top_gemv<8, false>(codes, sx, w8, pb.K, pb.N, tl, a8v, st);
    case 16: return w4 ? launch_top_gemv<16, true>(codes, sx, w4p, pb.K, pb.N, tl, a8v, st) : launch_top_gemv<16, false>(codes, sx, w8, pb.K, pb.N, tl, a8v, st);
    default: return STAMP_ERR_UNSUPPORTED;
  }
}

static int run_unpack_codes(const Problem& pb, const void* q_hi, const void* q_lo, int8_t* out, cudaStream_t st) {
  k_unpack_codes<<<(unsigned)pb.M, 256, 0, st>>>(static_cast<const int8_t*>(q_hi), static_cast<const uint8_t*>(q_lo),
                                                  pb.K, pb.n, pb.k_hi, out);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

// Resolve the weight operand to int8 [N, K]: either the caller's prepared copy or an expansion
// of the packed codes into the workspace.
static int weights_as_int8(const Problem& pb, const void* w, int w_format, int8_t* w8_ws, const int8_t** out,
                           cudaStream_t st) {
  if (w_format == STAMP_W_INT8 || w_format == STAMP_W_INT8_AND_PACKED4) {
    *out = static_cast<const int8_t*>(w);
    return STAMP_OK;
  }
  if (w_format != STAMP_W_PACKED4) return STAMP_ERR_INVALID_ARG;
  k_unpack_rows4<<<(unsigned)pb.N, 256, 0, st>>>(static_cast<const uint8_t*>(w), pb.K, w8_ws);
  STAMP_CHECK_LAUNCH();
  *out = w8_ws;
  return STAMP_OK;
}

// The packed copy of the weights when the caller's operand has one (kernels that only stream the weights read it).
static const uint8_t* weights_packed(const Problem& pb, const void* w, int w_format) {
  if (w_format == STAMP_W_PACKED4) return static_cast<const uint8_t*>(w);
  if (w_format == STAMP_W_INT8_AND_PACKED4) return static_cast<const uint8_t*>(w) + (size_t)pb.N * pb.K;
  return nullptr;
}

// ------------------------------------------------------------------------------------------
// Built-in scratch of stamp_inverse_noalloc(): one array per GPU that loads the library, held
// until the process exits.  In host code the array's name is only a handle for the runtime, not
// a device address, so the address is looked up once per device with that device current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[STAMP_NOALLOC_SCRATCH_BYTES];

static int noalloc_scratch_base(uint8_t** out) {
  static std::mutex mu;
  static uint8_t* base_of[MAX_DEVICES] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return STAMP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!base_of[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return STAMP_ERR_CUDA;
    }
    base_of[dev] = static_cast<uint8_t*>(p);
  }
  *out = base_of[dev];
  return STAMP_OK;
}

// ------------------------------------------------------------------------------------------
// Routes of the one-call layer and their transform+quantize stages (shared with the debug export of
// the fused operand, so that the export runs the very kernels the layer runs).
// ------------------------------------------------------------------------------------------
enum FusedRoute { ROUTE_PATCH2D = 0, ROUTE_ZP_GENERAL = 1, ROUTE_TILED = 2, ROUTE_DCT_TC = 3, ROUTE_GENERAL = 4 };

static FusedRoute fused_route(const Problem& pb, int x_dtype, CqChoice* cc, bool* have_cq) {
  const bool patch_fits = (size_t)64 * pb.K * (x_dtype == STAMP_BF16 ? 2 : 4) <= 224 * 1024;
  *have_cq = (pb.transform == STAMP_T_HAAR || pb.transform == STAMP_T_IDENTITY) && choose_cq(pb.K, cc);
  if (pb.group) {   // per-block scales: separate transform, group quantizer, CUDA-core product, inverse
    *have_cq = false;
    return ROUTE_GENERAL;
  }
  if (pb.transform == STAMP_T_HAAR2D && pb.levels == 3 && pb.M % 256 == 0 && (!pb.act_zp || patch_fits)) return ROUTE_PATCH2D;
  if (pb.act_zp) return ROUTE_ZP_GENERAL;
  if (*have_cq && pb.transform == STAMP_T_HAAR && pb.levels >= 5 && pb.n % 256 == 0) return ROUTE_TILED;
  if (dct_tc_ok(pb, x_dtype)) return ROUTE_DCT_TC;
  return ROUTE_GENERAL;
}

// Where the patch-order route keeps its per-row tables (the fp32 T of the general route is not materialised
// there, so its space is reused).
struct PatchTables {
  float* x_inv;
  float* sx_epi;
  int* zp_epi;
};
static PatchTables patch_tables(const Problem& pb, uint8_t* base, const Workspace& wl) {
  float* T = reinterpret_cast<float*>(base + wl.T);
  return PatchTables{T, T + pb.M, reinterpret_cast<int*>(T + 2 * pb.M)};
}

// Patch-order route: one CTA per 8 x 8 patch finds the row maxima (or minima and maxima, for zero-point
// codes) and writes codes in patch order.  w8 / w_sum: weight codes and the buffer of their row sums for the
// zero-point term (w8 may be null: no sums are taken).
static int fused_quantize_patch2d(const Problem& pb, const void* X, int x_dtype, uint8_t* base, const Workspace& wl,
                                  const int8_t* w8, int* w_sum, cudaStream_t st) {
  const PatchTables pt = patch_tables(pb, base, wl);
  unsigned* rowmax = reinterpret_cast<unsigned*>(base + wl.rowmax);
  float* x_scale = reinterpret_cast<float*>(base + wl.xscale);
  int8_t* a8 = reinterpret_cast<int8_t*>(base + wl.a8);
  if (x_dtype == STAMP_BF16)
    return run_quantize_haar2d_patch(pb, static_cast<const __nv_bfloat16*>(X), rowmax, x_scale, pt.x_inv, a8, pt.sx_epi,
                                     pt.zp_epi, w8, w_sum, st);
  return run_quantize_haar2d_patch(pb, static_cast<const float*>(X), rowmax, x_scale, pt.x_inv, a8, pt.sx_epi, pt.zp_epi,
                                   w8, w_sum, st);
}

// Tile-order route: the transform+quantize chain writes the token operand in tile order (rows of levels above
// 8 into the table behind it).  w8: weight codes to pull towards L2 during the first launch, or null.
static int fused_quantize_tiled(const Problem& pb, const CqChoice& cc, const void* X, int x_dtype, uint8_t* base,
                                const Workspace& wl, const int8_t* w8, CqTiled* tl_out, cudaStream_t st) {
  int8_t* a8 = reinterpret_cast<int8_t*>(base + wl.a8);
  float* x_scale = reinterpret_cast<float*>(base + wl.xscale);
  CqTiled tl{reinterpret_cast<int8_t*>(base + wl.a8top), reinterpret_cast<float*>(base + wl.sxtop), x_scale};
  // The first launch of the transform chain also pulls a small weight matrix towards L2: the chain's later
  // launches are small and leave HBM idle, and the GEMM (and the skinny top-row product before it) then
  // start on weights that are already there.  Measured: 8 to 20 % per step up to 16 MB of codes; nothing
  // to gain, or a loss, at 45 MB and above, whether the whole matrix or its first 16 MB are asked for.
  if (w8 && (size_t)pb.N * pb.K <= (size_t)24 << 20) {
    tl.pf_base = reinterpret_cast<const uint8_t*>(w8);
    tl.pf_bytes = (long)pb.N * pb.K;
  }
  *tl_out = tl;
  return run_quantize_haar(pb, cc, X, x_dtype, a8, nullptr, nullptr, x_scale, nullptr, base, wl, st, &tl);
}

}  // namespace stamp

// ============================================================================================
// C ABI
// ============================================================================================
using namespace stamp;

extern "C" {

int stamp_workspace_bytes(const stamp_config* cfg, int B, int L, int K, int N, size_t* out_bytes) {
  if (!out_bytes) return STAMP_ERR_INVALID_ARG;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  *out_bytes = layout(pb).total;
  return STAMP_OK;
}

int stamp_quantize_weights(const stamp_config* cfg, const void* W, int w_dtype, int N, int K, void* wq,
                           float* w_scale, void* stream) {
  t_launches = 0;
  if (!cfg || !W || !wq || !w_scale || N <= 0 || K <= 0 || !dtype_ok(w_dtype)) return STAMP_ERR_INVALID_ARG;
  if (cfg->bits_w != 4 || K % 128 != 0) return STAMP_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cfg->group > 0) {
    if (cfg->w_gran != STAMP_G_GROUP || cfg->group % 64 != 0 || !is_pow2(cfg->group) || K % cfg->group != 0)
      return STAMP_ERR_UNSUPPORTED;
    const size_t sm = (size_t)(K / 64) * 4;
    if (w_dtype == STAMP_BF16)
      k_quant_weights_grouped<__nv_bfloat16><<<N, 256, sm, st>>>(static_cast<const __nv_bfloat16*>(W), K, 7, cfg->group,
                                                                 static_cast<uint8_t*>(wq), w_scale);
    else
      k_quant_weights_grouped<float><<<N, 256, sm, st>>>(static_cast<const float*>(W), K, 7, cfg->group,
                                                         static_cast<uint8_t*>(wq), w_scale);
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  if (cfg->w_gran != STAMP_G_PER_CHANNEL) return STAMP_ERR_UNSUPPORTED;
  if (w_dtype == STAMP_BF16)
    k_quant_weights<__nv_bfloat16><<<N, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W), K, 7,
                                                      static_cast<uint8_t*>(wq), w_scale);
  else
    k_quant_weights<float><<<N, 256, 0, st>>>(static_cast<const float*>(W), K, 7, static_cast<uint8_t*>(wq), w_scale);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

int stamp_prepare_weights(const stamp_config* cfg, const void* wq_packed, int N, int K, void* w_int8, void* stream) {
  t_launches = 0;
  if (!cfg || !wq_packed || !w_int8 || N <= 0 || K <= 0) return STAMP_ERR_INVALID_ARG;
  if (cfg->bits_w != 4 || K % 128 != 0) return STAMP_ERR_UNSUPPORTED;
  k_unpack_rows4<<<N, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint8_t*>(wq_packed), K,
                                                                    static_cast<int8_t*>(w_int8));
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

int stamp_prepare_weights_both(const stamp_config* cfg, const void* wq_packed, int N, int K, void* w_both, void* stream) {
  int rc = stamp_prepare_weights(cfg, wq_packed, N, K, w_both, stream);
  if (rc) return rc;
  if (cudaMemcpyAsync(static_cast<uint8_t*>(w_both) + (size_t)N * K, wq_packed, (size_t)N * (K / 2), cudaMemcpyDeviceToDevice,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return STAMP_ERR_CUDA;
  return STAMP_OK;
}

int stamp_quantize(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, void* q_hi, void* q_lo,
                   float* x_scale, void* ws, size_t ws_bytes, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, 0, false, &pb);
  if (rc) return rc;
  if (!X || !x_scale || !dtype_ok(x_dtype)) return STAMP_ERR_INVALID_ARG;
  if ((pb.n_hi_rows() > 0 && !q_hi) || (pb.n_lo_rows() > 0 && !q_lo)) return STAMP_ERR_INVALID_ARG;
  const Workspace w = layout(pb);
  if ((rc = check_ws(w, ws, ws_bytes))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* T = reinterpret_cast<float*>(base + w.T);
  unsigned* rowmax = reinterpret_cast<unsigned*>(base + w.rowmax);
  if (pb.act_zp) {
    rc = run_transform_generic(pb, X, x_dtype, T, rowmax, reinterpret_cast<float*>(base + w.ping),
                               reinterpret_cast<float*>(base + w.pong), reinterpret_cast<float*>(base + w.dctmat), st, reinterpret_cast<float*>(base + w.skipa));
    if (rc) return rc;
    return run_quant_rows_zp(pb, T, nullptr, q_hi, q_lo, x_scale, reinterpret_cast<int*>(x_scale + pb.M), st);
  }
  if (pb.group) {
    rc = run_transform_generic(pb, X, x_dtype, T, nullptr, reinterpret_cast<float*>(base + w.ping),
                               reinterpret_cast<float*>(base + w.pong), reinterpret_cast<float*>(base + w.dctmat), st,
                               reinterpret_cast<float*>(base + w.skipa));
    if (rc) return rc;
    return run_quant_rows_grouped(pb, T, nullptr, q_hi, q_lo, x_scale, st);
  }
  CqChoice cc;
  if ((pb.transform == STAMP_T_HAAR || pb.transform == STAMP_T_IDENTITY) && choose_cq(pb.K, &cc))
    return run_quantize_haar(pb, cc, X, x_dtype, nullptr, q_hi, q_lo, x_scale, nullptr, base, w, st);
  if (dct_tc_ok(pb, x_dtype)) {
    int8_t* a8 = reinterpret_cast<int8_t*>(base + w.a8);
    if ((rc = run_quantize_dct_tc(pb, X, a8, x_scale, base, w, st))) return rc;
    k_pack_codes<<<(unsigned)pb.M, 256, 0, st>>>(a8, pb.K, pb.n, pb.k_hi, static_cast<int8_t*>(q_hi),
                                                  static_cast<uint8_t*>(q_lo));
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  rc = run_transform_generic(pb, X, x_dtype, T, rowmax, reinterpret_cast<float*>(base + w.ping),
                             reinterpret_cast<float*>(base + w.pong), reinterpret_cast<float*>(base + w.dctmat), st, reinterpret_cast<float*>(base + w.skipa));
  if (rc) return rc;
  return run_quant_rows(pb, T, rowmax, pb.n, nullptr, q_hi, q_lo, x_scale, st);
}

int stamp_linear(const stamp_config* cfg, const void* q_hi, const void* q_lo, const float* x_scale, const void* w,
                 int w_format, const float* w_scale, int B, int L, int K, int N, float* Yt, void* ws, size_t ws_bytes,
                 void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  if (!x_scale || !w || !w_scale || !Yt) return STAMP_ERR_INVALID_ARG;
  if ((pb.n_hi_rows() > 0 && !q_hi) || (pb.n_lo_rows() > 0 && !q_lo)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  int8_t* a8 = reinterpret_cast<int8_t*>(base + wl.a8);
  if ((rc = run_unpack_codes(pb, q_hi, q_lo, a8, st))) return rc;
  const int8_t* w8 = nullptr;
  if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8, st))) return rc;
  if (pb.group) return run_gemm_grouped(pb, a8, w8, x_scale, w_scale, Yt, st);
  if (pb.act_zp) {
    int* w_sum = reinterpret_cast<int*>(base + wl.wsum);
    if ((rc = run_weight_row_sums(w8, N, K, w_sum, st))) return rc;
    return launch_gemm(a8, w8, pb.M, N, K, x_scale, w_scale, Yt, EPI_DEQUANT_ZP_F32, st, nullptr, nullptr, 0,
                       reinterpret_cast<const int*>(x_scale + pb.M), w_sum);
  }
  return launch_gemm(a8, w8, pb.M, N, K, x_scale, w_scale, Yt, EPI_DEQUANT_F32, st);
}

int stamp_dequantize(const stamp_config* cfg, const void* q_hi, const void* q_lo, const float* x_scale, int B, int L,
                     int K, float* T, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, 0, false, &pb);
  if (rc) return rc;
  if (!x_scale || !T) return STAMP_ERR_INVALID_ARG;
  if ((pb.n_hi_rows() > 0 && !q_hi) || (pb.n_lo_rows() > 0 && !q_lo)) return STAMP_ERR_INVALID_ARG;
  const int* zero = pb.act_zp ? reinterpret_cast<const int*>(x_scale + pb.M) : nullptr;
  k_dequant_rows<<<(unsigned)pb.M, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const int8_t*>(q_hi), static_cast<const uint8_t*>(q_lo), x_scale, zero, K, pb.n, pb.k_hi, pb.group, T);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

static int inverse_stand_in_k(const stamp_config* cfg) { return (cfg && cfg->group > 128) ? cfg->group : 128; }

int stamp_inverse(const stamp_config* cfg, const float* Yt, const float* bias, int B, int L, int N, void* Y,
                  int y_dtype, void* ws, size_t ws_bytes, void* stream) {
  t_launches = 0;
  Problem pb;
  // the inverse does not touch K: validate with a stand-in that satisfies the K rules (a multiple of the scale group too)
  int rc = resolve(cfg, B, L, inverse_stand_in_k(cfg), N, true, &pb);
  if (rc) return rc;
  if (!Yt || !Y || !dtype_ok(y_dtype)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  uint8_t* base = static_cast<uint8_t*>(ws);
  return run_inverse_generic(pb, Yt, bias, Y, y_dtype, reinterpret_cast<float*>(base + wl.ping),
                             reinterpret_cast<float*>(base + wl.pong), reinterpret_cast<float*>(base + wl.dctmat),
                             static_cast<cudaStream_t>(stream), reinterpret_cast<float*>(base + wl.skipa));
}

int stamp_inverse_noalloc(const stamp_config* cfg, const float* Yt, const float* bias, int B, int L, int N, void* Y,
                          int y_dtype, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, inverse_stand_in_k(cfg), N, true, &pb);
  if (rc) return rc;
  if (!Yt || !Y || !dtype_ok(y_dtype)) return STAMP_ERR_INVALID_ARG;
  if (pb.transform == STAMP_T_HAAR_SKIP1) return STAMP_ERR_UNSUPPORTED;   // (its low-pass band would need half of Yt again)
  // partial sums between the coarse-to-fine passes: the only scratch the inverse needs
  const PassPlan pl = make_plan(pb.levels);
  const size_t ping_bytes = pl.npass > 1 ? align256(((size_t)pb.M >> pl.p[0]) * pb.N * 4) : 0;
  const size_t pong_bytes = pl.npass > 2 ? align256(((size_t)pb.M >> (pl.p[0] + pl.p[1])) * pb.N * 4) : 0;
  const size_t mat_bytes =
      (pb.transform == STAMP_T_DCT2 || pb.transform == STAMP_T_WHT) ? align256((size_t)pb.n * pb.n * 4) : 0;
  if (ping_bytes + pong_bytes + mat_bytes > (size_t)STAMP_NOALLOC_SCRATCH_BYTES) return STAMP_ERR_TOO_LARGE;
  uint8_t* base = nullptr;
  if ((rc = noalloc_scratch_base(&base))) return rc;
  return run_inverse_generic(pb, Yt, bias, Y, y_dtype, reinterpret_cast<float*>(base),
                             reinterpret_cast<float*>(base + ping_bytes),
                             reinterpret_cast<float*>(base + ping_bytes + pong_bytes), static_cast<cudaStream_t>(stream));
}

int stamp_linear_fused(const stamp_config* cfg, const void* X, int x_dtype, const void* w, int w_format,
                       const float* w_scale, const float* bias, int B, int L, int K, int N, void* Y, int y_dtype,
                       void* ws, size_t ws_bytes, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  if (!X || !w || !w_scale || !Y || !dtype_ok(x_dtype) || !dtype_ok(y_dtype)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* T = reinterpret_cast<float*>(base + wl.T);
  unsigned* rowmax = reinterpret_cast<unsigned*>(base + wl.rowmax);
  float* ping = reinterpret_cast<float*>(base + wl.ping);
  float* pong = reinterpret_cast<float*>(base + wl.pong);
  int8_t* a8 = reinterpret_cast<int8_t*>(base + wl.a8);
  float* x_scale = reinterpret_cast<float*>(base + wl.xscale);
  float* yt = reinterpret_cast<float*>(base + wl.yt);
  CqChoice cc;
  bool have_cq = false;
  const FusedRoute route = fused_route(pb, x_dtype, &cc, &have_cq);
  if (route == ROUTE_PATCH2D) {
    // Fused route of the paper's LVM transform: one CTA per 8 x 8 patch finds the row maxima (or minima and maxima,
    // for zero-point codes) and writes codes in patch order; the GEMM's epilogue inverts the four patches of its
    // 256-token tile.
    const PatchTables pt = patch_tables(pb, base, wl);
    const int8_t* w8p = nullptr;
    if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8p, st))) return rc;
    // (zero-point codes: the patch kernel also takes the weight row sums of the correction term)
    int* w_sum = pb.act_zp ? reinterpret_cast<int*>(base + wl.wsum) : nullptr;
    if ((rc = fused_quantize_patch2d(pb, X, x_dtype, base, wl, w8p, w_sum, st))) return rc;
    return launch_gemm(a8, w8p, pb.M, N, K, pt.sx_epi, w_scale, Y, y_dtype == STAMP_BF16 ? EPI_HAAR2D_BF16 : EPI_HAAR2D_F32,
                       st, bias, nullptr, 0, pb.act_zp ? pt.zp_epi : nullptr, w_sum, pb.grid_w, pb.n);
  }
  if (route == ROUTE_ZP_GENERAL) {
    // zero-point codes: transform, min-max quantizer, GEMM with the zero-point term in its epilogue, inverse
    int* x_zero = reinterpret_cast<int*>(base + wl.xzero);
    int* w_sum = reinterpret_cast<int*>(base + wl.wsum);
    if ((rc = run_transform_generic(pb, X, x_dtype, T, rowmax, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st, reinterpret_cast<float*>(base + wl.skipa))))
      return rc;
    const int8_t* w8z = nullptr;
    if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8z, st))) return rc;
    if ((rc = run_quant_rows_zp(pb, T, a8, nullptr, nullptr, x_scale, x_zero, st, w8z, w_sum))) return rc;
    if ((rc = launch_gemm(a8, w8z, pb.M, N, K, x_scale, w_scale, yt, EPI_DEQUANT_ZP_F32, st, nullptr, nullptr, 0, x_zero,
                          w_sum)))
      return rc;
    return run_inverse_generic(pb, yt, bias, Y, y_dtype, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st, reinterpret_cast<float*>(base + wl.skipa));
  }
  if (route == ROUTE_TILED) {
    // Fused route: the transform+quantize kernel writes the token operand in tile order, the GEMM's
    // epilogue de-quantizes and inverts the (up to) 8 levels that close inside its 256-token tile.
    // Levels above 8 live in M / 256 extra rows: a small GEMM and the general inverse turn them into
    // the level-8 approximation of every tile first.
    const int8_t* w8f = nullptr;
    if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8f, st))) return rc;
    CqTiled tl{};
    if ((rc = fused_quantize_tiled(pb, cc, X, x_dtype, base, wl, w8f, &tl, st))) return rc;
    const float* a8v = nullptr;
    if (pb.levels > 8) {
      float* yttop = reinterpret_cast<float*>(base + wl.yttop);
      float* a8v_w = reinterpret_cast<float*>(base + wl.a8v);
      rc = run_top_gemv(pb, tl.a8_top, tl.sx_top, w8f, weights_packed(pb, w, w_format), a8v_w, st);
      if (rc == STAMP_OK) {
        a8v = a8v_w;
      } else if (rc != STAMP_ERR_UNSUPPORTED) {
        return rc;
      } else {
      // (no weight scales here: they are applied once, after the synthesis, by the main GEMM's epilogue)
      if ((rc = launch_gemm(tl.a8_top, w8f, pb.M >> 8, N, K, tl.sx_top, nullptr, yttop, EPI_DEQUANT_F32, st))) return rc;
      Problem pt = pb;
      pt.n = pb.n >> 8;
      pt.L = pb.L >> 8;
      pt.M = pb.M >> 8;
      pt.levels = pb.levels - 8;
      if ((rc = run_inverse_generic(pt, yttop, nullptr, a8v_w, STAMP_F32, ping, pong,
                                    reinterpret_cast<float*>(base + wl.dctmat), st)))
        return rc;
      a8v = a8v_w;
      }
    }
    return launch_gemm(a8, w8f, pb.M, N, K, x_scale, w_scale, Y, y_dtype == STAMP_BF16 ? EPI_HAAR_BF16 : EPI_HAAR_F32, st,
                       bias, a8v, pb.levels < 8 ? pb.levels : 8);
  }
  if (route == ROUTE_DCT_TC) {
    if ((rc = run_quantize_dct_tc(pb, X, a8, x_scale, base, wl, st))) return rc;
    const int8_t* w8d = nullptr;
    if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8d, st))) return rc;
    if (N % 64 == 0) {   // the GEMM writes its output as two bf16 planes, the operand of the tensor-core inverse
      if ((rc = launch_gemm(a8, w8d, pb.M, N, K, x_scale, w_scale, yt, EPI_DEQUANT_BF16X2, st))) return rc;
      return run_inverse_dct_tc(pb, reinterpret_cast<const __nv_bfloat16*>(yt), bias, Y, y_dtype, base, wl, st);
    }
    if ((rc = launch_gemm(a8, w8d, pb.M, N, K, x_scale, w_scale, yt, EPI_DEQUANT_F32, st))) return rc;
    return run_inverse_generic(pb, yt, bias, Y, y_dtype, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st, reinterpret_cast<float*>(base + wl.skipa));
  }
  if (pb.group) {
    if ((rc = run_transform_generic(pb, X, x_dtype, T, nullptr, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st,
                                    reinterpret_cast<float*>(base + wl.skipa))))
      return rc;
    if ((rc = run_quant_rows_grouped(pb, T, a8, nullptr, nullptr, x_scale, st))) return rc;
    const int8_t* w8g = nullptr;
    if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8g, st))) return rc;
    if ((rc = run_gemm_grouped(pb, a8, w8g, x_scale, w_scale, yt, st))) return rc;
    return run_inverse_generic(pb, yt, bias, Y, y_dtype, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st,
                               reinterpret_cast<float*>(base + wl.skipa));
  }
  if (have_cq) {
    if ((rc = run_quantize_haar(pb, cc, X, x_dtype, a8, nullptr, nullptr, x_scale, nullptr, base, wl, st))) return rc;
  } else {
    if ((rc = run_transform_generic(pb, X, x_dtype, T, rowmax, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st, reinterpret_cast<float*>(base + wl.skipa))))
      return rc;
    if ((rc = run_quant_rows(pb, T, rowmax, pb.n, a8, nullptr, nullptr, x_scale, st))) return rc;
  }
  const int8_t* w8 = nullptr;
  if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8, st))) return rc;
  if ((rc = launch_gemm(a8, w8, pb.M, N, K, x_scale, w_scale, yt, EPI_DEQUANT_F32, st))) return rc;
  return run_inverse_generic(pb, yt, bias, Y, y_dtype, ping, pong, reinterpret_cast<float*>(base + wl.dctmat), st, reinterpret_cast<float*>(base + wl.skipa));
}

static size_t dtype_size(int d) { return d == STAMP_BF16 ? 2 : 4; }

int stamp_workspace_bytes_host(const stamp_config* cfg, int B, int L, int K, int N, int x_dtype, int y_dtype,
                               size_t* out_bytes) {
  if (!out_bytes || !dtype_ok(x_dtype) || !dtype_ok(y_dtype)) return STAMP_ERR_INVALID_ARG;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  *out_bytes = layout(pb).total + align256((size_t)pb.M * K * dtype_size(x_dtype)) +
               align256((size_t)pb.M * N * dtype_size(y_dtype));
  return STAMP_OK;
}

int stamp_linear_fused_host(const stamp_config* cfg, const void* X_host, int x_dtype, const void* w, int w_format,
                            const float* w_scale, const float* bias, int B, int L, int K, int N, void* Y_host,
                            int y_dtype, void* ws, size_t ws_bytes, void* stream) {
  size_t need = 0;
  int rc = stamp_workspace_bytes_host(cfg, B, L, K, N, x_dtype, y_dtype, &need);
  if (rc) return rc;
  if (!X_host || !Y_host) return STAMP_ERR_INVALID_ARG;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < need) return STAMP_ERR_WORKSPACE;
  Problem pb;
  resolve(cfg, B, L, K, N, true, &pb);
  const size_t dev_ws = layout(pb).total;
  const size_t xb = (size_t)pb.M * K * dtype_size(x_dtype), yb = (size_t)pb.M * N * dtype_size(y_dtype);
  uint8_t* base = static_cast<uint8_t*>(ws);
  void* Xd = base + dev_ws;
  void* Yd = base + dev_ws + align256(xb);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(Xd, X_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return STAMP_ERR_CUDA;
  rc = stamp_linear_fused(cfg, Xd, x_dtype, w, w_format, w_scale, bias, B, L, K, N, Yd, y_dtype, ws, dev_ws, stream);
  if (rc) return rc;
  if (cudaMemcpyAsync(Y_host, Yd, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return STAMP_ERR_CUDA;
  return STAMP_OK;
}

int stamp_debug_transform(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, float* T, void* ws,
                          size_t ws_bytes, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, 0, false, &pb);
  if (rc) return rc;
  if (!X || !T || !dtype_ok(x_dtype)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  uint8_t* base = static_cast<uint8_t*>(ws);
  CqChoice cc;
  if ((pb.transform == STAMP_T_HAAR || pb.transform == STAMP_T_IDENTITY) && choose_cq(pb.K, &cc))  // the product path's kernel with the fp32 export on
    return run_quantize_haar(pb, cc, X, x_dtype, nullptr, nullptr, nullptr, reinterpret_cast<float*>(base + wl.xscale), T,
                             base, wl, static_cast<cudaStream_t>(stream));
  return run_transform_generic(pb, X, x_dtype, T, nullptr, reinterpret_cast<float*>(base + wl.ping),
                               reinterpret_cast<float*>(base + wl.pong), reinterpret_cast<float*>(base + wl.dctmat),
                               static_cast<cudaStream_t>(stream), reinterpret_cast<float*>(base + wl.skipa));
}

int stamp_debug_unpack_codes(const stamp_config* cfg, const void* q_hi, const void* q_lo, int B, int L, int K,
                             int8_t* codes, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, 0, false, &pb);
  if (rc) return rc;
  if (!codes) return STAMP_ERR_INVALID_ARG;
  if ((pb.n_hi_rows() > 0 && !q_hi) || (pb.n_lo_rows() > 0 && !q_lo)) return STAMP_ERR_INVALID_ARG;
  return run_unpack_codes(pb, q_hi, q_lo, codes, static_cast<cudaStream_t>(stream));
}

int stamp_debug_gemm_i32(const stamp_config* cfg, const void* q_hi, const void* q_lo, const void* w, int w_format,
                         int B, int L, int K, int N, int32_t* acc, void* ws, size_t ws_bytes, void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  if (!w || !acc) return STAMP_ERR_INVALID_ARG;
  if ((pb.n_hi_rows() > 0 && !q_hi) || (pb.n_lo_rows() > 0 && !q_lo)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  int8_t* a8 = reinterpret_cast<int8_t*>(base + wl.a8);
  if ((rc = run_unpack_codes(pb, q_hi, q_lo, a8, st))) return rc;
  const int8_t* w8 = nullptr;
  if ((rc = weights_as_int8(pb, w, w_format, reinterpret_cast<int8_t*>(base + wl.w8), &w8, st))) return rc;
  return launch_gemm(a8, w8, pb.M, N, K, nullptr, nullptr, acc, EPI_RAW_I32, st);
}

int stamp_debug_fused_operand(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, int N,
                              int8_t* codes, float* factor, int32_t* level, int32_t* zero, void* ws, size_t ws_bytes,
                              void* stream) {
  t_launches = 0;
  Problem pb;
  int rc = resolve(cfg, B, L, K, N, true, &pb);
  if (rc) return rc;
  if (!X || !codes || !factor || !level || !dtype_ok(x_dtype)) return STAMP_ERR_INVALID_ARG;
  const Workspace wl = layout(pb);
  if ((rc = check_ws(wl, ws, ws_bytes))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  const int8_t* a8 = reinterpret_cast<const int8_t*>(base + wl.a8);
  CqChoice cc;
  bool have_cq = false;
  const FusedRoute route = fused_route(pb, x_dtype, &cc, &have_cq);
  if (route == ROUTE_TILED) {
    CqTiled tl{};
    if ((rc = fused_quantize_tiled(pb, cc, X, x_dtype, base, wl, nullptr, &tl, st))) return rc;
    k_debug_gather_tiled<<<(unsigned)pb.M, 256, 0, st>>>(a8, tl.sx_epi, tl.sx_top, pb.M, pb.n, pb.levels, K, codes, factor,
                                                         level);
    STAMP_CHECK_LAUNCH();
    if (zero && cudaMemsetAsync(zero, 0, (size_t)pb.M * 4, st) != cudaSuccess) return STAMP_ERR_CUDA;
    return STAMP_OK;
  }
  if (route == ROUTE_PATCH2D) {
    if (pb.act_zp && !zero) return STAMP_ERR_INVALID_ARG;
    if ((rc = fused_quantize_patch2d(pb, X, x_dtype, base, wl, nullptr, nullptr, st))) return rc;
    const PatchTables pt = patch_tables(pb, base, wl);
    k_debug_gather_patch<<<(unsigned)pb.M, 256, 0, st>>>(a8, pt.sx_epi, pb.act_zp ? pt.zp_epi : nullptr, pb.M, pb.n,
                                                         pb.grid_w, K, codes, factor, level, zero);
    STAMP_CHECK_LAUNCH();
    return STAMP_OK;
  }
  return STAMP_ERR_UNSUPPORTED;   // the other routes keep their operand in logical order: stamp_quantize shows it
}

int stamp_last_device_status(void* stream, int* status) {
  if (!status) return STAMP_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return STAMP_ERR_CUDA;
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) return STAMP_ERR_CUDA;
  if (v != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return STAMP_ERR_CUDA;
  }
  *status = v;
  return STAMP_OK;
}

int stamp_profile_gemm_events(void* start_event, void* stop_event) {
  if ((start_event == nullptr) != (stop_event == nullptr)) return STAMP_ERR_INVALID_ARG;
  t_gemm_ev_start = static_cast<cudaEvent_t>(start_event);
  t_gemm_ev_stop = static_cast<cudaEvent_t>(stop_event);
  return STAMP_OK;
}

int stamp_measure_i8_mma_issue(int nbatch, long long* ops_out, void* stream) {
  t_launches = 0;
  if (nbatch <= 0 || nbatch > (1 << 20) || !ops_out) return STAMP_ERR_INVALID_ARG;
  if (int rc = ensure_dyn_smem(reinterpret_cast<const void*>(k_peak_mma_i8), PEAK_SMEM)) return rc;
  const int grid = sm_count();
  k_peak_mma_i8<<<grid, PEAK_THREADS, PEAK_SMEM, static_cast<cudaStream_t>(stream)>>>(nbatch);
  STAMP_CHECK_LAUNCH();
  *ops_out = (long long)grid * nbatch * PEAK_BATCH * (2LL * 128 * 256 * 32);
  return STAMP_OK;
}

int stamp_debug_expire_wait(long long limit_cycles, void* stream) {
  t_launches = 0;
  if (limit_cycles <= 0 || limit_cycles > 2000000000LL) return STAMP_ERR_INVALID_ARG;
  k_expire_wait<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles);
  STAMP_CHECK_LAUNCH();
  return STAMP_OK;
}

int stamp_last_launch_count(void) { return t_launches; }

const char* stamp_status_string(int status) {
  switch (status) {
    case STAMP_OK: return "ok";
    case STAMP_ERR_INVALID_ARG: return "invalid argument";
    case STAMP_ERR_UNSUPPORTED: return "unsupported shape or configuration";
    case STAMP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case STAMP_ERR_CUDA: return "CUDA call failed";
    case STAMP_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case STAMP_ERR_TOO_LARGE: return "problem needs more scratch than the built-in array of the allocation-free call holds";
    default: return "unknown status";
  }
}

}  // extern "C"
