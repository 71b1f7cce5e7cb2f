/*
 * stamp.h -- C ABI of the B200 (sm_100a) STaMP-quantized linear layer.
 *
 * STaMP (Sequence Transformation and Mixed Precision, arXiv 2510.26771) mixes an activation
 * X [L tokens x K features] along the TOKEN axis with an orthonormal sequence transform L
 * (multi-level Haar DWT or DCT-II), quantizes each transformed token with its own scale --
 * the first k_hi tokens of each transform block at bits_hi (8), the others at bits_lo (4) --
 * multiplies the integer codes with per-output-channel quantized weights, de-quantizes, and
 * applies the inverse sequence transform to the output:
 *
 *        Y = L^-1 ( Q(L X) Q(W)^T ) + 1 bias^T            (Algorithm "STaMP Linear";
 *                                                          Method section, second equation)
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers owned by the caller; tensors are dense,
 *     row-major.  X: [B, L, K];  W: [N, K];  Y, Yt: [B, L, N].  B independent sequences.
 *   - Scratch space is the caller's `ws` buffer of at least stamp_workspace_bytes() bytes,
 *     256-byte aligned.  Calls that share a workspace must be ordered on one stream.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; they never synchronize the stream.
 *   - Every function returns a stamp_status.  Argument problems are detected on the host
 *     before anything is launched.  Device-side problems (a bounded wait inside a kernel that
 *     ran out) are recorded in a device status word read by stamp_last_device_status().
 *   - Shape rules: K % 128 == 0, N % 8 == 0, the transform block length (cfg.block, or L when
 *     0) is a power of two that divides L, Haar levels <= log2(block).  Anything else returns
 *     STAMP_ERR_UNSUPPORTED.
 *   - Transformed-token ("logical") order inside a block of n tokens:
 *       Haar, l levels: [a_l (n/2^l rows) | d_l | d_(l-1) | ... | d_1 (n/2 rows)], with
 *         a[i] = (x[2i] + x[2i+1]) / sqrt2,  d[i] = (x[2i] - x[2i+1]) / sqrt2  per level;
 *       DCT-II (orthonormal): row u = frequency u, row 0 = DC.
 *       Walsh-Hadamard (STAMP_T_WHT; the DCT reduced to its signs, same Section): orthonormal,
 *         sequency order -- row u changes sign u times along the block's tokens, row 0 = DC.
 *       2-D Haar (STAMP_T_HAAR2D; Sec. "Efficient Energy Concentration", LVM set-up: 3 levels on the
 *         64 x 64 patch grid leave 64 low-pass tokens): the block's n tokens are a raster-ordered
 *         grid of n / grid_w rows x grid_w columns; per level every 2 x 2 cell (a b / c d) gives
 *         LL = (a+b+c+d)/2, LH = (a-b+c-d)/2, HL = (a+b-c-d)/2, HH = (a-b-c+d)/2 and LL recurses;
 *         order [LL_l | LH_l | HL_l | HH_l | LH_(l-1) | ... | HH_1], bands in raster order;
 *         levels = 1..3, 2^levels divides both grid sides.
 *       Haar with the first token excluded (STAMP_T_HAAR_SKIP1; App. "Experimental details / LLMs", STaMP paragraph:
 *         the first token of an LLM sequence carries massive outliers, stays at 8 bits and is not transformed):
 *         row 0 of a block is its token 0 itself; the other n - 1 tokens go through a Haar transform whose first level
 *         pairs (x1, x2), (x3, x4), ... and carries the last token, which has no partner, into the low-pass band
 *         unchanged (that band has n / 2 entries, so all deeper levels are ordinary dyadic steps; the paper gives no
 *         rule for the odd length, this is the reading taken).  Order [x0 | a_l | d_l | ... | d_2 | d_1 (n/2 - 1 rows)],
 *         levels = 1..log2(n) (0 => log2 n).  Runs as separate transform, quantize, GEMM and inverse kernels.
 *     The 8-bit tokens are the rows {i : i mod n < k_hi}: the two-level allocation at the end of
 *     Sec. "Optimal bit allocation" (k_hi leading transformed tokens at bits_hi, the rest at bits_lo).
 *   - Quantizer (Sec. 2.1, first equation, symmetric form): scale = absmax / qmax,
 *     code = clamp(round_half_even(t / scale), -qmax, +qmax), qmax = 2^(bits-1) - 1; a zero
 *     row gets scale 1.  Nothing clips (min-max range setting of Sec. 2.1).
 */
#ifndef STAMP_H_
#define STAMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  STAMP_OK = 0,
  STAMP_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad enum value            */
  STAMP_ERR_UNSUPPORTED = 2, /* valid request outside the shape / transform rules above    */
  STAMP_ERR_WORKSPACE = 3,   /* ws is null, misaligned or smaller than required            */
  STAMP_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (launch, tensor map)   */
  STAMP_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (device status only)    */
  STAMP_ERR_TOO_LARGE = 6    /* stamp_inverse_noalloc: scratch need exceeds the built-in array */
} stamp_status;

typedef enum { STAMP_F32 = 0, STAMP_BF16 = 1 } stamp_dtype;

typedef enum { STAMP_T_IDENTITY = 0, STAMP_T_HAAR = 1, STAMP_T_DCT2 = 2, STAMP_T_HAAR2D = 3, STAMP_T_WHT = 4,
               STAMP_T_HAAR_SKIP1 = 5 } stamp_transform;

typedef enum { STAMP_G_PER_TOKEN = 0, STAMP_G_PER_CHANNEL = 1, STAMP_G_GROUP = 2 } stamp_granularity;

/* Weight operand formats accepted by the GEMM entry points. */
typedef enum {
  STAMP_W_PACKED4 = 0, /* [N, K/2] two's-complement nibbles, low nibble = even k (the output of
                          stamp_quantize_weights); expanded into the workspace on every call  */
  STAMP_W_INT8 = 1,    /* [N, K] one 4-bit code per int8 (the output of stamp_prepare_weights):
                          the tensor-core operand format, made once for static weights        */
  STAMP_W_INT8_AND_PACKED4 = 2 /* both: [N, K] int8 directly followed by [N, K/2] packed (the output of
                          stamp_prepare_weights_both).  The tensor cores read the first part; kernels that only
                          stream the weights (the product with the few tokens above the GEMM's tiles, for
                          short sequences) read the packed part and move half the bytes               */
} stamp_weight_format;

/* The knobs of the paper's problem statement. */
typedef struct {
  int32_t transform; /* stamp_transform: the sequence transform L                              */
  int32_t block;     /* tokens per transform block; 0 => the whole sequence (L tokens)         */
  int32_t levels;    /* Haar: number of levels, 1..log2(block); 0 => full depth. DCT: ignored  */
  int32_t k_hi;      /* the first k_hi transformed tokens OF EACH BLOCK use bits_hi            */
  int32_t bits_hi;   /* 8                                                                      */
  int32_t bits_lo;   /* 4                                                                      */
  int32_t bits_w;    /* 4 (weights, per output channel)                                        */
  int32_t act_gran;  /* STAMP_G_PER_TOKEN   (scales shared across features, Sec. 2.1)          */
  int32_t w_gran;    /* STAMP_G_PER_CHANNEL (one scale per output channel, Sec. "Set-up")      */
  int32_t grid_w;    /* STAMP_T_HAAR2D: width of the patch grid a block's tokens form; else 0  */
  int32_t act_zero_point; /* 0: symmetric activation codes (zero point 0, range +-(2^(b-1) - 1)).
                        1: the zero-point form Sec. 2.1's first equation prints, min-max range:
                           s = (max_j t_j - min_j t_j) / (2^b - 1)  (1 for a constant row),
                           z = rne(-min_j t_j / s),  x_int = clamp(rne(t / s) + z, 0, 2^b - 1).
                           Codes are STORED as c = x_int - 2^(b-1) in the same signed byte / nibble
                           formats as the symmetric ones, and the zero point handed out is that of
                           the stored code, zc = z - 2^(b-1):  t ~ s * (c - zc).  Every transform is
                           accepted; the layer then runs as separate transform, quantize, GEMM and
                           inverse kernels.                                                       */
  int32_t group;     /* 0: one scale per transformed token / per output channel (the fields above).
                        > 0: per-block scales (the LVM table's setting, "W4A4 per-block quantization with block size
                        64"): every run of `group` consecutive input features of a transformed token, and of a weight
                        row, has its own scale = absmax / qmax; act_gran and w_gran must both be STAMP_G_GROUP.
                        group = 64 * 2^i and divides K; symmetric codes only.  x_scale is then [B, L, K / group] and
                        w_scale [N, K / group], and
                          Yt[m, n] = sum_g (sum_{k in g} q[m,k] wq[n,k]) * x_scale[m, g] * w_scale[n, g].
                        The layer runs as separate transform, group quantizer, CUDA-core product and inverse kernels. */
} stamp_config;

/* Bytes of scratch any call below may need for this problem size (the maximum over the calls). */
int stamp_workspace_bytes(const stamp_config* cfg, int B, int L, int K, int N, size_t* out_bytes);

/*
 * Weight quantization (offline; weights are untouched by the sequence transform, Method
 * section): per output channel n, w_scale[n] = max_k |W[n,k]| / 7 and
 * wq[n,k] = clamp(rne(W[n,k] / w_scale[n]), -7, 7).
 *   W        [N, K]   w_dtype (STAMP_F32 or STAMP_BF16)      in
 *   wq       [N, K/2] packed 4-bit codes (STAMP_W_PACKED4)    out
 *   w_scale  [N]      float                                   out
 */
int stamp_quantize_weights(const stamp_config* cfg, const void* W, int w_dtype, int N, int K, void* wq,
                           float* w_scale, void* stream);

/* Expand packed weight codes into the tensor-core operand format (STAMP_W_INT8), once per
 * weight matrix.  wq_packed [N, K/2] in; w_int8 [N, K] out.  No counterpart in the paper: it
 * is a storage choice of this implementation (the int8 MMA consumes one code per byte). */
int stamp_prepare_weights(const stamp_config* cfg, const void* wq_packed, int N, int K, void* w_int8,
                          void* stream);

/* The same, with the packed codes kept behind the expanded ones (STAMP_W_INT8_AND_PACKED4): w_both holds
 * N * K + N * K / 2 bytes.  No counterpart in the paper. */
int stamp_prepare_weights_both(const stamp_config* cfg, const void* wq_packed, int N, int K, void* w_both, void* stream);

/*
 * Algorithm 1 ("STaMP linear layer"), its first two steps: sequence transform + per-token
 * mixed-precision quantization of one activation tensor.
 *   X        [B, L, K]   x_dtype                                                    in
 *   q_hi     [B * n_hi, K]        int8, the 8-bit tokens in logical order, where
 *            n_hi = k_hi * (L / block); row (b, blk, i) at index (b*(L/block)+blk)*k_hi + i   out
 *   q_lo     [B * (L-n_hi), K/2]  packed 4-bit codes of the remaining tokens in logical
 *            order (low nibble = even k)                                             out
 *   x_scale  [B, L]      float, per transformed token (logical order)                out
 *            With cfg->act_zero_point = 1 the buffer holds 2 * B * L words: the B * L scales, then the
 *            B * L zero points zc of the stored codes as int32.
 */
int stamp_quantize(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, void* q_hi,
                   void* q_lo, float* x_scale, void* ws, size_t ws_bytes, void* stream);

/*
 * Algorithm 1, the product step, on the integer codes, plus de-quantization (Sec. 2.1):
 *   Yt[m, n] = (sum_k q[m,k] * wq[n,k]) * x_scale[m] * w_scale[n],   int32 accumulation on the
 * tensor cores.  Output stays in the transformed token domain.
 *   q_hi, q_lo, x_scale : as written by stamp_quantize                               in
 *            With cfg->act_zero_point = 1 (x_scale then carries the zero points zc as well)
 *              Yt[m, n] = (sum_k c[m,k] * wq[n,k] - zc[m] * sum_k wq[n,k]) * x_scale[m] * w_scale[n],
 *            the same sum over (c - zc) * wq with the constant term taken out of the product.
 *   w, w_format, w_scale: weight codes (stamp_weight_format) and per-channel scales  in
 *   Yt       [B, L, N]   float                                                       out
 */
int stamp_linear(const stamp_config* cfg, const void* q_hi, const void* q_lo, const float* x_scale,
                 const void* w, int w_format, const float* w_scale, int B, int L, int K, int N, float* Yt,
                 void* ws, size_t ws_bytes, void* stream);

/*
 * De-quantization of stored codes, s (x_int - z) of Sec. 2.1: the transformed activation as the quantizer left it.
 * With stamp_quantize before and stamp_inverse (N = K, no bias) after it, this is STaMP on a tensor that is stored
 * rather than multiplied at once -- the KV cache of the LLM experiments (Table "STaMP always improves LLM
 * quantization": KV cache at 4 bits with the first 64 transformed tokens at 8; App. "Experimental details / LLMs":
 * scales per token and head).  A cache of H heads of dimension 128 is the activation [B * H, L, 128]: the per-token
 * scale of every sequence is then a per-token, per-head scale.
 *   q_hi, q_lo, x_scale : as written by stamp_quantize (zero points and per-block scales included)     in
 *   T        [B, L, K]   float, transformed-token (logical) order                                      out
 */
int stamp_dequantize(const stamp_config* cfg, const void* q_hi, const void* q_lo, const float* x_scale, int B, int L,
                     int K, float* T, void* stream);

/*
 * Algorithm 1, its last two steps: inverse sequence transform along tokens
 * (L^-1 = L^T, L orthonormal: Theorem 1's premise) and optional bias.
 *   Yt       [B, L, N]   float                                                       in
 *   bias     [N] float or NULL                                                       in
 *   Y        [B, L, N]   y_dtype (STAMP_F32 or STAMP_BF16)                           out
 */
int stamp_inverse(const stamp_config* cfg, const float* Yt, const float* bias, int B, int L, int N, void* Y,
                  int y_dtype, void* ws, size_t ws_bytes, void* stream);

/*
 * stamp_inverse() for callers that cannot hand over a workspace and must not allocate one.
 * (No counterpart in the paper: this is a packaging variant of the inverse-transform call.)
 *
 * Who needs it: code that runs where device allocation is off the table -- an operator plug-in
 * called from a serving loop whose host framework owns every byte of device memory, a callback
 * on a latency-critical path where cudaMalloc would stall the whole device, or a thin language
 * binding that has no allocator to ask.  Such a caller still owns Yt, bias and Y; what it lacks
 * is the few MB of scratch the multi-pass inverse keeps between its passes.
 *
 * Here that scratch is an array compiled into the library, STAMP_NOALLOC_SCRATCH_BYTES per GPU
 * that loads the library, resident until the process exits.  The call performs no cudaMalloc,
 * cudaFree or any other allocating routine.
 *   - Limit: what the inverse keeps between its launches must fit the array, otherwise
 *     STAMP_ERR_TOO_LARGE is returned before anything is launched:
 *       Haar: the partial sums of the coarse-to-fine passes -- nothing up to 5 levels, B*L/32 * N * 4
 *         bytes for 6 to 10 levels, (B*L/32 + B*L/1024) * N * 4 bytes beyond;
 *       DCT-II and Walsh-Hadamard: the dense block x block fp32 matrix, block^2 * 4 bytes -- a block of
 *         1024 tokens fills the 4 MiB exactly, longer blocks are refused;
 *       2-D Haar and identity: nothing.
 *     The first-token-excluded Haar transform is not served by this call (STAMP_ERR_UNSUPPORTED).
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to be cleared between
 *     calls: each call writes every element before reading it, so leftovers of the previous
 *     call are never seen.  Two calls that overlap on the GPU (different streams, no ordering
 *     between them) would overwrite each other's partial sums: order them.
 * Arguments and results are those of stamp_inverse().
 */
#define STAMP_NOALLOC_SCRATCH_BYTES (4u << 20)
int stamp_inverse_noalloc(const stamp_config* cfg, const float* Yt, const float* bias, int B, int L, int N,
                          void* Y, int y_dtype, void* stream);

/*
 * The whole Algorithm in one call: Y = L^-1( Q(L X) Q(W)^T ) + bias.  Intermediates (codes,
 * scales, transformed-domain output) live in the workspace only.
 * The call enqueues kernels on `stream` only (no synchronisation, no allocation): it may be recorded in a CUDA
 * graph by stream capture once it has run once outside a capture (function attributes are set on first use).
 */
int stamp_linear_fused(const stamp_config* cfg, const void* X, int x_dtype, const void* w, int w_format,
                       const float* w_scale, const float* bias, int B, int L, int K, int N, void* Y,
                       int y_dtype, void* ws, size_t ws_bytes, void* stream);

/*
 * The same call for callers whose activation and output live in HOST memory (ideally pinned):
 * copies X host->device, runs the layer, copies Y device->host, all enqueued on `stream`.  The
 * weight operand, scales and bias are device pointers as above.  `ws` must hold at least
 * stamp_workspace_bytes_host() bytes (the device workspace plus staging for X and Y).
 * No counterpart in the paper: a convenience for end-to-end measurement and host-side callers.
 */
int stamp_workspace_bytes_host(const stamp_config* cfg, int B, int L, int K, int N, int x_dtype, int y_dtype,
                               size_t* out_bytes);
int stamp_linear_fused_host(const stamp_config* cfg, const void* X_host, int x_dtype, const void* w, int w_format,
                            const float* w_scale, const float* bias, int B, int L, int K, int N, void* Y_host,
                            int y_dtype, void* ws, size_t ws_bytes, void* stream);

/* ---- parity / debug exports: the intermediate stages, judged separately against the oracle ---- */

/* T = L X in fp32, logical token order.  T [B, L, K] float out. */
int stamp_debug_transform(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, float* T,
                          void* ws, size_t ws_bytes, void* stream);

/* Codes written by stamp_quantize, one per int8, logical order.  codes [B, L, K] int8 out. */
int stamp_debug_unpack_codes(const stamp_config* cfg, const void* q_hi, const void* q_lo, int B, int L, int K,
                             int8_t* codes, void* stream);

/* Raw int32 accumulators of the tensor-core GEMM.  acc [B*L, N] int32 out. */
int stamp_debug_gemm_i32(const stamp_config* cfg, const void* q_hi, const void* q_lo, const void* w,
                         int w_format, int B, int L, int K, int N, int32_t* acc, void* ws, size_t ws_bytes,
                         void* stream);

/*
 * The token operand of the GEMM as the one-call layer (stamp_linear_fused) produces it, mapped back to logical
 * order.  For a Haar transform of at least 5 levels over blocks that are multiples of 256 tokens, and for the
 * three-level 2-D Haar transform, that call's transform+quantize kernels store their codes in the order the GEMM's
 * fused inverse consumes (not through the stamp_quantize format).  This export runs those same kernels on X and
 * gathers, for every logical transformed token (the order of stamp_quantize's outputs):
 *   codes   [B, L, K] int8   its codes as stored (zero-point mode: offset by 2^(b-1), as in stamp_quantize)      out
 *   factor  [B, L]    float  what the fused inverse multiplies the row's accumulators with: scale * 2^(-j/2) for
 *                            a 1-D Haar row of level j <= 8, the plain scale for rows of levels above 8 (they go
 *                            through a separate small product), scale * 2^(-l) for a 2-D Haar row of level l    out
 *   level   [B, L]    int32  that level j (or l)                                                                  out
 *   zero    [B, L]    int32  zero points of the stored codes (zero-point mode; zeros otherwise); may be NULL in
 *                            symmetric mode                                                                       out
 * Other configurations keep their operand in logical order (what stamp_quantize returns): STAMP_ERR_UNSUPPORTED.
 * No counterpart in the paper: the row order of the operand is a layout choice of this implementation, and parity
 * is judged on logical order.
 */
int stamp_debug_fused_operand(const stamp_config* cfg, const void* X, int x_dtype, int B, int L, int K, int N,
                              int8_t* codes, float* factor, int32_t* level, int32_t* zero, void* ws, size_t ws_bytes,
                              void* stream);

/* Synchronizes `stream`, then reads and clears the device status word of the current device.
 * *status is STAMP_OK or STAMP_ERR_TIMEOUT (a bounded wait inside a kernel expired; outputs of
 * the calls since the last read are then invalid). */
int stamp_last_device_status(void* stream, int* status);

/* Measurement hook: while both events are non-NULL, every tensor-core GEMM launched by the
 * calling thread is bracketed by cudaEventRecord(start) / cudaEventRecord(stop) on its stream
 * (each launch re-records the pair).  Pass NULLs to switch it off.  Events are cudaEvent_t. */
int stamp_profile_gemm_events(void* start_event, void* stop_event);

/* Test hook for the failure path: launches one thread that waits, with the same bounded wait the product
 * kernels use, on a barrier nobody completes.  After limit_cycles SM clocks (1 .. 2e9) the wait gives up, the
 * kernel records STAMP_ERR_TIMEOUT in the device status word and returns normally; the next
 * stamp_last_device_status() reports it once.  Nothing faults or hangs.  No counterpart in the paper. */
int stamp_debug_expire_wait(long long limit_cycles, void* stream);

/* Measurement: the rate of the tensor cores' int8 instruction alone.  Launches one CTA per SM; each issues
 * nbatch * 64 tcgen05.mma kind::i8 instructions (M128 x N256 x K32, int32 accumulators in tensor memory) on
 * operand tiles that stay in shared memory -- no loads in the loop, waits bounded -- and *ops_out receives the
 * integer operations of the whole launch (2 * M * N * K per instruction).  The caller times the launch with
 * events on `stream`; ops / time is the ceiling the layer's GEMM is reported against.  No counterpart in the
 * paper: it measures the machine.  1 <= nbatch <= 2^20. */
int stamp_measure_i8_mma_issue(int nbatch, long long* ops_out, void* stream);

/* How many kernels of this library the calling thread's last API call launched. */
int stamp_last_launch_count(void);

const char* stamp_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* STAMP_H_ */
