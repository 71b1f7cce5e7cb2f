/*
 * CPU oracle for the STaMP-quantized linear layer (STaMP, arXiv 2510.26771).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the
 * layer computes, written from the paper.  It is used by the tests, by the smoke check
 * and by the benchmark's CPU-baseline leg; the CUDA product path never calls it and
 * shares no code, header, table or helper with it.
 *
 * What it follows:
 *   - Algorithm "STaMP Linear" (Method section): X <- L X; x_i <- Q(x_i; b_i);
 *     Y <- X W^T; Y <- L^{-1} Y; Y <- Y + bias.
 *   - Activation quantizer, Background Sec. 2.1, first equation (integer quantization with
 *     per-token scale shared across features), in its symmetric form: zero-point 0, codes
 *     in [-(2^(b-1)-1), +(2^(b-1)-1)], scale = absmax / qmax so that nothing clips (the
 *     min-max, "no clipping error" range setting of the same section); and, selectable, in
 *     the form the equation prints: unsigned codes with an integer zero point, s = range / (2^b - 1).
 *   - Two-level bit allocation (end of Sec. "Optimal bit allocation"): the first k_hi
 *     transformed tokens of each transform block use bits_hi, the rest bits_lo.
 *   - Sequence transforms (Sec. "Efficient Energy Concentration"): orthonormal multi-level
 *     Haar DWT and orthonormal DCT-II along the token axis, as explicit matrices.
 *   - Commutation identity (Method, second equation): the inverse sequence transform is
 *     applied after the matmul; for an orthonormal L, L^{-1} = L^T (Theorem 1's premise).
 *
 * Pins (tests/test_oracle_pins.py): orthonormality, closed-form Haar rows, SciPy's
 * orthonormal DCT-II, energy preservation, exact reconstruction, identity of the
 * unquantized pipeline with X W^T, the bias form l = L 1, rounding/error bounds, the
 * printed effective bit-widths 4.0625 and 4.125, brute force on tiny shapes; for the zero-point
 * quantizer a hand-computed row, the section's error bound d s^2 / 4, the nearest-level property by
 * brute force, and the integer product against a float product of the de-quantized operands.
 * Conventions that no pin can fix (they are choices shared with the CUDA path by
 * specification; "parity unpinned" for these): the sign of the Haar detail rows, the
 * round-half-to-even tie rule, symmetric instead of zero-point codes.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o libstamp_oracle.so stamp_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_T_IDENTITY = 0, ORACLE_T_HAAR = 1, ORACLE_T_DCT2 = 2, ORACLE_T_HAAR2D = 3, ORACLE_T_WHT = 4,
       ORACLE_T_HAAR_SKIP1 = 5 };

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------------------------
 * Sequence transform matrices (n x n, row-major, fp64).
 * ------------------------------------------------------------------------------------------ */

/* One Haar analysis step on the first `len` entries of v (the Haar wavelet the paper names in
 * Sec. "Efficient Energy Concentration"): averages go to the first half, differences to the
 * second half, both scaled by 1/sqrt(2) so the step is orthonormal.  Sign convention of the
 * difference: first minus second. */
static void haar_step(double* v, int len, double* tmp) {
  const double r = 1.0 / sqrt(2.0);
  int half = len / 2;
  for (int i = 0; i < half; ++i) {
    tmp[i] = (v[2 * i] + v[2 * i + 1]) * r;
    tmp[half + i] = (v[2 * i] - v[2 * i + 1]) * r;
  }
  memcpy(v, tmp, sizeof(double) * (size_t)len);
}

/* Multi-level Haar DWT of a length-n vector: each level re-applies the step to the low-pass
 * half, so that the energy moves into the leading entries level by level (Sec. "Efficient Energy
 * Concentration"); after `levels` levels the order
 * is [a_levels | d_levels | d_{levels-1} | ... | d_1]. */
static void haar_forward(double* v, int n, int levels, double* tmp) {
  int len = n;
  for (int l = 0; l < levels; ++l) {
    haar_step(v, len, tmp);
    len /= 2;
  }
}

/* Haar analysis of a block whose FIRST token is left alone (App. "Experimental details / LLMs", STaMP paragraph:
 * the first token of an LLM sequence carries massive outliers, stays at 8 bits, and the sequence transform is
 * not applied to it).  The paper gives no rule for the odd number of tokens that remain; the reading taken here:
 * the step pairs neighbours as usual and an element without a partner is CARRIED into the low-pass half
 * unchanged (so a step on m entries yields ceil(m/2) averages-or-carried and floor(m/2) differences, and is
 * still orthonormal: 2 x 2 rotations plus a 1 x 1 identity).  v[0] is the excluded token; the transform acts on
 * v[1..n-1].  Output order: [token 0 | a_levels | d_levels | ... | d_1]. */
static void haar_step_carry(double* v, int len, double* tmp) {
  const double r = 1.0 / sqrt(2.0);
  int pairs = len / 2, lows = len - pairs;   /* lows = ceil(len / 2) */
  for (int i = 0; i < pairs; ++i) {
    tmp[i] = (v[2 * i] + v[2 * i + 1]) * r;
    tmp[lows + i] = (v[2 * i] - v[2 * i + 1]) * r;
  }
  if (len & 1) tmp[pairs] = v[len - 1];      /* no partner: carried, unscaled */
  memcpy(v, tmp, sizeof(double) * (size_t)len);
}

static void haar_forward_skip_first(double* v, int n, int levels, double* tmp) {
  int len = n - 1;
  for (int l = 0; l < levels && len > 1; ++l) {
    haar_step_carry(v + 1, len, tmp);
    len = len - len / 2;
  }
}

static int ilog2_exact(int n) {
  int l = 0;
  while ((1 << l) < n) ++l;
  return ((1 << l) == n) ? l : -1;
}

/* Resolve levels: 0 means full depth log2(n). Returns -1 when unsupported. */
static int resolve_levels(int transform, int n, int levels) {
  if (transform != ORACLE_T_HAAR && transform != ORACLE_T_HAAR_SKIP1) return 0;
  int full = ilog2_exact(n);
  if (full < 0) return -1;
  if (levels == 0) return full;
  if (levels < 0 || levels > full) return -1;
  return levels;
}

/* Dense explicit transform matrix.  Column t of the Haar matrix is the transform of the unit
 * vector e_t; the DCT-II matrix is C[u][t] = c_u sqrt(2/n) cos(pi (2t+1) u / (2n)) with
 * c_0 = 1/sqrt(2) (orthonormal, row 0 = DC so low frequencies come first). */
int oracle_transform_matrix(int transform, int n, int levels, double* Lmat) {
  if (n <= 0) return 1;
  if (transform == ORACLE_T_IDENTITY) {
    memset(Lmat, 0, sizeof(double) * (size_t)n * n);
    for (int i = 0; i < n; ++i) Lmat[(size_t)i * n + i] = 1.0;
    return 0;
  }
  if (transform == ORACLE_T_HAAR || transform == ORACLE_T_HAAR_SKIP1) {
    int lv = resolve_levels(transform, n, levels);
    if (lv < 0) return 2;
    int err = 0;
#pragma omp parallel
    {
      double* v = (double*)malloc(sizeof(double) * (size_t)n);
      double* tmp = (double*)malloc(sizeof(double) * (size_t)n);
      if (!v || !tmp) {
#pragma omp atomic write
        err = 3;
      } else {
#pragma omp for schedule(static)
        for (int t = 0; t < n; ++t) {
          memset(v, 0, sizeof(double) * (size_t)n);
          v[t] = 1.0;
          if (transform == ORACLE_T_HAAR_SKIP1)
            haar_forward_skip_first(v, n, lv, tmp);
          else
            haar_forward(v, n, lv, tmp);
          for (int i = 0; i < n; ++i) Lmat[(size_t)i * n + t] = v[i];
        }
      }
      free(v);
      free(tmp);
    }
    return err;
  }
  if (transform == ORACLE_T_WHT) {
    /* Walsh-Hadamard transform (Sec. "Efficient Energy Concentration": the DCT with only the signs
     * of the basis kept).  Rows are the Walsh functions in SEQUENCY order -- row u changes sign u
     * times along the tokens -- so that, as for the DCT, the slowly varying rows come first.  Built
     * from the definition: the natural-order Hadamard matrix H[i][j] = (-1)^popcount(i & j), every
     * row put at the index given by its number of sign changes, scaled by 1 / sqrt n. */
    if (ilog2_exact(n) < 0) return 2;
    double r = 1.0 / sqrt((double)n);
    unsigned char* used = (unsigned char*)calloc((size_t)n, 1);
    if (!used) return 3;
    int bad = 0;
    for (int i = 0; i < n; ++i) {
      int changes = 0, prev = 0;
      for (int j = 0; j < n; ++j) {
        int bits = i & j, par = 0;
        while (bits) { par ^= 1; bits &= bits - 1; }
        if (j > 0 && par != prev) ++changes;
        prev = par;
      }
      if (used[changes]) bad = 1;
      used[changes] = 1;
      for (int j = 0; j < n; ++j) {
        int bits = i & j, par = 0;
        while (bits) { par ^= 1; bits &= bits - 1; }
        Lmat[(size_t)changes * n + j] = par ? -r : r;
      }
    }
    free(used);
    return bad ? 4 : 0;
  }
  if (transform == ORACLE_T_DCT2) {
    const double pi = 3.14159265358979323846264338327950288;
    for (int u = 0; u < n; ++u) {
      double cu = (u == 0) ? 1.0 / sqrt(2.0) : 1.0;
      for (int t = 0; t < n; ++t)
        Lmat[(size_t)u * n + t] = cu * sqrt(2.0 / n) * cos(pi * (2.0 * t + 1.0) * u / (2.0 * n));
    }
    return 0;
  }
  return 2;
}

/* ------------------------------------------------------------------------------------------
 * 2-D Haar DWT over a patch grid (Sec. "Efficient Energy Concentration": for image tokens the
 * wavelet transform is taken over the two spatial axes, "one quarter" of the tokens staying
 * low-pass per level; Set-up of the LVM experiments: 3 levels on a 64 x 64 grid leave 64 low-pass
 * tokens).  The n tokens of a block are a grid of h = n / w rows by w columns in raster order.
 * One level maps every 2 x 2 cell (a b / c d) to
 *     LL = (a + b + c + d) / 2   LH = (a - b + c - d) / 2   (difference along a row)
 *     HL = (a + b - c - d) / 2   HH = (a - b - c + d) / 2   (difference across rows / both)
 * and recurses on the LL grid.  Output order after l levels:
 *     [LL_l | LH_l | HL_l | HH_l | LH_(l-1) | HL_(l-1) | HH_(l-1) | ... | LH_1 | HL_1 | HH_1],
 * each band in raster order of its (h >> level) x (w >> level) grid.  Band order and signs are a
 * convention of this implementation (the paper fixes neither).
 * ------------------------------------------------------------------------------------------ */
static void haar2d_forward(double* v, int h, int w, int levels, double* tmp) {
  int n = h * w;
  /* grid[] holds the current LL grid in raster order at the front of v */
  int ch = h, cw = w;
  for (int l = 1; l <= levels; ++l) {
    int nh = ch / 2, nw = cw / 2, q = nh * nw;
    for (int y = 0; y < nh; ++y)
      for (int x = 0; x < nw; ++x) {
        double a = v[(2 * y) * cw + 2 * x], b = v[(2 * y) * cw + 2 * x + 1];
        double c = v[(2 * y + 1) * cw + 2 * x], d = v[(2 * y + 1) * cw + 2 * x + 1];
        int i = y * nw + x;
        tmp[i] = (a + b + c + d) * 0.5;
        tmp[q + i] = (a - b + c - d) * 0.5;
        tmp[2 * q + i] = (a + b - c - d) * 0.5;
        tmp[3 * q + i] = (a - b - c + d) * 0.5;
      }
    memcpy(v, tmp, sizeof(double) * (size_t)(4 * q));
    ch = nh;
    cw = nw;
  }
  (void)n;
}

/* Dense matrix of the 2-D Haar transform of a block of n tokens laid out as (n / grid_w) x grid_w. */
int oracle_transform_matrix2d(int n, int grid_w, int levels, double* Lmat) {
  if (n <= 0 || grid_w <= 0 || n % grid_w) return 1;
  int h = n / grid_w;
  if (levels <= 0 || (h >> levels) << levels != h || (grid_w >> levels) << levels != grid_w) return 2;
  double* v = (double*)malloc(sizeof(double) * (size_t)n);
  double* tmp = (double*)malloc(sizeof(double) * (size_t)n);
  if (!v || !tmp) { free(v); free(tmp); return 3; }
  for (int t = 0; t < n; ++t) {
    memset(v, 0, sizeof(double) * (size_t)n);
    v[t] = 1.0;
    haar2d_forward(v, h, grid_w, levels, tmp);
    for (int i = 0; i < n; ++i) Lmat[(size_t)i * n + t] = v[i];
  }
  free(v);
  free(tmp);
  return 0;
}

/* The same Haar matrix in CSR form for block lengths whose dense matrix would not fit in
 * memory.  Rows are produced from the same unit-vector construction, keeping the non-zeros.
 * row_ptr has n+1 entries; col/val must hold n*(levels+1) entries. */
int oracle_haar_matrix_csr(int n, int levels, int64_t* row_ptr, int32_t* col, double* val) {
  int lv = resolve_levels(ORACLE_T_HAAR, n, levels);
  if (lv < 0) return 2;
  /* pass 1: per-column non-zeros (each column has exactly lv+1 of them) */
  size_t per_col = (size_t)lv + 1;
  int32_t* crow = (int32_t*)malloc(sizeof(int32_t) * per_col * (size_t)n);
  double* cval = (double*)malloc(sizeof(double) * per_col * (size_t)n);
  if (!crow || !cval) { free(crow); free(cval); return 3; }
  int err = 0;
#pragma omp parallel
  {
    double* v = (double*)malloc(sizeof(double) * (size_t)n);
    double* tmp = (double*)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(static)
    for (int t = 0; t < n; ++t) {
      memset(v, 0, sizeof(double) * (size_t)n);
      v[t] = 1.0;
      haar_forward(v, n, lv, tmp);
      size_t c = 0;
      for (int i = 0; i < n; ++i)
        if (v[i] != 0.0) {
          if (c < per_col) { crow[(size_t)t * per_col + c] = i; cval[(size_t)t * per_col + c] = v[i]; }
          ++c;
        }
      if (c != per_col) {
#pragma omp atomic write
        err = 4;
      }
    }
    free(v);
    free(tmp);
  }
  if (err) { free(crow); free(cval); return err; }
  /* pass 2: transpose the column lists into CSR */
  for (int i = 0; i <= n; ++i) row_ptr[i] = 0;
  for (size_t e = 0; e < per_col * (size_t)n; ++e) row_ptr[crow[e] + 1]++;
  for (int i = 0; i < n; ++i) row_ptr[i + 1] += row_ptr[i];
  int64_t* fill = (int64_t*)malloc(sizeof(int64_t) * (size_t)n);
  if (!fill) { free(crow); free(cval); return 3; }
  for (int i = 0; i < n; ++i) fill[i] = row_ptr[i];
  for (int t = 0; t < n; ++t)
    for (size_t c = 0; c < per_col; ++c) {
      int i = crow[(size_t)t * per_col + c];
      col[fill[i]] = t;
      val[fill[i]] = cval[(size_t)t * per_col + c];
      fill[i]++;
    }
  free(fill);
  free(crow);
  free(cval);
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Applying the transform along the token axis: T_b = blockdiag(Lmat) * X_b  (the transform step of
 * Algorithm 1), or its transpose (the inverse-transform step, with L^{-1} = L^T).
 * X: [B, L, K] row-major.  Lmat: n x n, n divides L.  Plain triple loop; exact zeros of the
 * matrix are skipped (they contribute nothing).
 * ------------------------------------------------------------------------------------------ */
int oracle_apply_dense_f64(const double* Lmat, int n, int transpose, const double* X, int B, int L, int K,
                           double* out) {
  if (n <= 0 || L % n) return 1;
  long nblk = (long)B * (L / n);
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
  for (long blk = 0; blk < nblk; ++blk)
    for (int i = 0; i < n; ++i) {
      const double* xb = X + (size_t)blk * n * K;
      double* o = out + ((size_t)blk * n + i) * K;
      for (int j = 0; j < K; ++j) o[j] = 0.0;
      for (int t = 0; t < n; ++t) {
        double l = transpose ? Lmat[(size_t)t * n + i] : Lmat[(size_t)i * n + t];
        if (l == 0.0) continue;
        const double* xr = xb + (size_t)t * K;
        for (int j = 0; j < K; ++j) o[j] += l * xr[j];
      }
    }
  return 0;
}

int oracle_apply_dense_f32in(const double* Lmat, int n, const float* X, int B, int L, int K, double* out) {
  if (n <= 0 || L % n) return 1;
  long nblk = (long)B * (L / n);
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
  for (long blk = 0; blk < nblk; ++blk)
    for (int i = 0; i < n; ++i) {
      const float* xb = X + (size_t)blk * n * K;
      double* o = out + ((size_t)blk * n + i) * K;
      for (int j = 0; j < K; ++j) o[j] = 0.0;
      for (int t = 0; t < n; ++t) {
        double l = Lmat[(size_t)i * n + t];
        if (l == 0.0) continue;
        const float* xr = xb + (size_t)t * K;
        for (int j = 0; j < K; ++j) o[j] += l * (double)xr[j];
      }
    }
  return 0;
}

/* CSR forward apply (float input): out[blk*n + i, :] = sum_e val[e] * X[blk*n + col[e], :]. */
int oracle_apply_csr_f32in(const int64_t* row_ptr, const int32_t* col, const double* val, int n,
                           const float* X, int B, int L, int K, double* out) {
  if (n <= 0 || L % n) return 1;
  long nblk = (long)B * (L / n);
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
  for (long blk = 0; blk < nblk; ++blk)
    for (int i = 0; i < n; ++i) {
      const float* xb = X + (size_t)blk * n * K;
      double* o = out + ((size_t)blk * n + i) * K;
      for (int j = 0; j < K; ++j) o[j] = 0.0;
      for (int64_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
        double l = val[e];
        const float* xr = xb + (size_t)col[e] * K;
        for (int j = 0; j < K; ++j) o[j] += l * (double)xr[j];
      }
    }
  return 0;
}

/* CSR transpose apply: out[blk*n + t, :] = sum_i L[i][t] * Yt[blk*n + i, :].
 * Parallel over column chunks so that rows of `out` are never shared between threads. */
int oracle_apply_csr_transpose_f64(const int64_t* row_ptr, const int32_t* col, const double* val, int n,
                                   const double* Yt, int B, int L, int K, double* out) {
  if (n <= 0 || L % n) return 1;
  long nblk = (long)B * (L / n);
  const int chunk = 64;
  int nchunk = (K + chunk - 1) / chunk;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (long blk = 0; blk < nblk; ++blk)
    for (int c = 0; c < nchunk; ++c) {
      int j0 = c * chunk, j1 = (j0 + chunk < K) ? j0 + chunk : K;
      for (int t = 0; t < n; ++t) {
        double* o = out + ((size_t)blk * n + t) * K;
        for (int j = j0; j < j1; ++j) o[j] = 0.0;
      }
      for (int i = 0; i < n; ++i) {
        const double* yr = Yt + ((size_t)blk * n + i) * K;
        for (int64_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
          double l = val[e];
          double* o = out + ((size_t)blk * n + col[e]) * K;
          for (int j = j0; j < j1; ++j) o[j] += l * yr[j];
        }
      }
    }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Bit allocation: bits[i] for each transformed token of one sequence of length L made of
 * blocks of n tokens: the first k_hi rows of every block get bits_hi, the others bits_lo.
 * ------------------------------------------------------------------------------------------ */
int oracle_bit_map(int L, int n, int k_hi, int bits_hi, int bits_lo, int32_t* bits) {
  if (n <= 0 || L % n || k_hi < 0 || k_hi > n) return 1;
  for (int i = 0; i < L; ++i) bits[i] = ((i % n) < k_hi) ? bits_hi : bits_lo;
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Per-row symmetric round-to-nearest quantizer (Sec. 2.1, first equation, with z = 0).
 *   amax  = max_j |t_j|                        (fp64)
 *   scale = (float)amax / (float)qmax          (evaluated in fp32: the scale is an fp32
 *                                               output of the method); amax == 0 -> scale 1
 *   q_j   = clamp(rne((float)t_j / scale), -qmax, qmax),   qmax = 2^(bits-1) - 1
 * rne = round half to even (rintf in the default rounding mode).
 * The rounding decision is taken in fp32: the transformed value is rounded to fp32 and
 * divided by the fp32 scale with an IEEE fp32 division.  The paper fixes no precision for this
 * step; low-precision inputs (bf16 activations and weights) land EXACTLY on rounding
 * boundaries often (whenever absmax has a mantissa divisible by qmax), so the precision in
 * which the tie is seen decides the code, and fp32 is the precision of the scale itself.
 * The other reading -- the quotient t_j / (double)scale evaluated and rounded in fp64 -- can be
 * selected with oracle_set_rounding_decision(1); tests/test_oracle_pins.py counts how many codes
 * the two readings disagree on for the named configurations.
 * bits_per_row has `period` entries and row r uses bits_per_row[r % period].
 * ------------------------------------------------------------------------------------------ */
static int g_decide_fp64 = 0;

/* 0 (default): rounding decision on the fp32 quotient; 1: on the fp64 quotient.  Returns the old value. */
int oracle_set_rounding_decision(int fp64) {
  int old = g_decide_fp64;
  g_decide_fp64 = fp64 ? 1 : 0;
  return old;
}

int oracle_quantize_rows(const double* T, long rows, int K, const int32_t* bits_per_row, int period,
                         float* scale, int8_t* codes) {
  if (period <= 0) return 1;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const double* t = T + (size_t)r * K;
    int bits = bits_per_row[r % period];
    float qmaxf = (float)((1 << (bits - 1)) - 1);
    double amax = 0.0;
    for (int j = 0; j < K; ++j) {
      double a = fabs(t[j]);
      if (a > amax) amax = a;
    }
    float s = (amax > 0.0) ? ((float)amax / qmaxf) : 1.0f;
    if (!(s > 0.0f)) s = 1.0f; /* amax so small that the fp32 scale underflowed */
    scale[r] = s;
    for (int j = 0; j < K; ++j) {
      float q = g_decide_fp64 ? (float)nearbyint(t[j] / (double)s) : rintf((float)t[j] / s);
      if (q > qmaxf) q = qmaxf;
      if (q < -qmaxf) q = -qmaxf;
      codes[(size_t)r * K + j] = (int8_t)q;
    }
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Per-row asymmetric (zero-point) round-to-nearest quantizer: Sec. 2.1, first equation, as printed,
 *   x_int = clamp(rne(x / s) + z, 0, 2^b - 1),      de-quantized value  s * (x_int - z),
 * with the min-max range setting of the same section (the one under which its error bound holds):
 *   s = range(x) / (2^b - 1),  range(x) = max_j x_j - min_j x_j,      z = rne(-min_j x_j / s).
 * The printed scale formula of that passage is the reciprocal of the s used in the equation and in
 * the bound; the reading taken here is the one consistent with both.  z is an integer (it is added
 * to an integer code) and is not clamped to the code range: a row that does not straddle zero has
 * z < 0 or z > 2^b - 1 and still uses all its codes.  |z| is limited to 2^30 so that it fits an
 * int32 (only a row whose range is ~1e-7 of its offset gets there).  range == 0 (a constant row; the
 * zero row of a padded sequence) takes s = 1.
 * As in the symmetric quantizer, min, max, s and the rounding decision are taken in fp32.
 * ------------------------------------------------------------------------------------------ */
int oracle_quantize_rows_asym(const double* T, long rows, int K, const int32_t* bits_per_row, int period,
                              float* scale, int32_t* zero, uint8_t* codes) {
  if (period <= 0) return 1;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const double* t = T + (size_t)r * K;
    int bits = bits_per_row[r % period];
    float top = (float)((1 << bits) - 1);
    float mn = (float)t[0], mx = (float)t[0];
    for (int j = 1; j < K; ++j) {
      float v = (float)t[j];
      if (v < mn) mn = v;
      if (v > mx) mx = v;
    }
    float s = (mx - mn) / top;
    if (!(s > 0.0f)) s = 1.0f;
    float zf = rintf(-mn / s);
    if (zf > 1073741824.0f) zf = 1073741824.0f;
    if (zf < -1073741824.0f) zf = -1073741824.0f;
    scale[r] = s;
    zero[r] = (int32_t)zf;
    for (int j = 0; j < K; ++j) {
      float q = rintf((float)t[j] / s) + zf;
      if (q > top) q = top;
      if (q < 0.0f) q = 0.0f;
      codes[(size_t)r * K + j] = (uint8_t)q;
    }
  }
  return 0;
}

/* Integer matmul on zero-point codes: acc[m][n] = sum_k (q[m][k] - z[m]) * wq[n][k]  (the de-quantized
 * activation of Sec. 2.1 is s (x_int - z); the scale is applied afterwards).  int64 accumulation,
 * checked to fit int32 (returns 5 otherwise). */
int oracle_gemm_zp_i32(const uint8_t* q, const int32_t* zero, const int8_t* wq, long M, int N, int K,
                       int32_t* acc) {
  int overflow = 0;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      int64_t s = 0;
      const uint8_t* a = q + (size_t)m * K;
      const int8_t* b = wq + (size_t)n * K;
      for (int k = 0; k < K; ++k) s += ((int64_t)a[k] - (int64_t)zero[m]) * (int64_t)b[k];
      if (s > INT32_MAX || s < INT32_MIN) {
#pragma omp atomic write
        overflow = 1;
      }
      acc[(size_t)m * N + n] = (int32_t)s;
    }
  return overflow ? 5 : 0;
}

/* float-input convenience for the weights (per output channel, Sec. "Set-up": a separate
 * scale for each weight output channel; round-to-nearest). */
int oracle_quantize_rows_f32in(const float* W, long rows, int K, int bits, float* scale, int8_t* codes) {
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const float* t = W + (size_t)r * K;
    float qmaxf = (float)((1 << (bits - 1)) - 1);
    double amax = 0.0;
    for (int j = 0; j < K; ++j) {
      double a = fabs((double)t[j]);
      if (a > amax) amax = a;
    }
    float s = (amax > 0.0) ? ((float)amax / qmaxf) : 1.0f;
    if (!(s > 0.0f)) s = 1.0f;
    scale[r] = s;
    for (int j = 0; j < K; ++j) {
      float q = rintf(t[j] / s);
      if (q > qmaxf) q = qmaxf;
      if (q < -qmaxf) q = -qmaxf;
      codes[(size_t)r * K + j] = (int8_t)q;
    }
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Per-block ("group") scales along the feature axis (the LVM table's setting: W4A4 per-block quantization with
 * block size 64; App. "Experimental details / LVMs": per-block weight and activation quantization as in SVDQuant).
 * Every run of `group` consecutive features of a row has a scale of its own,
 *   s[r][g] = (float)max_{k in g}|t[r][k]| / (float)qmax   (1 for an all-zero group),
 *   q[r][k] = clamp(rne((float)t[r][k] / s[r][k / group]), -qmax, qmax),
 * the symmetric quantizer of oracle_quantize_rows applied group by group (same fp32 rounding decision).  The
 * paper names the scheme and the block size, not its formulas: symmetric codes and absmax range are the
 * reading shared with the per-token quantizer.  K must be a multiple of group.  scale is [rows][K / group].
 * ------------------------------------------------------------------------------------------ */
int oracle_quantize_rows_grouped(const double* T, long rows, int K, const int32_t* bits_per_row, int period, int group,
                                 float* scale, int8_t* codes) {
  if (period <= 0 || group <= 0 || K % group) return 1;
  int ng = K / group;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const double* t = T + (size_t)r * K;
    int bits = bits_per_row[r % period];
    float qmaxf = (float)((1 << (bits - 1)) - 1);
    for (int g = 0; g < ng; ++g) {
      double amax = 0.0;
      for (int j = g * group; j < (g + 1) * group; ++j) {
        double a = fabs(t[j]);
        if (a > amax) amax = a;
      }
      float s = (amax > 0.0) ? ((float)amax / qmaxf) : 1.0f;
      if (!(s > 0.0f)) s = 1.0f;
      scale[(size_t)r * ng + g] = s;
      for (int j = g * group; j < (g + 1) * group; ++j) {
        float q = rintf((float)t[j] / s);
        if (q > qmaxf) q = qmaxf;
        if (q < -qmaxf) q = -qmaxf;
        codes[(size_t)r * K + j] = (int8_t)q;
      }
    }
  }
  return 0;
}

int oracle_quantize_rows_grouped_f32in(const float* W, long rows, int K, int bits, int group, float* scale, int8_t* codes) {
  if (group <= 0 || K % group) return 1;
  double* t = (double*)malloc(sizeof(double) * (size_t)rows * K);
  if (!t) return 3;
  for (size_t i = 0; i < (size_t)rows * K; ++i) t[i] = (double)W[i];
  int32_t b = bits;
  int rc = oracle_quantize_rows_grouped(t, rows, K, &b, 1, group, scale, codes);
  free(t);
  return rc;
}

/* Product of two group-scaled operands, de-quantized (Sec. 2.1: (x_int - z) s with z = 0, once per group):
 *   Yt[m][n] = sum_g ( sum_{k in g} q[m][k] wq[n][k] ) * sx[m][g] * sw[n][g]
 * The inner sums are exact integers (int64, far from overflow for a group); the outer sum runs over the groups
 * in increasing order in fp64. */
int oracle_gemm_grouped(const int8_t* q, const float* sx, const int8_t* wq, const float* sw, long M, int N, int K,
                        int group, double* Yt) {
  if (group <= 0 || K % group) return 1;
  int ng = K / group;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      const int8_t* a = q + (size_t)m * K;
      const int8_t* b = wq + (size_t)n * K;
      double y = 0.0;
      for (int g = 0; g < ng; ++g) {
        int64_t acc = 0;
        for (int k = g * group; k < (g + 1) * group; ++k) acc += (int64_t)a[k] * (int64_t)b[k];
        y += (double)acc * (double)sx[(size_t)m * ng + g] * (double)sw[(size_t)n * ng + g];
      }
      Yt[(size_t)m * N + n] = y;
    }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Integer matmul (the product step of Algorithm 1, on the integer codes): naive triple loop,
 * acc[m][n] = sum_k q[m][k] * wq[n][k], accumulated in int64 and checked to fit int32.
 * Returns 5 if any accumulator would overflow int32.
 * ------------------------------------------------------------------------------------------ */
int oracle_gemm_i32(const int8_t* q, const int8_t* wq, long M, int N, int K, int32_t* acc) {
  int overflow = 0;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      int64_t s = 0;
      const int8_t* a = q + (size_t)m * K;
      const int8_t* b = wq + (size_t)n * K;
      for (int k = 0; k < K; ++k) s += (int64_t)a[k] * (int64_t)b[k];
      if (s > INT32_MAX || s < INT32_MIN) {
#pragma omp atomic write
        overflow = 1;
      }
      acc[(size_t)m * N + n] = (int32_t)s;
    }
  return overflow ? 5 : 0;
}

/* De-quantization (Sec. 2.1: (x_int - z) s with z = 0, applied to the product of two
 * quantized operands): Yt[m][n] = acc[m][n] * s_x[m] * s_w[n]. */
int oracle_dequant(const int32_t* acc, const float* sx, const float* sw, long M, int N, double* Yt) {
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n)
      Yt[(size_t)m * N + n] = (double)acc[(size_t)m * N + n] * (double)sx[m] * (double)sw[n];
  return 0;
}

/* Unquantized reference product X W^T in fp64 (what the layer approximates). */
int oracle_matmul_f64(const float* X, const float* W, long M, int N, int K, double* Y) {
#pragma omp parallel for schedule(static)
  for (long m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      double s = 0.0;
      const float* a = X + (size_t)m * K;
      const float* b = W + (size_t)n * K;
      for (int k = 0; k < K; ++k) s += (double)a[k] * (double)b[k];
      Y[(size_t)m * N + n] = s;
    }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * The whole layer, in the Algorithm's order.  Every intermediate can be captured by passing a
 * non-null pointer.  X: [B, L, K] float (values already rounded to the storage dtype), W:
 * [N, K] float, bias: [N] or null.  The transform acts on blocks of n tokens (n = block, or L
 * when block == 0); Haar uses `levels` levels (0 = log2 n).
 *   T        [B*L, K]  fp64   transformed activations
 *   x_scale  [B*L]     fp32   per transformed token
 *   q        [B*L, K]  int8   activation codes (logical, transformed-row order)
 *   w_scale  [N]       fp32   per output channel
 *   wq       [N, K]    int8   weight codes
 *   acc      [B*L, N]  int32  integer accumulators
 *   Yt       [B*L, N]  fp64   de-quantized output, transformed domain
 *   Y        [B*L, N]  fp64   final output
 * act_asym != 0 selects the zero-point activation quantizer: q then holds UNSIGNED bytes, x_zero
 * [B*L] receives the zero points (it may be null otherwise) and acc is the sum over (q - z) * wq.
 * group > 0 selects per-block scales of `group` features for activations AND weights (symmetric codes only):
 * x_scale is then [B*L][K/group], w_scale [N][K/group], and acc is not produced (the integer partial sums are
 * scaled group by group).
 * Returns 0 on success.
 * ------------------------------------------------------------------------------------------ */
int oracle_stamp_linear(const float* X, const float* W, const float* bias, int B, int L, int K, int N,
                        int transform, int block, int levels, int k_hi, int bits_hi, int bits_lo,
                        int bits_w, double* T, float* x_scale, int8_t* q, float* w_scale, int8_t* wq,
                        int32_t* acc, double* Yt, double* Y, int grid_w, int act_asym, int32_t* x_zero, int group) {
  int n = block ? block : L;
  if (n <= 0 || L % n) return 1;
  long M = (long)B * L;
  int rc = 0;
  int own_T = 0, own_xs = 0, own_q = 0, own_ws = 0, own_wq = 0, own_acc = 0, own_Yt = 0, own_xz = 0;
  double* Lmat = NULL;
  int64_t* rp = NULL; int32_t* ci = NULL; double* cv = NULL;
  int32_t* bits = NULL;
  int use_csr = (transform == ORACLE_T_HAAR && n > 4096);

#define OWN(ptr, flag, type, count)                                   \
  if (!(ptr)) { ptr = (type*)malloc(sizeof(type) * (size_t)(count)); flag = 1; if (!(ptr)) { rc = 3; goto done; } }
  OWN(T, own_T, double, (size_t)M * K)
  if (group > 0 && (act_asym || K % group)) return 1;
  int ng = group > 0 ? K / group : 1;
  OWN(x_scale, own_xs, float, (size_t)M * ng)
  OWN(q, own_q, int8_t, (size_t)M * K)
  if (act_asym) { OWN(x_zero, own_xz, int32_t, M) }
  OWN(w_scale, own_ws, float, (size_t)N * ng)
  OWN(wq, own_wq, int8_t, (size_t)N * K)
  OWN(acc, own_acc, int32_t, (size_t)M * N)
  OWN(Yt, own_Yt, double, (size_t)M * N)
#undef OWN

  /* the explicit transform matrix */
  if (use_csr) {
    int lv = resolve_levels(transform, n, levels);
    if (lv < 0) { rc = 2; goto done; }
    rp = (int64_t*)malloc(sizeof(int64_t) * ((size_t)n + 1));
    ci = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * (lv + 1));
    cv = (double*)malloc(sizeof(double) * (size_t)n * (lv + 1));
    if (!rp || !ci || !cv) { rc = 3; goto done; }
    rc = oracle_haar_matrix_csr(n, levels, rp, ci, cv);
  } else {
    Lmat = (double*)malloc(sizeof(double) * (size_t)n * n);
    if (!Lmat) { rc = 3; goto done; }
    rc = (transform == ORACLE_T_HAAR2D) ? oracle_transform_matrix2d(n, grid_w, levels, Lmat)
                                        : oracle_transform_matrix(transform, n, levels, Lmat);
  }
  if (rc) goto done;

  /* X <- L X */
  rc = use_csr ? oracle_apply_csr_f32in(rp, ci, cv, n, X, B, L, K, T)
               : oracle_apply_dense_f32in(Lmat, n, X, B, L, K, T);
  if (rc) goto done;

  /* x_i <- Q(x_i; b_i) for every token */
  bits = (int32_t*)malloc(sizeof(int32_t) * (size_t)L);
  if (!bits) { rc = 3; goto done; }
  rc = oracle_bit_map(L, n, k_hi, bits_hi, bits_lo, bits);
  if (rc) goto done;
  rc = group > 0 ? oracle_quantize_rows_grouped(T, M, K, bits, L, group, x_scale, q)
       : act_asym ? oracle_quantize_rows_asym(T, M, K, bits, L, x_scale, x_zero, (uint8_t*)q)
                  : oracle_quantize_rows(T, M, K, bits, L, x_scale, q);
  if (rc) goto done;

  /* quantized weights (static; untouched by the sequence transform) */
  rc = group > 0 ? oracle_quantize_rows_grouped_f32in(W, N, K, bits_w, group, w_scale, wq)
                 : oracle_quantize_rows_f32in(W, N, K, bits_w, w_scale, wq);
  if (rc) goto done;

  /* Y <- X W^T on the integer codes, then de-quantize */
  if (group > 0) {
    rc = oracle_gemm_grouped(q, x_scale, wq, w_scale, M, N, K, group, Yt);
    if (rc) goto done;
  } else {
    rc = act_asym ? oracle_gemm_zp_i32((const uint8_t*)q, x_zero, wq, M, N, K, acc)
                  : oracle_gemm_i32(q, wq, M, N, K, acc);
    if (rc) goto done;
    rc = oracle_dequant(acc, x_scale, w_scale, M, N, Yt);
    if (rc) goto done;
  }

  /* Y <- L^{-1} Y  (= L^T Y), then Y <- Y + bias */
  if (Y) {
    rc = use_csr ? oracle_apply_csr_transpose_f64(rp, ci, cv, n, Yt, B, L, N, Y)
                 : oracle_apply_dense_f64(Lmat, n, 1, Yt, B, L, N, Y);
    if (rc) goto done;
    if (bias) {
#pragma omp parallel for schedule(static)
      for (long m = 0; m < M; ++m)
        for (int j = 0; j < N; ++j) Y[(size_t)m * N + j] += (double)bias[j];
    }
  }

done:
  free(Lmat); free(rp); free(ci); free(cv); free(bits);
  if (own_T) free(T);
  if (own_xs) free(x_scale);
  if (own_q) free(q);
  if (own_xz) free(x_zero);
  if (own_ws) free(w_scale);
  if (own_wq) free(wq);
  if (own_acc) free(acc);
  if (own_Yt) free(Yt);
  return rc;
}
