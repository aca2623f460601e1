/*
 * ROSAQ oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-file CPU restatement of what the ROSAQ hot path computes
 * (rotation-based saliency-aware weight quantization).  It exists only so that the
 * CUDA library can be checked against it.  It shares no code, headers, tables or
 * helpers with the CUDA path; only tests, the smoke check and the benchmark's
 * cpu-baseline leg may load it.
 *
 * Every function names the passage of the paper it follows.  Floating point is
 * fp64 except where the method itself fixes a precision (the fp32 rotate chain and
 * the fp32 round-to-nearest quantizer, whose integer results must be reproduced
 * bit for bit by any other implementation).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 *        (-mfma only makes fmaf() one instruction; its result is the same
 *        correctly rounded value either way).
 *
 * Parity status.  Pinned by identities / library routines / brute force in the
 * CPU tests: cov (Eq. 4), eigh_jacobi (Eq. 4), rotate_weights_f64 (Eq. 1),
 * scale_rows (scaling invariance), forward (Eq. 1, Eq. 3, Eq. 6 vs Eq. 7),
 * f16 conversions, pack/unpack.
 * The quantizer's free constants (range floor 1e-5, zero-point clamp, tie rule,
 * scale rounded to fp16 before the codes are taken), the bit layout of the packed
 * words, the fp32 summation order of rotate_weights_f32 and the choice of the
 * diagonal D of the scaled (AWQ-style) variant are NOT fixed by the
 * paper: for those this file is the definition ("parity unpinned" by the paper);
 * the tests pin their internal consistency (grid round trip, error bound,
 * bijection) only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* IEEE binary16 <-> binary32, written out from the format definition.        */
/* ------------------------------------------------------------------------- */

/* binary16 bits -> exact double value (inf/nan preserved). */
static double f16_bits_to_double(uint16_t h) {
  int sign = (h >> 15) & 1;
  int e = (h >> 10) & 0x1f;
  int m = h & 0x3ff;
  double v;
  if (e == 0)
    v = ldexp((double)m, -24); /* subnormal: m * 2^-24 */
  else if (e == 31)
    v = m ? NAN : INFINITY;
  else
    v = ldexp((double)(1024 + m), e - 25); /* (1 + m/1024) * 2^(e-15) */
  return sign ? -v : v;
}

/* fp32 -> binary16 bits, round to nearest, ties to even.  Overflow goes to inf,
 * subnormals are kept.  Uses only exact scalings and nearbyint() in the default
 * (ties-to-even) rounding mode. */
static uint16_t f32_to_f16_bits(float f) {
  uint16_t sign = signbit(f) ? 0x8000 : 0;
  double a = fabs((double)f);
  if (isnan(f)) return (uint16_t)(sign | 0x7e00);
  if (isinf(f)) return (uint16_t)(sign | 0x7c00);
  if (a == 0.0) return sign;
  int ex;
  (void)frexp(a, &ex); /* a = frac * 2^ex, frac in [0.5,1) => a in [2^(ex-1), 2^ex) */
  int e = ex - 1;      /* floor(log2 a) */
  if (e < -14) {
    /* subnormal range: unit is 2^-24 */
    double m = nearbyint(ldexp(a, 24));
    return (uint16_t)(sign | (uint16_t)m); /* m == 1024 is exactly the smallest normal */
  }
  double m = nearbyint(ldexp(a, 10 - e)); /* in [1024, 2048] */
  if (m == 2048.0) {
    m = 1024.0;
    e += 1;
  }
  if (e > 15) return (uint16_t)(sign | 0x7c00);
  return (uint16_t)(sign | ((uint16_t)(e + 15) << 10) | ((uint16_t)m - 1024));
}

void oracle_f16_to_f64(const uint16_t *h, int64_t n, double *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f16_bits_to_double(h[i]);
}

void oracle_f32_to_f16(const float *f, int64_t n, uint16_t *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f32_to_f16_bits(f[i]);
}

/* ------------------------------------------------------------------------- */
/* Eq. 4, left side: the calibration Gram matrix  C = X^T X.                   */
/* No centring and no 1/N: the equation has neither.                           */
/* Head-wise (Section 3.1.1): n_blocks independent Grams of the column slices   */
/* [h*dh, (h+1)*dh); C is [n_blocks][dh][dh].                                  */
/* ------------------------------------------------------------------------- */
void oracle_cov(const double *X, int64_t n_tokens, int d, int n_blocks, double *C) {
  int dh = d / n_blocks;
#pragma omp parallel for schedule(static)
  for (int bi = 0; bi < n_blocks * dh; ++bi) {
    int b = bi / dh, i = bi % dh;
    for (int j = 0; j < dh; ++j) {
      double acc = 0.0;
      for (int64_t t = 0; t < n_tokens; ++t)
        acc += X[t * d + b * dh + i] * X[t * d + b * dh + j];
      C[((int64_t)b * dh + i) * dh + j] = acc;
    }
  }
}

/* ------------------------------------------------------------------------- */
/* Eq. 4, right side: C = R Lambda R^T by the cyclic Jacobi method (textbook).  */
/* On return lambda[0..d) is sorted in DESCENDING order (Section 3.2: the larger */
/* eigenvalues are the salient ones), ties keep their original index order;     */
/* V[:, j] (row-major V[i*d+j]) is the unit eigenvector of lambda[j], with its   */
/* largest-magnitude entry (lowest index on ties) made positive.                */
/* Returns the number of sweeps used, or -1 if 100 sweeps did not converge.      */
/* ------------------------------------------------------------------------- */
static double off_norm2(const double *A, int d) {
  double s = 0.0;
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j)
      if (i != j) s += A[(int64_t)i * d + j] * A[(int64_t)i * d + j];
  return s;
}

int oracle_eigh_jacobi(const double *C, int d, double *lambda, double *V) {
  int64_t dd = (int64_t)d * d;
  double *A = (double *)malloc(sizeof(double) * dd);
  double *U = (double *)malloc(sizeof(double) * dd);
  memcpy(A, C, sizeof(double) * dd);
  /* symmetrise the input exactly once: A = (C + C^T)/2 */
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < i; ++j) {
      double m = 0.5 * (A[(int64_t)i * d + j] + A[(int64_t)j * d + i]);
      A[(int64_t)i * d + j] = m;
      A[(int64_t)j * d + i] = m;
    }
  for (int64_t i = 0; i < dd; ++i) U[i] = 0.0;
  for (int i = 0; i < d; ++i) U[(int64_t)i * d + i] = 1.0;

  double fro2 = 0.0;
  for (int64_t i = 0; i < dd; ++i) fro2 += A[i] * A[i];
  int sweeps = 0, converged = (fro2 == 0.0);
  while (!converged && sweeps < 100) {
    ++sweeps;
    for (int p = 0; p < d - 1; ++p) {
      for (int q = p + 1; q < d; ++q) {
        double apq = A[(int64_t)p * d + q];
        if (apq == 0.0) continue;
        double app = A[(int64_t)p * d + p], aqq = A[(int64_t)q * d + q];
        /* rotation angle that zeroes A[p][q]:  tan(2 phi) = 2 apq / (aqq - app) */
        double theta = (aqq - app) / (2.0 * apq);
        double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
        double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
        /* A <- J^T A J with J = [[c, s], [-s, c]] on the (p,q) plane */
        for (int k = 0; k < d; ++k) { /* columns p and q */
          double akp = A[(int64_t)k * d + p], akq = A[(int64_t)k * d + q];
          A[(int64_t)k * d + p] = c * akp - s * akq;
          A[(int64_t)k * d + q] = s * akp + c * akq;
        }
        for (int k = 0; k < d; ++k) { /* rows p and q */
          double apk = A[(int64_t)p * d + k], aqk = A[(int64_t)q * d + k];
          A[(int64_t)p * d + k] = c * apk - s * aqk;
          A[(int64_t)q * d + k] = s * apk + c * aqk;
        }
        for (int k = 0; k < d; ++k) { /* U <- U J accumulates the eigenvectors */
          double ukp = U[(int64_t)k * d + p], ukq = U[(int64_t)k * d + q];
          U[(int64_t)k * d + p] = c * ukp - s * ukq;
          U[(int64_t)k * d + q] = s * ukp + c * ukq;
        }
      }
    }
    converged = sqrt(off_norm2(A, d)) <= 1e-14 * sqrt(fro2);
  }

  /* stable descending sort of the diagonal (insertion sort on an index array) */
  int *idx = (int *)malloc(sizeof(int) * d);
  for (int i = 0; i < d; ++i) idx[i] = i;
  for (int i = 1; i < d; ++i) {
    int v = idx[i], j = i - 1;
    while (j >= 0 && A[(int64_t)idx[j] * d + idx[j]] < A[(int64_t)v * d + v]) {
      idx[j + 1] = idx[j];
      --j;
    }
    idx[j + 1] = v;
  }
  for (int j = 0; j < d; ++j) {
    int src = idx[j];
    lambda[j] = A[(int64_t)src * d + src];
    double nrm = 0.0, big = 0.0;
    int bigi = 0;
    for (int i = 0; i < d; ++i) {
      double u = U[(int64_t)i * d + src];
      nrm += u * u;
      if (fabs(u) > big) {
        big = fabs(u);
        bigi = i;
      }
    }
    nrm = sqrt(nrm);
    double sgn = (U[(int64_t)bigi * d + src] < 0.0) ? -1.0 : 1.0;
    for (int i = 0; i < d; ++i) V[(int64_t)i * d + j] = sgn * U[(int64_t)i * d + src] / nrm;
  }
  free(idx);
  free(A);
  free(U);
  return converged ? sweeps : -1;
}

/* ------------------------------------------------------------------------- */
/* Eq. 1 / Eq. 3 / Eq. 6: the rotated weight  W' = R^T W.                       */
/*                                                                             */
/* R is given as n_blocks square blocks Rb[h] (dh x dh, row-major) on the        */
/* diagonal, followed by an optional column permutation: column j of R is        */
/* column perm[j] of blockdiag(Rb) (perm == NULL: identity).  n_blocks == 1 is   */
/* the layer-wise dense rotation; n_blocks == H is the head-wise one of Eq. 6.   */
/* So  W'[j][n] = sum_k Rb[h][k][c] * W[h*dh + k][n]  with p = perm[j],          */
/* h = p / dh, c = p % dh, k over the block's dh rows only.                      */
/*                                                                             */
/* Only the output columns listed in cols[0..n_cols) are produced:               */
/* out is [d_in][n_cols].                                                       */
/* ------------------------------------------------------------------------- */

/* fp64 version, for the identity checks. */
void oracle_rotate_weights_f64(const double *Rb, int d_in, int n_blocks, const int32_t *perm,
                               const double *W, int d_out, const int32_t *cols, int n_cols,
                               double *out) {
  int dh = d_in / n_blocks;
#pragma omp parallel for schedule(static)
  for (int j = 0; j < d_in; ++j) {
    int p = perm ? perm[j] : j;
    int h = p / dh, c = p % dh;
    const double *R = Rb + (int64_t)h * dh * dh;
    for (int ci = 0; ci < n_cols; ++ci) {
      int n = cols[ci];
      double acc = 0.0;
      for (int k = 0; k < dh; ++k) acc += R[(int64_t)k * dh + c] * W[((int64_t)h * dh + k) * d_out + n];
      out[(int64_t)j * n_cols + ci] = acc;
    }
  }
}

/* The canonical fp32 chain whose result defines the integer codes: one fused
 * multiply-add per term, k ascending, a single accumulator started at +0, no
 * blocking and no reassociation.  Wc holds the needed columns of W in fp32:
 * Wc[k][ci]. */
static void rotate_chain_f32(const float *Rb, int d_in, int n_blocks, const int32_t *perm,
                             const float *Wc, int n_cols, float *out) {
  int dh = d_in / n_blocks;
#pragma omp parallel for schedule(static)
  for (int j = 0; j < d_in; ++j) {
    int p = perm ? perm[j] : j;
    int h = p / dh, c = p % dh;
    const float *R = Rb + (int64_t)h * dh * dh;
    for (int ci = 0; ci < n_cols; ++ci) {
      float acc = 0.0f;
      for (int k = 0; k < dh; ++k)
        acc = fmaf(R[(int64_t)k * dh + c], Wc[((int64_t)h * dh + k) * n_cols + ci], acc);
      out[(int64_t)j * n_cols + ci] = acc;
    }
  }
}

/* R is fp32, W is binary16 (widened exactly). */
void oracle_rotate_weights_f32(const float *Rb, int d_in, int n_blocks, const int32_t *perm,
                               const uint16_t *W16, int d_out, const int32_t *cols, int n_cols,
                               float *out) {
  float *Wc = (float *)malloc(sizeof(float) * (size_t)d_in * n_cols);
  for (int k = 0; k < d_in; ++k)
    for (int ci = 0; ci < n_cols; ++ci)
      Wc[(int64_t)k * n_cols + ci] = (float)f16_bits_to_double(W16[(int64_t)k * d_out + cols[ci]]);
  rotate_chain_f32(Rb, d_in, n_blocks, perm, Wc, n_cols, out);
  free(Wc);
}

/* The same chain on a weight that is already fp32 (the scaled weight D W below). */
void oracle_rotate_weights_f32_w32(const float *Rb, int d_in, int n_blocks, const int32_t *perm,
                                   const float *W32, int d_out, const int32_t *cols, int n_cols,
                                   float *out) {
  float *Wc = (float *)malloc(sizeof(float) * (size_t)d_in * n_cols);
  for (int k = 0; k < d_in; ++k)
    for (int ci = 0; ci < n_cols; ++ci) Wc[(int64_t)k * n_cols + ci] = W32[(int64_t)k * d_out + cols[ci]];
  rotate_chain_f32(Rb, d_in, n_blocks, perm, Wc, n_cols, out);
  free(Wc);
}

/* ------------------------------------------------------------------------- */
/* Scaling invariance (appendix on rotational and scaling invariance):          */
/*   X W = (X D^-1)(D W)  for an invertible diagonal D, so a linear layer may    */
/* quantize D W and be fed X D^-1.  The weight-splitting appendix uses this      */
/* (AWQ-style per-input-channel scaling) for the down projection W_D, which it   */
/* does not rotate.  The paper prints no rule for D: D is an input here.         */
/*   out[i][n] = d[i] * W[i][n]                                                  */
/* fp64 for the identity checks; fp32 (binary16 weight widened exactly, one      */
/* rounding per product) for the version the integer codes are taken from.       */
/* ------------------------------------------------------------------------- */
void oracle_scale_rows_f64(const double *W, int d_in, int d_out, const double *d, double *out) {
  for (int i = 0; i < d_in; ++i)
    for (int n = 0; n < d_out; ++n) out[(int64_t)i * d_out + n] = d[i] * W[(int64_t)i * d_out + n];
}

void oracle_scale_rows_f32(const uint16_t *W16, int d_in, int d_out, const float *d, float *out) {
  for (int i = 0; i < d_in; ++i)
    for (int n = 0; n < d_out; ++n)
      out[(int64_t)i * d_out + n] = d[i] * (float)f16_bits_to_double(W16[(int64_t)i * d_out + n]);
}

/* ------------------------------------------------------------------------- */
/* Eq. 3 and Section 3.3: the mixed-precision split of W' (here [d_in][n_cols]  */
/* fp32).  Rows [0, k_salient) are the salient channels and are kept in         */
/* binary16.  The remaining rows are quantized per group of `group` consecutive */
/* input channels and per output column with asymmetric min/max                */
/* round-to-nearest to `bits` bits -- the paper names per-group INT3/INT4 with   */
/* groups of 128 channels but prints no formula; this is the plain one:         */
/*   qmax = 2^bits - 1                                                         */
/*   s = fp16( max(hi - lo, 1e-5) / qmax )   (0 -> smallest subnormal,          */
/*                                            inf -> 65504)                    */
/*   z = clamp(-rint(lo / s), 0, qmax)                                         */
/*   q = clamp(rint(w / s) + z, 0, qmax)                                       */
/* all in IEEE fp32 with round-to-nearest-even; the stored (rounded) scale is   */
/* the one the codes are taken with.  Dequantised value = (q - z) * s.          */
/* Outputs: salient [k_salient][n_cols] f16 bits, scales / zeros                */
/* [(d_in-k_salient)/group][n_cols] f16 bits, codes [d_in-k_salient][n_cols].   */
/* ------------------------------------------------------------------------- */
void oracle_quantize(const float *Wp, int d_in, int n_cols, int bits, int group, int k_salient,
                     uint16_t *salient, uint16_t *scales, uint16_t *zeros, uint8_t *codes) {
  const float qmax = (float)((1 << bits) - 1);
  for (int i = 0; i < k_salient; ++i)
    for (int n = 0; n < n_cols; ++n)
      salient[(int64_t)i * n_cols + n] = f32_to_f16_bits(Wp[(int64_t)i * n_cols + n]);
  int n_groups = (d_in - k_salient) / group;
  for (int g = 0; g < n_groups; ++g) {
    const float *Wg = Wp + ((int64_t)k_salient + (int64_t)g * group) * n_cols;
    for (int n = 0; n < n_cols; ++n) {
      float lo = Wg[n], hi = Wg[n];
      for (int r = 1; r < group; ++r) {
        float w = Wg[(int64_t)r * n_cols + n];
        if (w < lo) lo = w;
        if (w > hi) hi = w;
      }
      float range = hi - lo;
      if (range < 1e-5f) range = 1e-5f;
      float s32 = range / qmax;
      uint16_t sb = f32_to_f16_bits(s32);
      if (sb == 0x0000) sb = 0x0001;
      if (sb == 0x7c00) sb = 0x7bff;
      float sf = (float)f16_bits_to_double(sb);
      float z = -rintf(lo / sf);
      if (z <= 0.0f) z = 0.0f; /* also turns -0 (lo == +0) into +0 */
      if (z > qmax) z = qmax;
      scales[(int64_t)g * n_cols + n] = sb;
      zeros[(int64_t)g * n_cols + n] = f32_to_f16_bits(z); /* small integer: exact */
      for (int r = 0; r < group; ++r) {
        float q = rintf(Wg[(int64_t)r * n_cols + n] / sf) + z;
        if (q < 0.0f) q = 0.0f;
        if (q > qmax) q = qmax;
        codes[((int64_t)g * group + r) * n_cols + n] = (uint8_t)q;
      }
    }
  }
}

/* ------------------------------------------------------------------------- */
/* The packed-code container (interchange layout; the paper is silent on it).   */
/* r = row index inside the non-salient part.                                  */
/* INT4: word qw[r/8][n], code of row r in bits [4*(r%8), +4).                  */
/* INT3: rows in blocks of 32; a block is the 96-bit little-endian string made  */
/*       of words qw[3*(r/32)+0..2][n]; code of row r sits in bits              */
/*       [3*(r%32), +3) of that string (rows 10 and 21 straddle two words).      */
/* ------------------------------------------------------------------------- */
void oracle_pack(const uint8_t *codes, int n_rows, int n_cols, int bits, uint32_t *qw) {
  int64_t n_words = (bits == 4) ? (int64_t)n_rows / 8 : (int64_t)n_rows / 32 * 3;
  memset(qw, 0, sizeof(uint32_t) * n_words * n_cols);
  for (int r = 0; r < n_rows; ++r)
    for (int n = 0; n < n_cols; ++n) {
      uint32_t q = codes[(int64_t)r * n_cols + n];
      if (bits == 4) {
        qw[(int64_t)(r / 8) * n_cols + n] |= q << (4 * (r % 8));
      } else {
        int bit = 3 * (r % 32); /* position in the 96-bit string */
        for (int b = 0; b < 3; ++b, ++bit)
          qw[((int64_t)(r / 32) * 3 + bit / 32) * n_cols + n] |= ((q >> b) & 1u) << (bit % 32);
      }
    }
}

void oracle_unpack(const uint32_t *qw, int n_rows, int n_cols, int bits, uint8_t *codes) {
  for (int r = 0; r < n_rows; ++r)
    for (int n = 0; n < n_cols; ++n) {
      uint32_t q = 0;
      if (bits == 4) {
        q = (qw[(int64_t)(r / 8) * n_cols + n] >> (4 * (r % 8))) & 0xf;
      } else {
        int bit = 3 * (r % 32);
        for (int b = 0; b < 3; ++b, ++bit)
          q |= ((qw[((int64_t)(r / 32) * 3 + bit / 32) * n_cols + n] >> (bit % 32)) & 1u) << b;
      }
      codes[(int64_t)r * n_cols + n] = (uint8_t)q;
    }
}

/* ------------------------------------------------------------------------- */
/* Eq. 3 (Eq. 6 when n_blocks > 1): the forward reference in fp64.              */
/*   x'  = (x . blockdiag(Rb))[:, perm]      (Rb == NULL: x is already rotated)  */
/*   W^[i][n] = salient[i][n]                      for i <  k_salient           */
/*            = (code - zero_g) * scale_g          for i >= k_salient           */
/*   y = x' . W^                                                               */
/* x and Rb hold the binary16 values widened exactly to fp64 by the caller;     */
/* nothing is rounded in between.  All weight-side arrays are [..][n_cols].      */
/* xrot_out (optional) receives x' [M][d_in].                                   */
/* ------------------------------------------------------------------------- */
void oracle_forward(const double *x, int M, int d_in, const double *Rb, int n_blocks,
                    const int32_t *perm, const uint16_t *salient, const uint16_t *scales,
                    const uint16_t *zeros, const uint8_t *codes, int bits, int group,
                    int k_salient, int n_cols, double *y, double *xrot_out) {
  (void)bits;
  double *xr = (double *)malloc(sizeof(double) * (size_t)M * d_in);
  if (Rb) {
    int dh = d_in / n_blocks;
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d_in; ++j) {
      int p = perm ? perm[j] : j;
      int h = p / dh, c = p % dh;
      const double *R = Rb + (int64_t)h * dh * dh;
      for (int m = 0; m < M; ++m) {
        double acc = 0.0;
        for (int k = 0; k < dh; ++k) acc += x[(int64_t)m * d_in + h * dh + k] * R[(int64_t)k * dh + c];
        xr[(int64_t)m * d_in + j] = acc;
      }
    }
  } else {
    memcpy(xr, x, sizeof(double) * (size_t)M * d_in);
  }
  if (xrot_out) memcpy(xrot_out, xr, sizeof(double) * (size_t)M * d_in);
#pragma omp parallel for schedule(static)
  for (int n = 0; n < n_cols; ++n) {
    double *wh = (double *)malloc(sizeof(double) * (size_t)d_in); /* column n of W^ */
    for (int i = 0; i < d_in; ++i) {
      if (i < k_salient) {
        wh[i] = f16_bits_to_double(salient[(int64_t)i * n_cols + n]);
      } else {
        int r = i - k_salient, g = r / group;
        double q = (double)codes[(int64_t)r * n_cols + n];
        double z = f16_bits_to_double(zeros[(int64_t)g * n_cols + n]);
        double s = f16_bits_to_double(scales[(int64_t)g * n_cols + n]);
        wh[i] = (q - z) * s;
      }
    }
    for (int m = 0; m < M; ++m) {
      double acc = 0.0;
      for (int i = 0; i < d_in; ++i) acc += xr[(int64_t)m * d_in + i] * wh[i];
      y[(int64_t)m * n_cols + n] = acc;
    }
    free(wh);
  }
  free(xr);
}

int oracle_num_threads(void) {
  int n = 1;
#pragma omp parallel
  {
#pragma omp single
    n =
#ifdef _OPENMP
        omp_get_num_threads();
#else
        1;
#endif
  }
  return n;
}
