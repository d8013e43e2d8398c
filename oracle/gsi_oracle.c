/*
 * Plain fp64 CPU oracle for the gated subspace linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or
 * import this file; it exists so that the CUDA library can be checked against
 * an independent, slow, obviously-correct restatement of the method.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * Notation (paper -> this file):
 *   V_k  (rank-k activation basis, d x k)          -> P   [d][k] row-major
 *   M = W V_k (cached image, d_out x k)            -> M   [o][k] row-major
 *   g = V_k^T x (coefficients)                     -> g   [k]
 *   r = x - V_k g (residual)                       -> r   [d]
 *   rho = ||r|| / ||x|| (residual ratio)           -> rho
 *   "slow path" / "gated" / "fired" token          -> gate byte 1
 *
 * Every step is the literal definition, in double precision, on exactly the
 * stored input values (bf16 weights and basis, fp32 activations; each widens
 * to double without rounding).  There is no blocking, fusion or reordering.
 *
 * Pinning: see tests/test_oracle_pins.py.  Every function below is pinned by
 * special cases that reduce to a library mat-vec, by the exact identity of
 * Eq. (3.2), by the bound of Theorem 3.1, by the monotonicity of
 * Proposition 2.3 and by brute force in rational arithmetic on tiny shapes;
 * the online basis extension by a library QR, by the orthogonality its second
 * pass restores, and by its special cases (empty, full, in-span).
 * What the paper measures on real model activations (gate rates, perplexity;
 * Tables 4-9) has no counterpart here: parity unpinned for those, they are out
 * of scope.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define GSI_ORACLE_BF16 0
#define GSI_ORACLE_F32 1

/* A bf16 value is the upper 16 bits of an IEEE fp32 value. */
static double bf16_bits_to_f64(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* Element (i, j) of the stored basis, widened exactly. */
static double basis_at(const void* P, int p_dtype, size_t idx) {
  if (p_dtype == GSI_ORACLE_F32) return (double)((const float*)P)[idx];
  return bf16_bits_to_f64(((const uint16_t*)P)[idx]);
}

int gsi_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void gsi_oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* Widen a bf16 array to double (used by tests to hand the same stored values
 * to numpy). */
void gsi_oracle_bf16_to_f64(const uint16_t* src, size_t n, double* dst) {
  for (size_t i = 0; i < n; ++i) dst[i] = bf16_bits_to_f64(src[i]);
}

/*
 * Round a double to the nearest bf16 (ties to even), returned as bits.
 * Diagnostic only: it lets a test separate "the stored image is rounded to
 * bf16" (Section 4.2: images are kept in BF16) from kernel error.  Done in two
 * exact steps: double -> nearest-even at 8 significant bits, by integer
 * arithmetic on the double's own bit pattern (no intermediate fp32 rounding).
 */
uint16_t gsi_oracle_f64_to_bf16_rne(double v) {
  if (v != v) return 0x7FC0;
  uint16_t sign = signbit(v) ? 0x8000 : 0;
  double a = fabs(v);
  if (a == 0.0) return sign;
  if (isinf(a)) return (uint16_t)(sign | 0x7F80);
  int e;
  (void)frexp(a, &e); /* a = m * 2^e, m in [0.5, 1)  =>  a in [2^(e-1), 2^e) */
  int E = e - 1;
  if (E < -126) E = -126; /* subnormals share the spacing of the lowest binade */
  /* bf16 numbers in this binade are spaced 2^(E-7) apart (7 fraction bits);
   * scaling by a power of two is exact. */
  double scaled = ldexp(a, 7 - E);
  double fl = floor(scaled);
  double rem = scaled - fl;
  uint64_t q = (uint64_t)fl;
  if (rem > 0.5 || (rem == 0.5 && (q & 1))) q += 1;
  if (q >= 256) { /* rounding carried into the next binade */
    q = 128;
    E += 1;
  }
  uint32_t bits;
  if (q >= 128) { /* normal: hidden bit set */
    int biased = E + 127;
    if (biased >= 255) return (uint16_t)(sign | 0x7F80);
    bits = ((uint32_t)biased << 7) | (uint32_t)(q - 128);
  } else {
    bits = (uint32_t)q; /* subnormal: biased exponent 0 */
  }
  return (uint16_t)(sign | bits);
}

void gsi_oracle_f64_to_bf16_rne_array(const double* src, size_t n, uint16_t* dst) {
  for (size_t i = 0; i < n; ++i) dst[i] = gsi_oracle_f64_to_bf16_rne(src[i]);
}

/*
 * Cached image, Eq. (3.2) and Section 4.2:  M = W V_k,
 *   M[a][j] = sum_i W[a][i] * P[i][j],   a < o, j < k,
 * in double, NOT rounded to bf16.
 * W: [o][d] bf16 bits.  P: [d][k] of p_dtype.  M: [o][k] double (out).
 */
int gsi_oracle_image(const uint16_t* W, const void* P, int p_dtype, int o, int d,
                     int k, double* M) {
  if (!W || !P || !M || o < 0 || d <= 0 || k <= 0) return 1;
#pragma omp parallel for schedule(static)
  for (int a = 0; a < o; ++a) {
    double* Ma = M + (size_t)a * k;
    for (int j = 0; j < k; ++j) Ma[j] = 0.0;
    for (int i = 0; i < d; ++i) {
      double w = bf16_bits_to_f64(W[(size_t)a * d + i]);
      for (int j = 0; j < k; ++j) Ma[j] += w * basis_at(P, p_dtype, (size_t)i * k + j);
    }
  }
  return 0;
}

/*
 * Steps 1-3 of Algorithm 1 plus the gate test of Section 3.2, per token t:
 *   g   = V_k^T x                      (Algorithm 1, line 1)
 *   r   = x - V_k g                    (line 2; explicit, Eq. (3.1))
 *   rho = ||r||_2 / ||x||_2            (line 3; Eq. (3.3))
 *   fast path iff rho < eps            (line 4; strict, as in Definition 2.2)
 * The comparison is taken in the division-free form ||r|| < eps * ||x|| so
 * that x = 0 (rho = 0/0) is well defined: 0 < 0 is false, the token fires.
 * eps is the caller's float widened to double.
 * gate[t] = 1 for a slow-path (fired) token, 0 for a fast-path token.
 * x: [T][d] fp32.  Outputs (any may be NULL): g [T][k], r [T][d], rho [T],
 * norm_x [T], norm_r [T], gate [T].
 */
int gsi_oracle_project(const float* x, int T, const void* P, int p_dtype, int d,
                       int k, float eps, double* g, double* r, double* rho,
                       double* norm_x, double* norm_r, uint8_t* gate) {
  if (!x || !P || T < 0 || d <= 0 || k <= 0) return 1;
  const double eps_d = (double)eps;
  int bad = 0;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float* xt = x + (size_t)t * d;
    double* gt = (double*)malloc((size_t)k * sizeof(double));
    if (!gt) {
#pragma omp atomic write
      bad = 1;
      continue;
    }
    for (int j = 0; j < k; ++j) {
      double s = 0.0;
      for (int i = 0; i < d; ++i) s += basis_at(P, p_dtype, (size_t)i * k + j) * (double)xt[i];
      gt[j] = s;
    }
    double sx = 0.0, sr = 0.0;
    for (int i = 0; i < d; ++i) {
      double pg = 0.0;
      for (int j = 0; j < k; ++j) pg += basis_at(P, p_dtype, (size_t)i * k + j) * gt[j];
      double ri = (double)xt[i] - pg;
      if (r) r[(size_t)t * d + i] = ri;
      sx += (double)xt[i] * (double)xt[i];
      sr += ri * ri;
    }
    double nx = sqrt(sx), nr = sqrt(sr);
    int fast = (nr < eps_d * nx);
    if (g)
      for (int j = 0; j < k; ++j) g[(size_t)t * k + j] = gt[j];
    if (rho) rho[t] = nr / nx;
    if (norm_x) norm_x[t] = nx;
    if (norm_r) norm_r[t] = nr;
    if (gate) gate[t] = fast ? 0 : 1;
    free(gt);
  }
  return bad;
}

/*
 * Output of one linear map for T tokens, given g, r and the gate bytes:
 *   y     = M g                 for every token          (Algorithm 1, line 5)
 *   y    += W r                 for tokens with gate = 1 (Eq. (3.2): y = M g + W r)
 *   y_alt = gate ? W x : M g    Algorithm 1 read literally (lines 5 and 7)
 * The two forms agree exactly in real arithmetic; a test checks that they
 * agree to rounding here.  The gate bytes are an INPUT so that a test can
 * evaluate the method with a given decision for tokens whose rho sits on the
 * threshold.
 * M: [o][k] double.  W: [o][d] bf16 bits.  g: [T][k].  r: [T][d].  x: [T][d].
 * y, y_alt: [T][o] double (y_alt and x may be NULL together).
 */
int gsi_oracle_map(const double* M, const uint16_t* W, const double* g,
                   const double* r, const float* x, const uint8_t* gate, int T,
                   int o, int d, int k, double* y, double* y_alt) {
  if (!M || !W || !g || !r || !gate || !y || T < 0 || o < 0 || d <= 0 || k <= 0) return 1;
  if (y_alt && !x) return 1;
#pragma omp parallel for schedule(static)
  for (int a = 0; a < o; ++a) {
    const double* Ma = M + (size_t)a * k;
    const uint16_t* Wa = W + (size_t)a * d;
    for (int t = 0; t < T; ++t) {
      double mg = 0.0;
      for (int j = 0; j < k; ++j) mg += Ma[j] * g[(size_t)t * k + j];
      double yv = mg;
      if (gate[t]) {
        double wr = 0.0;
        for (int i = 0; i < d; ++i) wr += bf16_bits_to_f64(Wa[i]) * r[(size_t)t * d + i];
        yv += wr;
      }
      y[(size_t)t * o + a] = yv;
      if (y_alt) {
        if (gate[t]) {
          double wx = 0.0;
          for (int i = 0; i < d; ++i)
            wx += bf16_bits_to_f64(Wa[i]) * (double)x[(size_t)t * d + i];
          y_alt[(size_t)t * o + a] = wx;
        } else {
          y_alt[(size_t)t * o + a] = mg;
        }
      }
    }
  }
  return 0;
}

/*
 * Online extension of the basis by one vector (the paper's "time-dimension
 * tracking" of Section 5.4 and "online basis adaptation" of Section 7.2):
 * a token x is tested against the current basis, and if
 *     rho = ||x - V V^T x|| / ||x||
 * exceeds the threshold tau the basis is extended by one orthonormal vector.
 * The vector is the residual orthogonalised against V TWICE and normalised
 * (classical Gram-Schmidt with one re-orthogonalisation, the "DGKS" update):
 *     r1 = x  - V (V^T x),   r2 = r1 - V (V^T r1),   v = r2 / ||r2||.
 * The paper gives no further detail; readings taken here: the test uses the
 * first-pass residual (the formula the paper prints, the same rho the layer's
 * gate uses); nothing is appended when the basis is full or r2 vanishes.
 *
 * P: [d][k_cap] stored basis of which columns [0, k_act) are in use.
 * x: [d] double.  Outputs: *rho_out; v_out [d] (unit vector, unrounded; written
 * only when the function returns 1).  Returns 1 = extended, 0 = not, -1 = bad
 * arguments.
 */
int gsi_oracle_extend(const void* P, int p_dtype, int d, int k_cap, int k_act,
                      const double* x, double tau, double* rho_out, double* v_out) {
  if (!P || !x || !rho_out || !v_out || d <= 0 || k_cap <= 0 || k_act < 0 || k_act > k_cap)
    return -1;
  double* r = (double*)malloc((size_t)d * sizeof(double));
  double* g = (double*)malloc((size_t)(k_act > 0 ? k_act : 1) * sizeof(double));
  if (!r || !g) {
    free(r);
    free(g);
    return -1;
  }
  double sx = 0.0;
  for (int i = 0; i < d; ++i) {
    r[i] = x[i];
    sx += x[i] * x[i];
  }
  double rho = 0.0;
  for (int pass = 0; pass < 2; ++pass) {
    for (int j = 0; j < k_act; ++j) {
      double s = 0.0;
      for (int i = 0; i < d; ++i) s += basis_at(P, p_dtype, (size_t)i * k_cap + j) * r[i];
      g[j] = s;
    }
    double sr = 0.0;
    for (int i = 0; i < d; ++i) {
      double pg = 0.0;
      for (int j = 0; j < k_act; ++j) pg += basis_at(P, p_dtype, (size_t)i * k_cap + j) * g[j];
      r[i] -= pg;
      sr += r[i] * r[i];
    }
    if (pass == 0) rho = sqrt(sr) / sqrt(sx);
  }
  *rho_out = rho;
  double s2 = 0.0;
  for (int i = 0; i < d; ++i) s2 += r[i] * r[i];
  int extended = 0;
  if (rho > tau && k_act < k_cap && s2 > 0.0) {
    const double inv = 1.0 / sqrt(s2);
    for (int i = 0; i < d; ++i) v_out[i] = r[i] * inv;
    extended = 1;
  }
  free(r);
  free(g);
  return extended;
}

/* ------------------------------------------------------------------------ *
 * FP8 storage of the cached image (Section 7.4: the image M = W V_k kept in
 * FP8 halves the fast-path read volume).  The paper names no format, scaling
 * or rounding; this reading is the common one: E4M3 codes (1 sign, 4 exponent
 * bits with bias 7, 3 fraction bits; no infinities, S.1111.111 is NaN, largest
 * finite value 448; exponent field 0 holds the subnormals m/8 * 2^-6), one
 * fp32 scale per output row chosen so that the row's largest magnitude maps to
 * 448, round to nearest with ties to the even code, saturating.
 * ------------------------------------------------------------------------ */

/* Value of an E4M3 code, from the definition of the format. */
double gsi_oracle_e4m3_decode(uint8_t code) {
  int s = code >> 7, e = (code >> 3) & 0xF, m = code & 7;
  if (e == 15 && m == 7) return NAN;
  double v = e == 0 ? ldexp((double)m / 8.0, -6) : ldexp(1.0 + (double)m / 8.0, e - 7);
  return s ? -v : v;
}

/*
 * Nearest E4M3 code of a float (ties to the even code), saturating at +-448;
 * NaN gives the NaN code.  By exact arithmetic: within the binade 2^E the
 * codes are spaced 2^(E-3) apart (E >= -6; below, the subnormal spacing 2^-9).
 */
uint8_t gsi_oracle_f32_to_e4m3_rne_sat(float vf) {
  double v = (double)vf;
  if (v != v) return 0x7F;
  uint8_t sign = signbit(v) ? 0x80 : 0;
  double a = fabs(v);
  if (a >= 448.0) return (uint8_t)(sign | 0x7E); /* also +-inf: saturating */
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);
  int E = e - 1;
  if (E < -6) E = -6;
  double scaled = ldexp(a, 3 - E); /* in units of the spacing: [8, 16) for normals, [0, 8) below */
  double fl = floor(scaled);
  double rem = scaled - fl;
  unsigned q = (unsigned)fl;
  if (rem > 0.5 || (rem == 0.5 && (q & 1))) q += 1;
  if (q >= 16) { /* carried into the next binade */
    q = 8;
    E += 1;
  }
  unsigned bits;
  if (q >= 8) {
    bits = ((unsigned)(E + 7) << 3) | (q - 8);
    if (bits > 0x7E) bits = 0x7E; /* 464 and above round past the largest code */
  } else {
    bits = q;
  }
  return (uint8_t)(sign | bits);
}

void gsi_oracle_e4m3_decode_array(const uint8_t* src, size_t n, double* dst) {
  for (size_t i = 0; i < n; ++i) dst[i] = gsi_oracle_e4m3_decode(src[i]);
}
void gsi_oracle_f32_to_e4m3_array(const float* src, size_t n, uint8_t* dst) {
  for (size_t i = 0; i < n; ++i) dst[i] = gsi_oracle_f32_to_e4m3_rne_sat(src[i]);
}

/*
 * The image as stored in FP8.  Input: the image M [o][k] in double (Eq. (3.2)).
 * Per row a:  m_j     = bf16_rne(M[a][j])            (the BF16 image of Section 4.2 is what gets quantised)
 *             amax    = max_j |m_j|
 *             scale_a = amax / 448 in fp32           (1 when the row is zero)
 *             code_j  = e4m3_rne_sat( m_j / scale_a in fp32 )
 *             Mq[a][j] = decode(code_j) * scale_a    (double)
 * The two divisions are single fp32 operations, so that an implementation in
 * fp32 arrives at the same codes from the same m_j.
 * Outputs (any may be NULL): codes [o][k], scales [o], Mq [o][k].
 */
int gsi_oracle_quantise_image_e4m3(const double* M, int o, int k, uint8_t* codes,
                                   float* scales, double* Mq) {
  if (!M || o < 0 || k <= 0) return 1;
#pragma omp parallel for schedule(static)
  for (int a = 0; a < o; ++a) {
    const double* Ma = M + (size_t)a * k;
    float amax = 0.0f;
    for (int j = 0; j < k; ++j) {
      float m = (float)bf16_bits_to_f64(gsi_oracle_f64_to_bf16_rne(Ma[j]));
      float am = fabsf(m);
      if (am > amax) amax = am;
    }
    volatile float scale_v = amax > 0.0f ? amax / 448.0f : 1.0f;
    const float scale = scale_v;
    if (scales) scales[a] = scale;
    for (int j = 0; j < k; ++j) {
      float m = (float)bf16_bits_to_f64(gsi_oracle_f64_to_bf16_rne(Ma[j]));
      volatile float t = m / scale;
      uint8_t c = gsi_oracle_f32_to_e4m3_rne_sat(t);
      if (codes) codes[(size_t)a * k + j] = c;
      if (Mq) Mq[(size_t)a * k + j] = gsi_oracle_e4m3_decode(c) * (double)scale;
    }
  }
  return 0;
}
