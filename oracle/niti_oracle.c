/*
 * NITI CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct restatement of the integer training ops of
 * "NITI: Training Integer Neural Networks Using Integer-only Arithmetic"
 * (arXiv 2009.13108).  Everything is computed in int64_t with direct loops:
 * no blocking, no im2col, no intrinsics, no code shared with the CUDA library.
 * Only tests, the smoke check and the bench's cpu_baseline / reference arm may
 * load this file; the GPU library never does.
 *
 * OpenMP is used only over independent output elements (each output is still
 * one straight loop), so results do not depend on the thread count.
 *
 * Pins (see tests/test_oracle_*.py): every function here is checked against
 * something other than itself -- hand-enumerated worked cases, closed forms
 * over all 2^bp discarded fractions, exact adjoint identities, float64 library
 * matmul / conv (exact below 2^53), Python int.bit_length, Fraction arithmetic
 * for the Taylor polynomial, and a second brute-force implementation in pure
 * Python on tiny shapes.  The composed training step (Algorithm 1) has no
 * number printed in the paper to compare with: "parity unpinned" as a whole;
 * it is pinned only as the composition of the individually pinned ops plus the
 * pure-Python cross-check on tiny nets.
 *
 * Layouts: activations / errors row-major [M][K] (fully connected) or NHWC
 * (convolution); weights [N_out][K_in] or [Cout][R][S][Cin]; gradients in the
 * weight's layout.  Scalars (exponents, bit-widths) are int32.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define NITI_REF_OK 0
#define NITI_REF_ERR_ARG 1
#define NITI_REF_ERR_RANGE 4
#define NITI_REF_ERR_OVERFLOW 7 /* an accumulator left the int32 range */

#define ROUND_PSR 0
#define ROUND_NEAREST 1

static int64_t abs64(int64_t x) { return x < 0 ? -x : x; }

/* ------------------------------------------------------------------------- */
/* Effective bit-width B(V), Section 3.2: the minimum number of bits needed   */
/* for the largest magnitude in the tensor (sign bit not counted; B = 0 for   */
/* the all-zero tensor).                                                      */
/* ------------------------------------------------------------------------- */
int32_t niti_ref_bitwidth(const int64_t *v, int64_t n) {
  int64_t mx = 0;
  for (int64_t i = 0; i < n; ++i) {
    int64_t m = abs64(v[i]);
    if (m > mx) mx = m;
  }
  int32_t b = 0;
  while (mx > 0) {
    ++b;
    mx >>= 1;
  }
  return b;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 3, pseudo-stochastic rounding of one fixed-point number whose    */
/* binary point sits at bit `bp`.  Works on the magnitude; the sign is put    */
/* back at the end.  The integer part keeps `mbits` magnitude bits and        */
/* saturates at 2^mbits - 1 when the increment would overflow it.             */
/* ------------------------------------------------------------------------- */
int32_t niti_ref_psr(int64_t x, int32_t bp, int32_t mbits) {
  int64_t m = abs64(x);
  int64_t q = m >> bp;                         /* integer part  |x|[..:bp]   */
  int64_t f = m & (((int64_t)1 << bp) - 1);    /* fraction      |x|[bp-1:0]  */
  int32_t w = bp;
  if (w & 1) { /* odd number of fraction bits: drop the lowest one */
    f >>= 1;
    w -= 1;
  }
  int32_t h = w / 2;
  int64_t top = f >> h;                        /* f[w-1 : w/2]   */
  int64_t bot = f & (((int64_t)1 << h) - 1);   /* f[w/2-1 : 0]   */
  if (top > bot) q += 1;
  int64_t qmax = ((int64_t)1 << mbits) - 1;
  if (q > qmax) q = qmax;
  return (int32_t)(x < 0 ? -q : q);
}

/* Round-to-nearest on the magnitude (half away from zero), same saturation.  */
/* The paper's accuracy runs use it for a and e (Section 4.3).                */
int32_t niti_ref_round_nearest(int64_t x, int32_t bp, int32_t mbits) {
  int64_t m = abs64(x);
  int64_t q = m >> bp;
  if (bp > 0) {
    int64_t f = m & (((int64_t)1 << bp) - 1);
    if (f >= ((int64_t)1 << (bp - 1))) q += 1;
  }
  int64_t qmax = ((int64_t)1 << mbits) - 1;
  if (q > qmax) q = qmax;
  return (int32_t)(x < 0 ? -q : q);
}

/* True stochastic rounding Rs (Section 3.4) with the random number r given   */
/* by the caller, 0 <= r < 2^bp: round up iff f > r.  Only the tests use it,  */
/* as the zero-bias ideal the pseudo-stochastic scheme is compared with.      */
int32_t niti_ref_round_stochastic(int64_t x, int32_t bp, int32_t mbits, int64_t r) {
  int64_t m = abs64(x);
  int64_t q = m >> bp;
  int64_t f = m & (((int64_t)1 << bp) - 1);
  if (f > r) q += 1;
  int64_t qmax = ((int64_t)1 << mbits) - 1;
  if (q > qmax) q = qmax;
  return (int32_t)(x < 0 ? -q : q);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2 applied to a whole tensor, with the call-site rule of          */
/* Algorithm 1: b = B(acc), bp = max(0, b - mbits), q = Round(acc, bp).       */
/* Returns b and bp through pointers; the caller adds bp to the exponent.     */
/* ------------------------------------------------------------------------- */
int niti_ref_shift_round(const int64_t *acc, int64_t n, int32_t mbits, int32_t round_mode,
                         int8_t *q, int32_t *b_out, int32_t *bp_out) {
  if (mbits < 1 || mbits > 7) return NITI_REF_ERR_ARG;
  int32_t b = niti_ref_bitwidth(acc, n);
  int32_t bp = b - mbits > 0 ? b - mbits : 0;
  for (int64_t i = 0; i < n; ++i) {
    int32_t r = round_mode == ROUND_NEAREST ? niti_ref_round_nearest(acc[i], bp, mbits)
                                            : niti_ref_psr(acc[i], bp, mbits);
    q[i] = (int8_t)r;
  }
  if (b_out) *b_out = b;
  if (bp_out) *bp_out = bp;
  return NITI_REF_OK;
}

/* 1 if some accumulator does not fit in int32 (the GPU contract is int32).   */
int niti_ref_overflows_int32(const int64_t *acc, int64_t n) {
  for (int64_t i = 0; i < n; ++i)
    if (acc[i] > 2147483647LL || acc[i] < -2147483648LL) return 1;
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Int8MatrixMultiply of Algorithm 1 for fully connected layers.              */
/*   forward  acc[m][n] = sum_k a[m][k] * w[n][k]                             */
/*   dgrad    acc[m][k] = sum_n e[m][n] * w[n][k]                             */
/*   wgrad    acc[n][k] = sum_m e[m][n] * a[m][k]                             */
/* ------------------------------------------------------------------------- */
void niti_ref_fc_fwd_acc(const int8_t *a, const int8_t *w, int64_t *acc, int64_t M, int64_t N,
                         int64_t K) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int64_t)a[m * K + k] * (int64_t)w[n * K + k];
      acc[m * N + n] = s;
    }
}

void niti_ref_fc_dgrad_acc(const int8_t *e, const int8_t *w, int64_t *acc, int64_t M, int64_t N,
                           int64_t K) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k) {
      int64_t s = 0;
      for (int64_t n = 0; n < N; ++n) s += (int64_t)e[m * N + n] * (int64_t)w[n * K + k];
      acc[m * K + k] = s;
    }
}

void niti_ref_fc_wgrad_acc(const int8_t *a, const int8_t *e, int64_t *acc, int64_t M, int64_t N,
                           int64_t K) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      int64_t s = 0;
      for (int64_t m = 0; m < M; ++m) s += (int64_t)e[m * N + n] * (int64_t)a[m * K + k];
      acc[n * K + k] = s;
    }
}

/* ------------------------------------------------------------------------- */
/* Convolution with stride `stride`, zero padding `pad`, R x S taps, NHWC /    */
/* [Co][R][S][Ci].  Direct loops over the definition (Section 3.2 reduces it   */
/* to a matrix multiply; the oracle deliberately does not).                    */
/*   y[b][i][j][co] = sum_{r,s,ci} x[b][i*stride+r-pad][j*stride+s-pad][ci]    */
/*                                 * w[co][r][s][ci]                           */
/* Output spatial size: Ho = (H + 2*pad - R) / stride + 1 (integer division),  */
/* Wo likewise.  The paper's measured layer has stride 1 (Section 5); its      */
/* networks also use stride 4 (AlexNet's first layer, Section 4).  The         */
/* functions without the _s suffix are the stride-1 case.                      */
/* ------------------------------------------------------------------------- */
void niti_ref_conv_fwd_acc_s(const int8_t *x, const int8_t *w, int64_t *acc, int64_t B, int64_t H,
                             int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S, int64_t pad,
                             int64_t stride) {
  int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(3) schedule(static)
  for (int64_t b = 0; b < B; ++b)
    for (int64_t i = 0; i < Ho; ++i)
      for (int64_t j = 0; j < Wo; ++j)
        for (int64_t co = 0; co < Co; ++co) {
          int64_t s = 0;
          for (int64_t r = 0; r < R; ++r)
            for (int64_t t = 0; t < S; ++t) {
              int64_t ii = i * stride + r - pad, jj = j * stride + t - pad;
              if (ii < 0 || ii >= H || jj < 0 || jj >= W) continue;
              for (int64_t ci = 0; ci < Ci; ++ci)
                s += (int64_t)x[((b * H + ii) * W + jj) * Ci + ci] *
                     (int64_t)w[((co * R + r) * S + t) * Ci + ci];
            }
          acc[((b * Ho + i) * Wo + j) * Co + co] = s;
        }
}

/* Error back-propagation through the convolution: the exact transpose of the */
/* forward map with respect to x:                                              */
/*   ex[b][ii][jj][ci] = sum over (r, s, co) and the output pixels (i, j) with */
/*   i*stride + r - pad == ii, j*stride + s - pad == jj of                     */
/*   e[b][i][j][co] * w[co][r][s][ci]                                          */
void niti_ref_conv_dgrad_acc_s(const int8_t *e, const int8_t *w, int64_t *acc, int64_t B, int64_t H,
                               int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S, int64_t pad,
                               int64_t stride) {
  int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(3) schedule(static)
  for (int64_t b = 0; b < B; ++b)
    for (int64_t ii = 0; ii < H; ++ii)
      for (int64_t jj = 0; jj < W; ++jj)
        for (int64_t ci = 0; ci < Ci; ++ci) {
          int64_t s = 0;
          for (int64_t r = 0; r < R; ++r)
            for (int64_t t = 0; t < S; ++t) {
              int64_t ti = ii - r + pad, tj = jj - t + pad;
              if (ti < 0 || tj < 0 || ti % stride || tj % stride) continue;
              int64_t i = ti / stride, j = tj / stride;
              if (i >= Ho || j >= Wo) continue;
              for (int64_t co = 0; co < Co; ++co)
                s += (int64_t)e[((b * Ho + i) * Wo + j) * Co + co] *
                     (int64_t)w[((co * R + r) * S + t) * Ci + ci];
            }
          acc[((b * H + ii) * W + jj) * Ci + ci] = s;
        }
}

/* Weight gradient: the exact transpose of the forward map with respect to w. */
/*   g[co][r][s][ci] = sum_{b,i,j} e[b][i][j][co]                              */
/*                                 * x[b][i*stride+r-pad][j*stride+s-pad][ci]  */
/* Loop nest: one output channel per OpenMP iteration; inside it the pixels    */
/* are the outer loops and (r, s, ci) the inner ones, so that x and e are read */
/* front to back once per output channel (with the pixel loops innermost every */
/* single output element streamed both tensors in full, which at 224 x 224,    */
/* batch 64 does not finish).  Each output is still the plain sum above; the   */
/* order of integer additions does not change it.                              */
void niti_ref_conv_wgrad_acc_s(const int8_t *x, const int8_t *e, int64_t *acc, int64_t B, int64_t H,
                               int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S, int64_t pad,
                               int64_t stride) {
  int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t co = 0; co < Co; ++co) {
    int64_t *g = acc + co * R * S * Ci;
    for (int64_t q = 0; q < R * S * Ci; ++q) g[q] = 0;
    for (int64_t b = 0; b < B; ++b)
      for (int64_t i = 0; i < Ho; ++i)
        for (int64_t j = 0; j < Wo; ++j) {
          int64_t ev = (int64_t)e[((b * Ho + i) * Wo + j) * Co + co];
          for (int64_t r = 0; r < R; ++r) {
            int64_t ii = i * stride + r - pad;
            if (ii < 0 || ii >= H) continue;
            for (int64_t t = 0; t < S; ++t) {
              int64_t jj = j * stride + t - pad;
              if (jj < 0 || jj >= W) continue;
              for (int64_t ci = 0; ci < Ci; ++ci)
                g[(r * S + t) * Ci + ci] += ev * (int64_t)x[((b * H + ii) * W + jj) * Ci + ci];
            }
          }
        }
  }
}

void niti_ref_conv_fwd_acc(const int8_t *x, const int8_t *w, int64_t *acc, int64_t B, int64_t H,
                           int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S, int64_t pad) {
  niti_ref_conv_fwd_acc_s(x, w, acc, B, H, W, Ci, Co, R, S, pad, 1);
}
void niti_ref_conv_dgrad_acc(const int8_t *e, const int8_t *w, int64_t *acc, int64_t B, int64_t H,
                             int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S,
                             int64_t pad) {
  niti_ref_conv_dgrad_acc_s(e, w, acc, B, H, W, Ci, Co, R, S, pad, 1);
}
void niti_ref_conv_wgrad_acc(const int8_t *x, const int8_t *e, int64_t *acc, int64_t B, int64_t H,
                             int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S,
                             int64_t pad) {
  niti_ref_conv_wgrad_acc_s(x, e, acc, B, H, W, Ci, Co, R, S, pad, 1);
}

/* ------------------------------------------------------------------------- */
/* Integer cross-entropy gradient, Section 3.5, before rounding.              */
/* Per sample (row): e32[i] = T_i - [i == label] * sum_j T_j, where T_i is an  */
/* integer proportional to exp(a_i * 2^s_a):                                  */
/*   s_a <= -7 (Eq. 2): second-order Taylor polynomial scaled by 2^(1-2 s_a): */
/*        T_i = 2^(1-2s) + a_i * 2^(1-s) + a_i^2                              */
/*   s_a >  -7 (Eq. 3-4): xh_i = (47274 * a_i) * 2^(s_a-15), truncated by an  */
/*        arithmetic right shift; p = the smallest xh_i that is larger than   */
/*        max(xh) - 10; xt_i = max(0, xh_i - p); T_i = 1 << xt_i.             */
/* The 1/C factor and 2^p only change the (unused) exponent of e.             */
/* Supported domain: -22 <= s_a <= 24.                                        */
/* ------------------------------------------------------------------------- */
int niti_ref_xent_acc(const int8_t *a, int32_t s_a, const int32_t *labels, int64_t *e32, int64_t B,
                      int64_t N) {
  if (s_a < -22 || s_a > 24) return NITI_REF_ERR_RANGE;
  int64_t *T = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
  if (!T) return NITI_REF_ERR_ARG;
  for (int64_t r = 0; r < B; ++r) {
    const int8_t *row = a + r * N;
    if (labels[r] < 0 || labels[r] >= N) {
      free(T);
      return NITI_REF_ERR_ARG;
    }
    if (s_a <= -7) {
      int64_t s = s_a;
      for (int64_t i = 0; i < N; ++i) {
        int64_t ai = row[i];
        T[i] = ((int64_t)1 << (1 - 2 * s)) + ai * ((int64_t)1 << (1 - s)) + ai * ai;
      }
    } else {
      int64_t sh = 15 - (int64_t)s_a;
      int64_t mx = 0;
      for (int64_t i = 0; i < N; ++i) {
        int64_t P = 47274 * (int64_t)row[i];
        /* >> on a negative int64 is an arithmetic shift with gcc: floor.   */
        int64_t xh = sh >= 0 ? (P >> sh) : P * ((int64_t)1 << (-sh));
        T[i] = xh;
        if (i == 0 || xh > mx) mx = xh;
      }
      int64_t p = mx;
      for (int64_t i = 0; i < N; ++i)
        if (T[i] > mx - 10 && T[i] < p) p = T[i];
      for (int64_t i = 0; i < N; ++i) {
        int64_t xt = T[i] - p;
        if (xt < 0) xt = 0;
        T[i] = (int64_t)1 << xt;
      }
    }
    int64_t C = 0;
    for (int64_t i = 0; i < N; ++i) C += T[i];
    for (int64_t i = 0; i < N; ++i) e32[r * N + i] = T[i] - (i == labels[r] ? C : 0);
  }
  free(T);
  return NITI_REF_OK;
}

/* Number of rows whose first arg-max equals the label (a metric, not part of */
/* the paper's update rule).                                                   */
int32_t niti_ref_count_correct(const int8_t *a, const int32_t *labels, int64_t B, int64_t N) {
  int32_t c = 0;
  for (int64_t r = 0; r < B; ++r) {
    int64_t best = 0;
    for (int64_t i = 1; i < N; ++i)
      if (a[r * N + i] > a[r * N + best]) best = i;
    if (best == labels[r]) ++c;
  }
  return c;
}

/* ------------------------------------------------------------------------- */
/* Weight update of Algorithm 1: w <- w - g, kept inside [-127, 127].         */
/* ------------------------------------------------------------------------- */
void niti_ref_sgd_update(int8_t *w, const int8_t *g, int64_t n) {
  for (int64_t i = 0; i < n; ++i) {
    int64_t v = (int64_t)w[i] - (int64_t)g[i];
    if (v > 127) v = 127;
    if (v < -127) v = -127;
    w[i] = (int8_t)v;
  }
}

/* ------------------------------------------------------------------------- */
/* Support ops on int8 (implied by the paper's networks); exponents unchanged. */
/* ------------------------------------------------------------------------- */
void niti_ref_relu_fwd(const int8_t *x, int8_t *y, int64_t n) {
  for (int64_t i = 0; i < n; ++i) y[i] = x[i] > 0 ? x[i] : 0;
}

/* e_in = e_out where the ReLU output was positive, else 0. */
void niti_ref_relu_bwd(const int8_t *y, const int8_t *e_out, int8_t *e_in, int64_t n) {
  for (int64_t i = 0; i < n; ++i) e_in[i] = y[i] > 0 ? e_out[i] : 0;
}

/* 2x2 max-pool, stride 2, NHWC, H and W even. */
void niti_ref_maxpool2_fwd(const int8_t *x, int8_t *y, int64_t B, int64_t H, int64_t W, int64_t C) {
  int64_t Ho = H / 2, Wo = W / 2;
  for (int64_t b = 0; b < B; ++b)
    for (int64_t i = 0; i < Ho; ++i)
      for (int64_t j = 0; j < Wo; ++j)
        for (int64_t c = 0; c < C; ++c) {
          int8_t m = -128;
          for (int64_t di = 0; di < 2; ++di)
            for (int64_t dj = 0; dj < 2; ++dj) {
              int8_t v = x[((b * H + 2 * i + di) * W + 2 * j + dj) * C + c];
              if (v > m) m = v;
            }
          y[((b * Ho + i) * Wo + j) * C + c] = m;
        }
}

/* Routes each output error to the first maximum of its window in (row, col)  */
/* order; every other input position gets 0.                                   */
void niti_ref_maxpool2_bwd(const int8_t *x, const int8_t *e_out, int8_t *e_in, int64_t B, int64_t H,
                           int64_t W, int64_t C) {
  int64_t Ho = H / 2, Wo = W / 2;
  memset(e_in, 0, (size_t)(B * H * W * C));
  for (int64_t b = 0; b < B; ++b)
    for (int64_t i = 0; i < Ho; ++i)
      for (int64_t j = 0; j < Wo; ++j)
        for (int64_t c = 0; c < C; ++c) {
          int64_t best = -1;
          int8_t m = 0;
          for (int64_t di = 0; di < 2; ++di)
            for (int64_t dj = 0; dj < 2; ++dj) {
              int64_t idx = ((b * H + 2 * i + di) * W + 2 * j + dj) * C + c;
              if (best < 0 || x[idx] > m) {
                best = idx;
                m = x[idx];
              }
            }
          e_in[best] = e_out[((b * Ho + i) * Wo + j) * C + c];
        }
}

/* ------------------------------------------------------------------------- */
/* Composed layer ops: one matrix multiply followed by the bit-width, shift   */
/* and rounding of Algorithm 1, with the argument lists of the GPU library    */
/* (host pointers instead of device pointers).  Return NITI_REF_ERR_OVERFLOW  */
/* if an accumulator leaves the int32 range.                                  */
/* ------------------------------------------------------------------------- */
static int finish(int64_t *acc, int64_t n, int32_t mbits, int32_t round_mode, int8_t *out,
                  int32_t *b_out, int32_t *bp_out) {
  int ovf = niti_ref_overflows_int32(acc, n);
  int rc = niti_ref_shift_round(acc, n, mbits, round_mode, out, b_out, bp_out);
  free(acc);
  if (rc) return rc;
  return ovf ? NITI_REF_ERR_OVERFLOW : NITI_REF_OK;
}

int niti_ref_linear_fwd(const int8_t *a, int32_t s_a, const int8_t *w, int32_t s_w, int8_t *out,
                        int32_t *s_out, int32_t *b_out, int64_t M, int64_t N, int64_t K, int relu,
                        int round_mode) {
  int64_t *acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)(M * N));
  if (!acc) return NITI_REF_ERR_ARG;
  niti_ref_fc_fwd_acc(a, w, acc, M, N, K);
  int32_t bp = 0;
  int rc = finish(acc, M * N, 7, round_mode, out, b_out, &bp);
  if (relu) niti_ref_relu_fwd(out, out, M * N);
  if (s_out) *s_out = s_a + s_w + bp;
  return rc;
}

/* e_prev may be NULL (first layer: no error to propagate). mask may be NULL;  */
/* otherwise e_prev is zeroed where mask <= 0 (the ReLU that produced `a`).   */
int niti_ref_linear_bwd(const int8_t *a, const int8_t *e, const int8_t *w, int8_t *e_prev,
                        const int8_t *mask, int8_t *g, int32_t *b_e, int32_t *b_g, int64_t M,
                        int64_t N, int64_t K, int m_u, int round_mode) {
  int rc = NITI_REF_OK;
  int64_t *acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N * K));
  if (!acc) return NITI_REF_ERR_ARG;
  niti_ref_fc_wgrad_acc(a, e, acc, M, N, K);
  int r1 = finish(acc, N * K, m_u, round_mode, g, b_g, NULL);
  if (r1) rc = r1;
  if (e_prev) {
    acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)(M * K));
    if (!acc) return NITI_REF_ERR_ARG;
    niti_ref_fc_dgrad_acc(e, w, acc, M, N, K);
    int r2 = finish(acc, M * K, 7, round_mode, e_prev, b_e, NULL);
    if (r2) rc = r2;
    if (mask) niti_ref_relu_bwd(mask, e_prev, e_prev, M * K);
  }
  return rc;
}

int niti_ref_conv_fwd_s(const int8_t *x, int32_t s_x, const int8_t *w, int32_t s_w, int8_t *y,
                        int32_t *s_y, int32_t *b_y, int64_t B, int64_t H, int64_t W, int64_t Ci,
                        int64_t Co, int64_t R, int64_t S, int64_t pad, int64_t stride, int relu,
                        int round_mode) {
  int64_t Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
  int64_t n = B * Ho * Wo * Co;
  int64_t *acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
  if (!acc) return NITI_REF_ERR_ARG;
  niti_ref_conv_fwd_acc_s(x, w, acc, B, H, W, Ci, Co, R, S, pad, stride);
  int32_t bp = 0;
  int rc = finish(acc, n, 7, round_mode, y, b_y, &bp);
  if (relu) niti_ref_relu_fwd(y, y, n);
  if (s_y) *s_y = s_x + s_w + bp;
  return rc;
}

int niti_ref_conv_fwd(const int8_t *x, int32_t s_x, const int8_t *w, int32_t s_w, int8_t *y,
                      int32_t *s_y, int32_t *b_y, int64_t B, int64_t H, int64_t W, int64_t Ci,
                      int64_t Co, int64_t R, int64_t S, int64_t pad, int relu, int round_mode) {
  return niti_ref_conv_fwd_s(x, s_x, w, s_w, y, s_y, b_y, B, H, W, Ci, Co, R, S, pad, 1, relu, round_mode);
}

int niti_ref_conv_dgrad_s(const int8_t *e, const int8_t *w, int8_t *e_prev, const int8_t *mask,
                          int32_t *b_e, int64_t B, int64_t H, int64_t W, int64_t Ci, int64_t Co,
                          int64_t R, int64_t S, int64_t pad, int64_t stride, int round_mode) {
  int64_t n = B * H * W * Ci;
  int64_t *acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
  if (!acc) return NITI_REF_ERR_ARG;
  niti_ref_conv_dgrad_acc_s(e, w, acc, B, H, W, Ci, Co, R, S, pad, stride);
  int rc = finish(acc, n, 7, round_mode, e_prev, b_e, NULL);
  if (mask) niti_ref_relu_bwd(mask, e_prev, e_prev, n);
  return rc;
}

int niti_ref_conv_dgrad(const int8_t *e, const int8_t *w, int8_t *e_prev, const int8_t *mask,
                        int32_t *b_e, int64_t B, int64_t H, int64_t W, int64_t Ci, int64_t Co,
                        int64_t R, int64_t S, int64_t pad, int round_mode) {
  return niti_ref_conv_dgrad_s(e, w, e_prev, mask, b_e, B, H, W, Ci, Co, R, S, pad, 1, round_mode);
}

int niti_ref_conv_wgrad_s(const int8_t *x, const int8_t *e, int8_t *g, int32_t *b_g, int64_t B,
                          int64_t H, int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S,
                          int64_t pad, int64_t stride, int m_u, int round_mode) {
  int64_t n = Co * R * S * Ci;
  int64_t *acc = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
  if (!acc) return NITI_REF_ERR_ARG;
  niti_ref_conv_wgrad_acc_s(x, e, acc, B, H, W, Ci, Co, R, S, pad, stride);
  return finish(acc, n, m_u, round_mode, g, b_g, NULL);
}

int niti_ref_conv_wgrad(const int8_t *x, const int8_t *e, int8_t *g, int32_t *b_g, int64_t B,
                        int64_t H, int64_t W, int64_t Ci, int64_t Co, int64_t R, int64_t S,
                        int64_t pad, int m_u, int round_mode) {
  return niti_ref_conv_wgrad_s(x, e, g, b_g, B, H, W, Ci, Co, R, S, pad, 1, m_u, round_mode);
}

int niti_ref_int_xent(const int8_t *a, int32_t s_a, const int32_t *labels, int8_t *e, int32_t *b_e,
                      int32_t *n_correct, int64_t B, int64_t N, int round_mode) {
  int64_t *e32 = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B * N));
  if (!e32) return NITI_REF_ERR_ARG;
  int rc = niti_ref_xent_acc(a, s_a, labels, e32, B, N);
  if (rc) {
    free(e32);
    return rc;
  }
  if (n_correct) *n_correct = niti_ref_count_correct(a, labels, B, N);
  /* the loss accumulators are 64-bit quantities (up to 2^45 at s_a = -22): the int32 contract of
   * the matrix multiplies does not apply to them */
  rc = niti_ref_shift_round(e32, B * N, 7, round_mode, e, b_e, NULL);
  free(e32);
  return rc;
}
