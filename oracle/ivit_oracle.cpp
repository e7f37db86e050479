/*
 * CPU oracle for the integer-only ViT encoder forward pass (I-ViT).
 * TEST INFRASTRUCTURE ONLY - see ivit_oracle.h.  Plain C++17, int64
 * arithmetic, explicit floor helpers (C's >> and / are never applied to
 * negative values), OpenMP only over independent rows / batches.
 */
#include "ivit_oracle.h"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

/* floor(a / b) for b > 0 */
inline int64_t floordiv(int64_t a, int64_t b) {
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) q -= 1;
  return q;
}

/* arithmetic shift right = floor(a / 2^k), k >= 0 */
inline int64_t asr(int64_t a, int k) {
  if (k >= 63) return a < 0 ? -1 : 0;
  return floordiv(a, (int64_t)1 << k);
}

inline int64_t sat8(int64_t v) { return v > 127 ? 127 : (v < -128 ? -128 : v); }

/* Sec. 3.2: the dyadic requantisation (b * acc) >> c, with the rounding of
 * Eq. (I_A): half is added before the floor shift. */
inline int64_t rq(int64_t a, int64_t m, int s) {
  return floordiv(a * m + ((int64_t)1 << (s - 1)), (int64_t)1 << s);
}

inline bool scale_ok(const orc_scale& sc) {
  if (sc.mult_c) return sc.shift_c != nullptr;
  return sc.mult > 0 && sc.shift >= 1 && sc.shift <= 62;
}
inline int64_t sc_m(const orc_scale& sc, int64_t c) { return sc.mult_c ? sc.mult_c[c] : sc.mult; }
inline int sc_s(const orc_scale& sc, int64_t c) { return sc.mult_c ? sc.shift_c[c] : sc.shift; }

/* Algorithm 1, function ShiftExp.  I <= 0, I0 >= 1. */
inline int64_t shiftexp(int64_t I, int64_t I0, int N) {
  int64_t Ip = I + asr(I, 1) - asr(I, 4); /* I * log2(e), (1.0111)b */
  int64_t q = floordiv(-Ip, I0);          /* = floor(Ip / (-I0)), integer part */
  int64_t r = -(Ip + q * I0);             /* decimal part, 0 <= r < I0 */
  int64_t Ib = asr(-r, 1) + I0;           /* Eq. (linear): 2^x ~ 1 + x/2 */
  if (q <= N) return Ib * ((int64_t)1 << (N - q)); /* Ib << (N - q) */
  if (q - N >= 63) return 0;                         /* every bit of Ib (< 2^63) is shifted out */
  return asr(Ib, (int)(q - N));
}

/* Eq. (IntDiv) */
inline int64_t intdiv(int64_t I1, int64_t I2, int M, int k) {
  if (I2 == 0) return 0;
  __int128 f = (__int128)(((__int128)1 << M) / I2);
  __int128 prod = f * (__int128)I1;
  int sh = M - (k - 1);
  __int128 d = (__int128)1 << sh;
  __int128 q = prod / d;
  if (prod % d != 0 && prod < 0) q -= 1;
  return (int64_t)q;
}

inline int bitlen(int64_t n) {
  int b = 0;
  while (n > 0) { ++b; n = n / 2; }
  return b;
}

/* Sec. 3.5, Eq. (iterative): I_{i+1} = (I_i + floor(n / I_i)) >> 1, initial
 * value 2^floor(bit(n)/2), ten iterations.  Iterations 2..10 only accept a
 * decrease, which is the paper's stopping rule I_{i+1} >= I_i turned into a
 * fixed-count form (once the sequence stops decreasing it is held). */
inline int64_t isqrt10(int64_t n) {
  if (n <= 0) return 0;
  int64_t x = (int64_t)1 << (bitlen(n) / 2);
  x = asr(x + floordiv(n, x), 1);
  for (int i = 1; i < 10; ++i) {
    int64_t nx = asr(x + floordiv(n, x), 1);
    if (nx < x) x = nx;
  }
  return x;
}

inline int64_t isqrt_printed(int64_t n) {
  if (n <= 0) return 0;
  int64_t x = (int64_t)1 << (bitlen(n) / 2);
  for (int i = 0; i < 10; ++i) x = asr(x + floordiv(n, x), 1);
  return x;
}

bool exp_params_ok(const orc_exp_params& p, int64_t row_len, bool gelu) {
  if (p.I0 < 1 || p.I0 > (1 << 15)) return false;
  if (p.N < 0 || p.N > 24) return false;
  if (p.k_out < 2 || p.k_out > 8) return false; /* the output is stored as int8 */
  if (p.M < 32 || p.M > 60) return false;
  const int64_t top = (int64_t)p.I0 << p.N;
  if (gelu) {
    if (2 * top > 4294967295LL) return false;
  } else {
    if (row_len * top > 4294967295LL) return false;
  }
  return true;
}

}  // namespace

extern "C" {

int64_t orc_rq(int64_t a, int64_t m, int32_t s) { return rq(a, m, s); }
void orc_rq_array(const int64_t* a, int64_t n, int64_t m, int32_t s, int64_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = rq(a[i], m, s);
}

int orc_dyadic_from_double(double ratio, int32_t* mult, int32_t* shift) {
  if (!(ratio > 0.0) || !std::isfinite(ratio)) return -1;
  int e = 0;
  double mant = std::frexp(ratio, &e); /* ratio = mant * 2^e, mant in [0.5, 1) */
  int64_t b = (int64_t)std::llround(std::ldexp(mant, 31));
  int c = 31 - e;
  if (b == ((int64_t)1 << 31)) { b = (int64_t)1 << 30; c -= 1; }
  if (c < 1 || c > 62) return -2;
  *mult = (int32_t)b;
  *shift = c;
  return 0;
}

int64_t orc_shiftexp(int64_t I, int64_t I0, int32_t N) { return shiftexp(I, I0, N); }
int64_t orc_intdiv(int64_t I1, int64_t I2, int32_t M, int32_t k) { return intdiv(I1, I2, M, k); }
int64_t orc_isqrt(int64_t n) { return isqrt10(n); }
void orc_isqrt_array(const int64_t* n, int64_t count, int64_t* out) {
  for (int64_t i = 0; i < count; ++i) out[i] = isqrt10(n[i]);
}
int64_t orc_isqrt_as_printed(int64_t n) { return isqrt_printed(n); }

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int orc_linear(const int8_t* A, int64_t lda, const int8_t* W, int64_t ldw, const int32_t* bias,
               orc_scale scale, const int8_t* res, int64_t ldres, int64_t res_rows,
               orc_scale res_scale, void* out, int64_t ldo, int32_t out_dtype,
               int64_t out_group_rows, int64_t out_group_stride, int64_t M, int64_t N, int64_t K) {
  if (!A || !W || !out || M < 0 || N < 0 || K < 0 || K > 65536) return -1;
  if (!scale_ok(scale)) return -2;
  if (res && (!scale_ok(res_scale) || res_rows < 1)) return -2;
  if (out_dtype != ORC_I8 && out_dtype != ORC_I32) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    const int64_t ro = out_group_rows > 0
                           ? (r / out_group_rows) * out_group_stride + (r % out_group_rows)
                           : r;
    for (int64_t c = 0; c < N; ++c) {
      int64_t acc = 0;
      for (int64_t k = 0; k < K; ++k) acc += (int64_t)A[r * lda + k] * (int64_t)W[c * ldw + k];
      if (bias) acc += bias[c];
      int64_t v = rq(acc, sc_m(scale, c), sc_s(scale, c));
      if (res) v += rq((int64_t)res[(r % res_rows) * ldres + c], sc_m(res_scale, c), sc_s(res_scale, c));
      if (out_dtype == ORC_I8)
        ((int8_t*)out)[ro * ldo + c] = (int8_t)sat8(v);
      else
        ((int32_t*)out)[ro * ldo + c] = (int32_t)v;
    }
  }
  return 0;
}

int orc_matmul(const int8_t* A, int64_t lda, int64_t sAo, int64_t sAi, const int8_t* B, int64_t ldb,
               int64_t sBo, int64_t sBi, int32_t transB, const int32_t* bias32, int64_t ldbias,
               int64_t bias_batches, orc_scale scale, int8_t* C, int64_t ldc, int64_t sCo,
               int64_t sCi, int64_t batches_outer, int64_t batches_inner, int64_t Ma, int64_t Nb,
               int64_t K) {
  if (!A || !B || !C || K > 65536) return -1;
  if (!scale_ok(scale) || scale.mult_c) return -2;
  if (bias32 && bias_batches < 1) return -1;
  const int64_t nb = batches_outer * batches_inner;
#pragma omp parallel for schedule(static)
  for (int64_t b = 0; b < nb; ++b) {
    const int64_t bo = b / batches_inner, bi = b % batches_inner;
    const int8_t* Ab = A + bo * sAo + bi * sAi;
    const int8_t* Bb = B + bo * sBo + bi * sBi;
    int8_t* Cb = C + bo * sCo + bi * sCi;
    const int32_t* biasb = bias32 ? bias32 + (b % bias_batches) * Ma * ldbias : nullptr;
    for (int64_t i = 0; i < Ma; ++i)
      for (int64_t j = 0; j < Nb; ++j) {
        int64_t acc = 0;
        for (int64_t k = 0; k < K; ++k) {
          const int64_t bv = transB ? Bb[j * ldb + k] : Bb[k * ldb + j];
          acc += (int64_t)Ab[i * lda + k] * bv;
        }
        if (biasb) acc += biasb[i * ldbias + j];
        Cb[i * ldc + j] = (int8_t)sat8(rq(acc, scale.mult, scale.shift));
      }
  }
  return 0;
}

int orc_shiftmax(const void* in, int32_t in_dtype, int64_t ldin, const int32_t* bias32,
                 int64_t ldbias, int64_t bias_rows, orc_scale pre, orc_exp_params p, int8_t* out,
                 int64_t ldout, int64_t rows, int64_t d) {
  if (!in || !out || d < 1) return -1;
  if (!exp_params_ok(p, d, false)) return -3;
  if (in_dtype == ORC_I32 && (!scale_ok(pre) || pre.mult_c)) return -2;
  if (in_dtype != ORC_I8 && in_dtype != ORC_I32) return -1;
  const int64_t omax = ((int64_t)1 << (p.k_out - 1)) - 1;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<int64_t> x(d), e(d);
    for (int64_t i = 0; i < d; ++i) {
      if (in_dtype == ORC_I8) {
        x[i] = ((const int8_t*)in)[r * ldin + i];
      } else {
        int64_t a = ((const int32_t*)in)[r * ldin + i];
        if (bias32) a += bias32[(r % bias_rows) * ldbias + i];
        x[i] = sat8(rq(a, pre.mult, pre.shift));
      }
    }
    int64_t mx = x[0];
    for (int64_t i = 1; i < d; ++i) mx = x[i] > mx ? x[i] : mx;
    int64_t sum = 0;
    for (int64_t i = 0; i < d; ++i) {
      e[i] = shiftexp(x[i] - mx, p.I0, p.N); /* I_delta = I_in - max(I_in) */
      sum += e[i];
    }
    for (int64_t i = 0; i < d; ++i) {
      int64_t o = intdiv(e[i], sum, p.M, p.k_out);
      out[r * ldout + i] = (int8_t)(o > omax ? omax : o);
    }
  }
  return 0;
}

/* Algorithm 1 taken literally on wide inputs: no requantisation in front, I0 = round(1 / S_in) as large as
 * the score scale makes it, 64-bit exponentials and sums, M chosen by the caller. */
int orc_shiftmax_direct(const int32_t* in, int64_t ldin, orc_exp_params p, int8_t* out, int64_t ldout,
                        int64_t rows, int64_t d) {
  if (!in || !out || d < 1) return -1;
  if (p.I0 < 1 || p.I0 > (1 << 28) || p.N < 0 || p.N > 24) return -3;
  if (p.k_out < 2 || p.k_out > 8 || p.M < 32 || p.M > 62) return -3;
  /* largest possible sum d * I0 * 2^N must leave the reciprocal floor(2^M / sum) at least 13 bits */
  if ((__int128)d * p.I0 * ((__int128)1 << p.N) > ((__int128)1 << (p.M - 13))) return -3;
  const int64_t omax = ((int64_t)1 << (p.k_out - 1)) - 1;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<int64_t> e(d);
    int64_t mx = in[r * ldin];
    for (int64_t i = 1; i < d; ++i) mx = in[r * ldin + i] > mx ? in[r * ldin + i] : mx;
    int64_t sum = 0;
    for (int64_t i = 0; i < d; ++i) {
      e[i] = shiftexp((int64_t)in[r * ldin + i] - mx, p.I0, p.N); /* I_delta = I_in - max(I_in) */
      sum += e[i];
    }
    for (int64_t i = 0; i < d; ++i) {
      int64_t o = intdiv(e[i], sum, p.M, p.k_out);
      out[r * ldout + i] = (int8_t)(o > omax ? omax : o);
    }
  }
  return 0;
}

static int shiftgelu_rows(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                          int64_t ldout, int64_t rows, int64_t cols, bool static_max);

int orc_shiftgelu(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                  int64_t ldout, int64_t rows, int64_t cols) {
  return shiftgelu_rows(in, ldin, p, post, out, ldout, rows, cols, false);
}

int orc_shiftgelu_static(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                         int64_t ldout, int64_t rows, int64_t cols) {
  return shiftgelu_rows(in, ldin, p, post, out, ldout, rows, cols, true);
}

static int shiftgelu_rows(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                          int64_t ldout, int64_t rows, int64_t cols, bool static_max) {
  if (!in || !out || cols < 1) return -1;
  if (!exp_params_ok(p, cols, true)) return -3;
  if (!scale_ok(post) || post.mult_c) return -2;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<int64_t> Ip(cols);
    int64_t mx = 0; /* max(I_p), floored at 0 so both exponents are <= 0 */
    for (int64_t i = 0; i < cols; ++i) {
      const int64_t x = in[r * ldin + i];
      Ip[i] = x + asr(x, 1) + asr(x, 3) + asr(x, 4); /* 1.702 * I, (1.1011)b */
      if (Ip[i] > mx) mx = Ip[i];
    }
    if (static_max) mx = 127 + asr(127, 1) + asr(127, 3) + asr(127, 4); /* I_p(127) = 212 */
    const int64_t e1 = shiftexp(-mx, p.I0, p.N);
    for (int64_t i = 0; i < cols; ++i) {
      const int64_t x = in[r * ldin + i];
      const int64_t e = shiftexp(Ip[i] - mx, p.I0, p.N);
      const int64_t div = intdiv(e, e + e1, p.M, p.k_out); /* sigmoid in units of 2^-(k-1) */
      out[r * ldout + i] = (int8_t)sat8(rq(x * div, post.mult, post.shift));
    }
  }
  return 0;
}

int orc_layernorm(const void* in, int32_t in_dtype, int64_t ldin, orc_scale gamma_scale,
                  const int32_t* beta, int32_t M_ln, int8_t* out, int64_t ldout, int64_t rows,
                  int64_t C) {
  if (!in || !out || C < 1 || M_ln < 8 || M_ln > 30) return -1;
  if (!scale_ok(gamma_scale)) return -2;
  if (in_dtype != ORC_I8 && in_dtype != ORC_I32) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<int64_t> x(C);
    int64_t S1 = 0;
    for (int64_t i = 0; i < C; ++i) {
      x[i] = in_dtype == ORC_I8 ? (int64_t)((const int8_t*)in)[r * ldin + i]
                                : (int64_t)((const int32_t*)in)[r * ldin + i];
      S1 += x[i];
    }
    const int64_t mu = floordiv(2 * S1 + C, 2 * C); /* mean, round half up */
    int64_t V = 0;
    for (int64_t i = 0; i < C; ++i) {
      const int64_t y = x[i] - mu;
      V += y * y;
    }
    const int64_t sd = isqrt10(V);
    const int64_t F = sd == 0 ? 0 : floordiv((int64_t)1 << M_ln, sd);
    for (int64_t i = 0; i < C; ++i) {
      const int64_t y = x[i] - mu;
      int64_t v = rq(y * F, sc_m(gamma_scale, i), sc_s(gamma_scale, i));
      if (beta) v += beta[i];
      out[r * ldout + i] = (int8_t)sat8(v);
    }
  }
  return 0;
}

int orc_attention(const orc_block_params* p, const int8_t* QKV, int8_t* O) {
  const int64_t B = p->B, T = p->T, D = p->D, h = p->heads, d = D / h;
  if (d * h != D) return -1;
  const int64_t ldq = 3 * D;
  std::vector<int8_t> S8((size_t)(B * h * T * T)), P((size_t)(B * h * T * T));
  /* scores: Q_i * K_i^T (+ bias), requantised to int8 (1/sqrt(d) is inside qk_scale) */
  int rc = orc_matmul(QKV, ldq, T * ldq, d, QKV + D, ldq, T * ldq, d, 1, p->attn_bias, T,
                      p->attn_bias ? p->attn_bias_batches : 1, p->qk_scale, S8.data(), T,
                      h * T * T, T * T, B, h, T, T, d);
  if (rc) return rc;
  orc_scale none = {nullptr, nullptr, 1, 1};
  rc = orc_shiftmax(S8.data(), ORC_I8, T, nullptr, 0, 1, none, p->smax, P.data(), T, B * h * T, T);
  if (rc) return rc;
  /* Attn_i = P_i * V_i, heads concatenated along the feature dimension */
  rc = orc_matmul(P.data(), T, h * T * T, T * T, QKV + 2 * D, ldq, T * ldq, d, 0, nullptr, 0, 1,
                  p->pv_scale, O, D, T * D, d, B, h, T, d, T);
  return rc;
}

int orc_block_forward(const orc_block_params* p, const int8_t* X, int8_t* Y) {
  const int64_t M = p->B * p->T, D = p->D, H = p->H;
  std::vector<int8_t> A((size_t)(M * D)), QKV((size_t)(M * 3 * D)), O((size_t)(M * D)),
      Xh((size_t)(M * D)), G((size_t)(M * H)), Hh((size_t)(M * H));
  orc_scale none = {nullptr, nullptr, 1, 1};
  int rc;
  /* X^ = MSA(LayerNorm(X)) + X */
  if ((rc = orc_layernorm(X, ORC_I8, D, p->ln1_gamma, p->ln1_beta, p->M_ln, A.data(), D, M, D))) return rc;
  if ((rc = orc_linear(A.data(), D, p->Wqkv, D, p->bqkv, p->qkv_scale, nullptr, 0, 1, none, QKV.data(),
                       3 * D, ORC_I8, 0, 0, M, 3 * D, D))) return rc;
  if ((rc = orc_attention(p, QKV.data(), O.data()))) return rc;
  if ((rc = orc_linear(O.data(), D, p->Wo, D, p->bo, p->o_scale, X, D, M, p->res1_scale, Xh.data(), D,
                       ORC_I8, 0, 0, M, D, D))) return rc;
  /* Y = MLP(LayerNorm(X^)) + X^ */
  if ((rc = orc_layernorm(Xh.data(), ORC_I8, D, p->ln2_gamma, p->ln2_beta, p->M_ln, A.data(), D, M, D))) return rc;
  if ((rc = orc_linear(A.data(), D, p->W1, D, p->b1, p->fc1_scale, nullptr, 0, 1, none, G.data(), H,
                       ORC_I8, 0, 0, M, H, D))) return rc;
  if ((rc = shiftgelu_rows(G.data(), H, p->gelu, p->gelu_post, Hh.data(), H, M, H, p->gelu_static_max != 0))) return rc;
  if ((rc = orc_linear(Hh.data(), H, p->W2, H, p->b2, p->fc2_scale, Xh.data(), D, M, p->res2_scale, Y, D,
                       ORC_I8, 0, 0, M, D, H))) return rc;
  return 0;
}

int orc_patchify(const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi, int64_t P,
                 int64_t window, int8_t* out) {
  if (!img || !out || P < 1 || Hi % P || Wi % P) return -1;
  const int64_t gh = Hi / P, gw = Wi / P, K = C * P * P;
  if (window > 0 && (gh % window || gw % window)) return -1;
  for (int64_t b = 0; b < B; ++b)
    for (int64_t gy = 0; gy < gh; ++gy)
      for (int64_t gx = 0; gx < gw; ++gx) {
        int64_t row;
        if (window > 0) {
          const int64_t wy = gy / window, wx = gx / window, iy = gy % window, ix = gx % window;
          row = (wy * (gw / window) + wx) * window * window + iy * window + ix;
        } else {
          row = gy * gw + gx;
        }
        int8_t* o = out + (b * gh * gw + row) * K;
        for (int64_t c = 0; c < C; ++c)
          for (int64_t py = 0; py < P; ++py)
            for (int64_t px = 0; px < P; ++px)
              o[(c * P + py) * P + px] = img[((b * C + c) * Hi + gy * P + py) * Wi + gx * P + px];
      }
  return 0;
}

int orc_gather_rows(const int8_t* src, int64_t ldsrc, const int32_t* index, int64_t n_rows,
                    int64_t width, int8_t* dst, int64_t lddst) {
  if (!src || !dst || !index) return -1;
  for (int64_t i = 0; i < n_rows; ++i)
    for (int64_t c = 0; c < width; ++c) dst[i * lddst + c] = src[(int64_t)index[i] * ldsrc + c];
  return 0;
}

int orc_token_mean(const int8_t* in, int64_t ldin, int64_t groups, int64_t T, int64_t C,
                   orc_scale scale, int8_t* out, int64_t ldout) {
  if (!in || !out || !scale_ok(scale) || scale.mult_c) return -1;
  for (int64_t g = 0; g < groups; ++g)
    for (int64_t c = 0; c < C; ++c) {
      int64_t s = 0;
      for (int64_t t = 0; t < T; ++t) s += in[(g * T + t) * ldin + c];
      out[g * ldout + c] = (int8_t)sat8(rq(s, scale.mult, scale.shift));
    }
  return 0;
}

int orc_vit_forward(const orc_vit_params* p, const int8_t* image, int32_t* logits, int8_t* x_last) {
  const int64_t B = p->B, T = p->T, D = p->D, np = T - 1, Kpe = 3 * p->patch * p->patch;
  const int64_t g = p->img / p->patch;
  if (g * g != np) return -1;
  std::vector<int8_t> patches((size_t)(B * np * Kpe)), X((size_t)(B * T * D)), Y((size_t)(B * T * D));
  int rc;
  if ((rc = orc_patchify(image, B, 3, p->img, p->img, p->patch, 0, patches.data()))) return rc;
  /* patch embedding as a Dense layer; position embedding enters through the
   * residual port; patch p of image b lands in row b*T + 1 + p */
  if ((rc = orc_linear(patches.data(), Kpe, p->Wpe, Kpe, p->bpe, p->pe_scale, p->pos, D, np,
                       p->pos_scale, X.data() + D, D, ORC_I8, np, T, B * np, D, Kpe))) return rc;
  for (int64_t b = 0; b < B; ++b) std::memcpy(X.data() + b * T * D, p->cls, (size_t)D);
  for (int64_t l = 0; l < p->depth; ++l) {
    if ((rc = orc_block_forward(&p->blocks[l], X.data(), Y.data()))) return rc;
    X.swap(Y);
  }
  if (x_last) std::memcpy(x_last, X.data(), (size_t)(B * T * D));
  /* final LayerNorm on the class-token rows, then the classifier */
  std::vector<int8_t> Z((size_t)(B * D));
  if ((rc = orc_layernorm(X.data(), ORC_I8, T * D, p->lnf_gamma, p->lnf_beta, p->blocks[0].M_ln,
                          Z.data(), D, B, D))) return rc;
  orc_scale none = {nullptr, nullptr, 1, 1};
  return orc_linear(Z.data(), D, p->Whead, D, p->bhead, p->head_scale, nullptr, 0, 1, none, logits,
                    p->classes, ORC_I32, 0, 0, B, p->classes, D);
}

}  /* extern "C" */
