/*
 * CPU oracle for the integer-only ViT encoder forward pass (I-ViT).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * single-precision-free (int64) restatement of the paper's integer pipeline,
 * written step by step in the paper's order and notation.  It shares no code,
 * header, table or helper with the CUDA library; only tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it.
 *
 * All pointers are HOST pointers owned by the caller.  All matrices are
 * row-major with a leading dimension given in elements.  Every function
 * returns 0 on success and a negative number when an argument violates a
 * stated bound (nothing is written in that case).
 *
 * Parity status: every primitive below is pinned by CPU tests against closed
 * forms, exact rational arithmetic, brute force or a float reference with a
 * committed numeric bound.  orc_block_forward, orc_vit_forward and the Python
 * composition oracle.api.swin_forward are pinned as compositions: each equals
 * the same model written out in the test from the pinned primitives with
 * plain numpy indexing (raster-order tokens, windows cut by slicing, np.roll
 * for the shifted windows, a strided slice for patch merging), mutations of
 * the outer layers are shown to break that equality, and a float64 shadow of
 * the block and of the whole ViT agrees within stated bounds.  There is no
 * published activation dump to compare with.
 */
#ifndef IVIT_ORACLE_H
#define IVIT_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_I8 = 0, ORC_I32 = 1 };

/* Requantisation scale.  Per-channel when mult_c != NULL (arrays of length N,
 * one dyadic number per output channel); otherwise the per-tensor pair
 * (mult, shift).  Dyadic number b / 2^c of Sec. 3.2: mult = b, shift = c. */
typedef struct {
  const int32_t* mult_c;
  const uint8_t* shift_c;
  int32_t mult;
  int32_t shift;
} orc_scale;

/* Constants of Algorithm 1 / 2: I0 = round(1/S_in), N = pre-shift of
 * ShiftExp, M = width of the IntDiv reciprocal, k_out = output bit width. */
typedef struct {
  int32_t I0, N, M, k_out;
} orc_exp_params;

/* ---- scalar primitives (exposed so tests can pin them one by one) ---- */

/* Sec. 3.2, Eq. (I_A) with rounding: floor((a*m + 2^(s-1)) / 2^s). */
int64_t orc_rq(int64_t a, int64_t m, int32_t s);
void orc_rq_array(const int64_t* a, int64_t n, int64_t m, int32_t s, int64_t* out);
/* Sec. 3.2, DN(): ratio > 0 -> (b, c) with b in [2^30, 2^31). */
int orc_dyadic_from_double(double ratio, int32_t* mult, int32_t* shift);
/* Algorithm 1, function ShiftExp, for I <= 0. */
int64_t orc_shiftexp(int64_t I, int64_t I0, int32_t N);
/* Eq. (IntDiv): (floor(2^M / I2) * I1) >> (M - (k-1)); 0 when I2 == 0. */
int64_t orc_intdiv(int64_t I1, int64_t I2, int32_t M, int32_t k);
/* Sec. 3.5, Eq. (iterative): integer square root, 10 iterations. */
int64_t orc_isqrt(int64_t n);
void orc_isqrt_array(const int64_t* n, int64_t count, int64_t* out);
/* The iteration exactly as printed (no monotone guard), for the test that
 * documents why the guarded reading is used. */
int64_t orc_isqrt_as_printed(int64_t n);

/* ---- tensor operations ---- */

/* Dense layer, Sec. 3.2:
 *   acc       = sum_k A[r,k]*W[c,k] + bias[c]
 *   v         = rq(acc; scale[c]) + (res ? rq(res[(r % res_rows), c]; res_scale) : 0)
 *   out[ro,c] = out_dtype == ORC_I8 ? sat8(v) : v
 * with ro = (r / out_group_rows) * out_group_stride + (r % out_group_rows)
 * (out_group_rows <= 0 means ro = r). */
int orc_linear(const int8_t* A, int64_t lda, const int8_t* W, int64_t ldw, const int32_t* bias,
               orc_scale scale, const int8_t* res, int64_t ldres, int64_t res_rows,
               orc_scale res_scale, void* out, int64_t ldo, int32_t out_dtype,
               int64_t out_group_rows, int64_t out_group_stride, int64_t M, int64_t N, int64_t K);

/* Batched MatMul, Sec. 3.2.  Batch index b = bo*batches_inner + bi; operand
 * base offsets are bo*stride_outer + bi*stride_inner (elements).
 *   C_b = sat8( rq( A_b (Ma x K) * op(B_b) + bias32[b % bias_batches]; scale ) )
 * transB != 0: B_b is [Nb, K] (C = A*B^T); transB == 0: B_b is [K, Nb]. */
int orc_matmul(const int8_t* A, int64_t lda, int64_t sAo, int64_t sAi, const int8_t* B, int64_t ldb,
               int64_t sBo, int64_t sBi, int32_t transB, const int32_t* bias32, int64_t ldbias,
               int64_t bias_batches, orc_scale scale, int8_t* C, int64_t ldc, int64_t sCo,
               int64_t sCi, int64_t batches_outer, int64_t batches_inner, int64_t Ma, int64_t Nb,
               int64_t K);

/* Algorithm 1 on each row.  in_dtype ORC_I8: rows are the int8 scores.
 * ORC_I32: x8 = sat8(rq(in32 + bias32[(row % bias_rows), :]; pre)) first. */
int orc_shiftmax(const void* in, int32_t in_dtype, int64_t ldin, const int32_t* bias32,
                 int64_t ldbias, int64_t bias_rows, orc_scale pre, orc_exp_params p, int8_t* out,
                 int64_t ldout, int64_t rows, int64_t d);

/* Algorithm 1 on each row of int32 scores with nothing in front: I_delta = in - max(in) (up to 33 bits),
 * ShiftExp with I0 = round(1 / S_in) <= 2^28, 64-bit sum, IntDiv with the caller's M (32..62) and k_out (2..8);
 * out int8 in [0, 2^(k_out-1) - 1].  Requires d * I0 * 2^N <= 2^(M-13). */
int orc_shiftmax_direct(const int32_t* in, int64_t ldin, orc_exp_params p, int8_t* out, int64_t ldout,
                        int64_t rows, int64_t d);

/* Algorithm 2 on each row (max over the row), then out = sat8(rq(I_in*I_div; post)). */
int orc_shiftgelu(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                  int64_t ldout, int64_t rows, int64_t cols);
/* Variant of Algorithm 2 (not the paper's): I_max is the constant I_p(127) = 212, the largest value I_p can
 * take for an int8 input, instead of the row maximum.  The sigmoid identity of Eq. (sigmoid) holds for any
 * I_max >= max I_p; only the integer precision differs.  The function is then element-wise. */
int orc_shiftgelu_static(const int8_t* in, int64_t ldin, orc_exp_params p, orc_scale post, int8_t* out,
                         int64_t ldout, int64_t rows, int64_t cols);

/* Sec. 3.5.  in_dtype ORC_I8 or ORC_I32 (|x| <= 2^20).
 *   mu = round-half-up(mean), y = x - mu, V = sum y^2, sd = isqrt(V),
 *   F = sd ? floor(2^M_ln / sd) : 0, out = sat8( rq(y*F; gamma_scale[c]) + beta[c] ). */
int orc_layernorm(const void* in, int32_t in_dtype, int64_t ldin, orc_scale gamma_scale,
                  const int32_t* beta, int32_t M_ln, int8_t* out, int64_t ldout, int64_t rows,
                  int64_t C);

/* ---- block and model composition (Sec. 3.1) ---- */

typedef struct {
  int64_t B, T, D, heads, H; /* B images (or windows) of T tokens; D = heads*d; H = MLP width */
  int32_t M_ln;
  orc_scale ln1_gamma; const int32_t* ln1_beta;
  const int8_t* Wqkv; const int32_t* bqkv; orc_scale qkv_scale; /* [3D,D]; Q|K|V thirds, head-major */
  orc_scale qk_scale; const int32_t* attn_bias; int64_t attn_bias_batches; /* [bb,T,T] or NULL */
  orc_exp_params smax; orc_scale pv_scale;
  const int8_t* Wo; const int32_t* bo; orc_scale o_scale; orc_scale res1_scale;
  orc_scale ln2_gamma; const int32_t* ln2_beta;
  const int8_t* W1; const int32_t* b1; orc_scale fc1_scale;
  orc_exp_params gelu; orc_scale gelu_post;
  const int8_t* W2; const int32_t* b2; orc_scale fc2_scale; orc_scale res2_scale;
  int32_t gelu_static_max; /* 0: Algorithm 2 (row maximum); 1: the static-maximum variant above */
} orc_block_params;

/* X, Y: [B*T, D] int8, contiguous. */
int orc_block_forward(const orc_block_params* p, const int8_t* X, int8_t* Y);

/* Attention core only (QK^T -> requant -> Shiftmax -> P*V -> requant) on a
 * QKV tensor [B*T, 3D]; O is [B*T, D].  Used by orc_block_forward. */
int orc_attention(const orc_block_params* p, const int8_t* QKV, int8_t* O);

/* img [B,C,Hi,Wi] int8 -> rows [B*(Hi/P)*(Wi/P), C*P*P], column order (c,py,px).
 * window > 0: rows of one image are emitted window-major (window x window
 * patches per window, windows in raster order, raster order inside). */
int orc_patchify(const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi, int64_t P,
                 int64_t window, int8_t* out);
/* dst[i, 0:width] = src[index[i], 0:width] */
int orc_gather_rows(const int8_t* src, int64_t ldsrc, const int32_t* index, int64_t n_rows,
                    int64_t width, int8_t* dst, int64_t lddst);
/* out[g, c] = sat8( rq( sum_t in[g*T + t, c]; scale ) ) */
int orc_token_mean(const int8_t* in, int64_t ldin, int64_t groups, int64_t T, int64_t C,
                   orc_scale scale, int8_t* out, int64_t ldout);

typedef struct {
  int64_t B, img, patch, T, D, depth, classes; /* T = (img/patch)^2 + 1 */
  const int8_t* Wpe; const int32_t* bpe; orc_scale pe_scale;  /* [D, 3*patch*patch] */
  const int8_t* pos; orc_scale pos_scale;                     /* [T-1, D], added via the residual port */
  const int8_t* cls;                                          /* [D], row 0 of every image */
  const orc_block_params* blocks;                             /* depth entries */
  orc_scale lnf_gamma; const int32_t* lnf_beta;
  const int8_t* Whead; const int32_t* bhead; orc_scale head_scale; /* [classes, D] */
} orc_vit_params;

/* image [B,3,img,img] int8 -> logits [B, classes] int32.  Optionally copies
 * the encoder output of the last block ([B*T, D]) to x_last when non-NULL. */
int orc_vit_forward(const orc_vit_params* p, const int8_t* image, int32_t* logits, int8_t* x_last);

int orc_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
