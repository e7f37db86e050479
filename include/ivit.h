/*
 * ivit.h - C ABI of the B200 (sm_100a) integer-only ViT encoder library.
 *
 * The library implements the integer pipeline of I-ViT ("Integer-only
 * Quantization for Efficient Vision Transformer Inference"): INT8xINT8->INT32
 * linear operations with dyadic requantisation (Sec. 3.2), Shiftmax
 * (Sec. 3.3, Algorithm 1), ShiftGELU (Sec. 3.4, Algorithm 2), I-LayerNorm
 * (Sec. 3.5) and their composition into an encoder block (Sec. 3.1).
 * No floating point is used on the device.
 *
 * Conventions (all entry points unless stated otherwise)
 *  - Every call returns IVIT_OK (0) or a negative IVIT_ERR_* code; nothing is
 *    enqueued when a call fails argument validation.
 *  - Tensor and parameter-array pointers are DEVICE pointers owned by the
 *    caller.  The operator, block and model entry points that take device
 *    buffers allocate no memory per call; scratch comes from a
 *    caller-provided workspace (ivit_*_workspace_bytes).  ivit_ctx_create
 *    allocates a few hundred KB once (status word, ShiftGELU table cache).
 *    Exceptions: ivit_vit_forward_host creates a stream and four events on
 *    its first call and, with graph replay switched on, instantiates CUDA
 *    graphs (which allocate on the device); ivit_ctx_profile_start creates
 *    its events on first use.
 *  - Work is enqueued on the CUDA stream held by the context; the entry
 *    points do not synchronise (ivit_ctx_profile_stop and ivit_ctx_destroy
 *    do).  Device-side failures (a bounded wait that ran out) are
 *    reported by ivit_ctx_poll_status after the stream has been synchronised.
 *  - A context belongs to one device; the caller keeps that device current
 *    (cudaSetDevice) while calling into the library with that context.
 *    Kernel attributes are set per device by ivit_ctx_create, so several
 *    contexts on several devices may live in one process.
 *  - Matrices are row-major; leading dimensions (ld*) and strides are in
 *    elements.  int8 tensors: pointer 16-byte aligned and ld a multiple of 16.
 *    int32 tensors: pointer 16-byte aligned and ld a multiple of 4.  Otherwise
 *    IVIT_ERR_ALIGNMENT.  A 197-wide int8 score matrix is therefore stored
 *    with ld = 208.
 *  - rq(a; m, s) = floor((a*m + 2^(s-1)) / 2^s) evaluated in 64 bits
 *    (round-half-up dyadic requantisation, Sec. 3.2 Eq. (I_A)).
 *    sat8(v) = min(127, max(-128, v)).
 *  - For every input there is exactly one correct output (integer arithmetic).
 */
#ifndef IVIT_H
#define IVIT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  IVIT_OK = 0,
  IVIT_ERR_INVALID_ARG = -1,    /* null pointer, negative size, bad enum */
  IVIT_ERR_ALIGNMENT = -2,      /* pointer or leading dimension not aligned as stated above */
  IVIT_ERR_RANGE = -3,          /* a quantisation constant violates a stated bound */
  IVIT_ERR_UNSUPPORTED = -4,    /* shape / dtype combination not built */
  IVIT_ERR_WORKSPACE = -5,      /* workspace missing, misaligned or too small */
  IVIT_ERR_CUDA = -6,           /* a CUDA runtime / driver call failed */
  IVIT_ERR_DEVICE_TIMEOUT = -7  /* a bounded device-side wait ran out (see ivit_ctx_poll_status) */
};

enum { IVIT_I8 = 0, IVIT_I32 = 1 };

typedef struct ivit_ctx ivit_ctx; /* opaque */

/* Dyadic number b / 2^c of Sec. 3.2 (DN()).  Per-channel when mult_c != NULL:
 * device arrays of one (mult, shift) per output channel.  Otherwise the
 * per-tensor pair (mult, shift), passed by value.  Bounds: 0 < mult < 2^31,
 * 31 <= shift <= 62, i.e. ratios below 1 (per-channel arrays are checked by
 * ivit_validate_scale at model-load time; kernels clamp the shift into
 * range).  With these bounds rq() of any int32 value fits 32 bits, so the
 * saturation that follows sees the exact value. */
typedef struct {
  const int32_t* mult_c;
  const uint8_t* shift_c;
  int32_t mult;
  int32_t shift;
} ivit_scale;

/* Constants of Algorithm 1 / Algorithm 2: I0 = round(1 / S_in); N = the
 * left pre-shift of ShiftExp (footnote of Algorithm 1); M = width of the
 * reciprocal in Eq. (IntDiv); k_out = output bit width (results are stored
 * as int8 in [0, 2^(k_out-1) - 1], scale 1 / 2^(k_out-1)).
 * Bounds (IVIT_ERR_RANGE otherwise): 1 <= I0 <= 2^15, 0 <= N <= 24, M == 45,
 * 2 <= k_out <= 8; Shiftmax: row_len * I0 * 2^N < 2^32 and I0 * 2^N >= 2^14;
 * ShiftGELU: 2 * I0 * 2^N < 2^32.  ivit_shiftmax_direct has wider bounds of
 * its own. */
typedef struct {
  int32_t I0, N, M, k_out;
} ivit_exp_params;

/* ---- context ---- */

/* Dense layers with a long contraction (K >= 1024, output channels a multiple of 256, enough rows to give every pair of
 * SMs a tile of 256 x 256, int8 output in one of the staged forms) run on pairs of CTAs: two SMs share a tile of 256 channels x 256 rows (tcgen05
 * cta_group::2; a CUDA implementation choice, the paper has no counterpart), each loading its own 128 weight rows and
 * half of the activation rows.  On by default; results are identical in both modes.  enable: 0 = off, non-zero = on.
 * Host graphs kept by the context are dropped.  Returns IVIT_OK, or IVIT_ERR_INVALID_ARG for a null context. */
int ivit_ctx_set_gemm_pairs(ivit_ctx* ctx, int enable);

/* Creates a context on `device` that enqueues on `cuda_stream` (a
 * cudaStream_t; NULL = the legacy default stream).  Fails with IVIT_ERR_CUDA
 * when no usable sm_100 device is present: there is no CPU fallback. */
int ivit_ctx_create(ivit_ctx** ctx, int device, void* cuda_stream);
int ivit_ctx_destroy(ivit_ctx* ctx);
int ivit_ctx_set_stream(ivit_ctx* ctx, void* cuda_stream);
/* Non-blocking: IVIT_OK, or the last device-side error recorded by a kernel
 * of this context (cleared by the call). */
int ivit_ctx_poll_status(ivit_ctx* ctx);
/* Number of kernels this context has launched since creation. */
int64_t ivit_ctx_launch_count(const ivit_ctx* ctx);
/* How many of those were Dense launches on CTA pairs (ivit_ctx_set_gemm_pairs); 0 for a null context. */
int64_t ivit_ctx_pair_launch_count(const ivit_ctx* ctx);
/* ShiftGELU look-up tables (one per parameter set: I0, N, M, k_out, post) are built on first use and cached in
 * the context, 16 sets at a time, the oldest slot being rebuilt for a 17th.  This counter changes whenever a slot
 * is built or rebuilt.  A CUDA graph that the CALLER captured around library calls holds the addresses of the
 * tables those calls used: it stays valid while this counter keeps the value it had when the capture ended, and
 * must be captured again otherwise (or keep the models that share a context to at most 16 parameter sets).  The
 * library's own graphs (ivit_ctx_set_host_graph) check this themselves. */
uint64_t ivit_ctx_table_generation(const ivit_ctx* ctx);
/* Selects the GEMM engine: 0 = tcgen05 tensor-core kernels where the shape
 * qualifies (default), 1 = force the CUDA-core (dp4a) kernels everywhere.
 * Both are bit-exact; the switch exists for testing and measurement. */
int ivit_ctx_set_gemm_engine(ivit_ctx* ctx, int engine);
/* Row-operator fusion (off by default).  1: inside ivit_block_forward and the model forwards, LayerNorm 2, ShiftGELU
 * (Algorithm 2 with its row maximum) and the LayerNorm 1 of the following block run inside the Dense kernel that
 * produces their input rows, where the shapes allow it: the kernel's warps count the finished channel tiles of every
 * block of rows and, after their last tile, run the operator on slices of the completed rows.  0: every operator
 * is a kernel of its own.  Both give the same bytes.  On the measured workloads the separate kernels, whose launch
 * overlaps the previous kernel's tail, are as fast or faster, which is why they are the default.  (2 / 4 switch on
 * the LayerNorm / ShiftGELU part alone, for measurements.) */
int ivit_ctx_set_row_fusion(ivit_ctx* ctx, int enable);
const char* ivit_strerror(int code);

/* ---- Sec. 3.2: Dense layer with dyadic requantisation ----
 *   acc        = sum_k A[r,k] * W[c,k] + (bias ? bias[c] : 0)          (int32)
 *   v          = rq(acc; scale[c]) + (res ? rq(res[r % res_rows, c]; res_scale) : 0)
 *   out[ro, c] = out_dtype == IVIT_I8 ? sat8(v) : v
 *   ro         = out_group_rows > 0 ? (r / out_group_rows) * out_group_stride + r % out_group_rows : r
 * A [M,K] int8, W [N,K] int8 (one row per output channel), bias int32 [N] or
 * NULL, res int8 [res_rows, N] or NULL (res_scale per-tensor), out int8 or
 * int32 [*, N].  K <= 65536 so the accumulator cannot overflow; K % 16 == 0.
 * The output-row grouping lets the patch embedding write token rows 1..T-1 of
 * every image directly. */
int ivit_linear(ivit_ctx* ctx, const int8_t* A, int64_t lda, const int8_t* W, int64_t ldw,
                const int32_t* bias, ivit_scale scale, const int8_t* res, int64_t ldres,
                int64_t res_rows, ivit_scale res_scale, void* out, int64_t ldo, int32_t out_dtype,
                int64_t out_group_rows, int64_t out_group_stride, int64_t M, int64_t N, int64_t K);

/* ---- Sec. 3.2: batched MatMul with dyadic requantisation ----
 * Batch b = bo * batches_inner + bi; operand bases are offset by
 * bo * s?o + bi * s?i elements (two-level strides address one head of one
 * image inside a [tokens, 3D] QKV tensor without a copy).
 *   C_b = sat8( rq( A_b (Ma x K) * op(B_b) + bias32[b % bias_batches]; scale ) )
 * transB != 0: B_b is [Nb, K] and C = A * B^T (scores Q K^T); transB == 0:
 * B_b is [K, Nb] (attention times V).  bias32 int32 [bias_batches, Ma, ldbias]
 * or NULL; scale per-tensor.  All offsets must keep 4-byte alignment
 * (strides and ld multiples of 4); K arbitrary. */
int ivit_matmul(ivit_ctx* ctx, const int8_t* A, int64_t lda, int64_t sAo, int64_t sAi,
                const int8_t* B, int64_t ldb, int64_t sBo, int64_t sBi, int32_t transB,
                const int32_t* bias32, int64_t ldbias, int64_t bias_batches, ivit_scale scale,
                int8_t* C, int64_t ldc, int64_t sCo, int64_t sCi, int64_t batches_outer,
                int64_t batches_inner, int64_t Ma, int64_t Nb, int64_t K);

/* ---- Sec. 3.3, Algorithm 1: Shiftmax over each row ----
 * in_dtype IVIT_I8: rows of int8 scores.  IVIT_I32: rows of int32
 * accumulators, x8 = sat8(rq(in32 + bias32[row % bias_rows, :]; pre)) first
 * (bias32 may be NULL), which is bit-identical to requantising to int8 and
 * then calling the int8 form.  out int8 in [0, 2^(k_out-1) - 1]
 * (Eq. (IntDiv), S_out = 1/2^(k_out-1); [0, 127] at k_out = 8).  Columns d .. roundup(d,16)-1 of out
 * are written as 0.  1 <= d <= 8192. */
int ivit_shiftmax(ivit_ctx* ctx, const void* in, int32_t in_dtype, int64_t ldin,
                  const int32_t* bias32, int64_t ldbias, int64_t bias_rows, ivit_scale pre,
                  ivit_exp_params p, int8_t* out, int64_t ldout, int64_t rows, int64_t d);

/* ---- Sec. 3.3, Algorithm 1 on int32 scores with no requantisation in front ----
 * The general form of the algorithm: in is int32 [rows, ldin] (for instance
 * the accumulators of Q K^T at scale S_in), I_delta = in - max(in) takes up to
 * 33 bits, I0 = round(1 / S_in) may be as large as 2^28, exponentials and
 * their sum are 64-bit, and the caller chooses M.  out int8 [rows, ldout] in
 * [0, 2^(k_out-1) - 1]; columns d .. roundup(d,16)-1 are written as 0.
 * Bounds (IVIT_ERR_RANGE otherwise): 1 <= I0 <= 2^28, 0 <= N <= 24,
 * 32 <= M <= 62, 2 <= k_out <= 8, d * I0 * 2^N <= 2^(M-13) (so that the
 * reciprocal floor(2^M / sum) keeps at least 13 bits).  1 <= d <= 8192,
 * ldin % 4 == 0, ldout % 16 == 0, both pointers 16-byte aligned (device). */
int ivit_shiftmax_direct(ivit_ctx* ctx, const int32_t* in, int64_t ldin, ivit_exp_params p,
                         int8_t* out, int64_t ldout, int64_t rows, int64_t d);

/* ---- Sec. 3.4, Algorithm 2: ShiftGELU over each row, then requantisation ----
 *   I_p = x + (x>>1) + (x>>3) + (x>>4); I_max = max(0, max_row I_p);
 *   I_div = IntDiv(ShiftExp(I_p - I_max), ShiftExp(I_p - I_max) + ShiftExp(-I_max), k_out)
 *   out = sat8( rq(x * I_div; post) )            (post per-tensor)
 * in == out (in place) is allowed.  cols % 16 == 0, cols <= 16384. */
int ivit_shiftgelu(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p,
                   ivit_scale post, int8_t* out, int64_t ldout, int64_t rows, int64_t cols);
/* Variant of Algorithm 2 that is NOT the paper's function: I_max is the constant I_p(127) = 212
 * (the largest value I_p takes for an int8 input) instead of the row maximum.  The sigmoid identity
 * behind Algorithm 2 holds for any I_max >= max I_p, only the integer precision of the two
 * exponentials differs (outputs differ from ivit_shiftgelu by at most a few steps, and are equal on
 * rows that contain 127).  The function is element-wise, which lets ivit_block_forward apply it
 * inside the FC1 epilogue (ivit_block_params.gelu_static_max).  Arguments as for ivit_shiftgelu. */
int ivit_shiftgelu_static(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p,
                          ivit_scale post, int8_t* out, int64_t ldout, int64_t rows, int64_t cols);

/* ---- Sec. 3.5: I-LayerNorm over each row ----
 *   mu = floor((2*sum x + C) / (2C)); y = x - mu; V = sum y^2;
 *   sd = integer sqrt of V: the value of Eq. (iterative) with 10 guarded iterations, floor(sqrt(V)) (int8 rows
 *        of up to 1024 channels take it bit by bit without divisions, see ivit_isqrt_range);
 *   F = sd ? floor(2^M_ln / sd) : 0;
 *   out[c] = sat8( rq(y[c] * F; gamma_scale[c]) + beta[c] )
 * gamma_scale per-channel or per-tensor; beta int32 [C] or NULL.
 * in_dtype IVIT_I8, or IVIT_I32 with |x| <= 2^20.  8 <= M_ln <= 29 (so that y * F fits 32 bits).
 * C % 4 == 0, C <= 16384. */
int ivit_layernorm(ivit_ctx* ctx, const void* in, int32_t in_dtype, int64_t ldin,
                   ivit_scale gamma_scale, const int32_t* beta, int32_t M_ln, int8_t* out,
                   int64_t ldout, int64_t rows, int64_t C);

/* ---- Sec. 3.1: one encoder block ----
 *   X^ = MSA(LayerNorm(X)) + X ;  Y = MLP(LayerNorm(X^)) + X^
 * with every arrow an int8 tensor: LN -> QKV Dense -> per head
 * [Q K^T (+attn_bias) -> rq(qk_scale) -> sat8 -> Shiftmax -> P V -> rq(pv_scale) -> sat8]
 * -> output Dense + rq(X; res1_scale) -> LN -> FC1 -> ShiftGELU -> FC2 + rq(X^; res2_scale).
 * B images (or attention windows) of T tokens; D = heads * d, d % 16 == 0;
 * H = MLP width.  Wqkv is [3D, D]: Q | K | V thirds, head-major inside each.
 * attn_bias int32 [attn_bias_batches, T, T] (row stride T) or NULL; batch
 * (b*heads + h) uses entry (b*heads + h) % attn_bias_batches. */
typedef struct {
  int64_t B, T, D, heads, H;
  int32_t M_ln;
  ivit_scale ln1_gamma; const int32_t* ln1_beta;
  const int8_t* Wqkv; const int32_t* bqkv; ivit_scale qkv_scale;
  ivit_scale qk_scale; const int32_t* attn_bias; int64_t attn_bias_batches;
  ivit_exp_params smax; ivit_scale pv_scale;
  const int8_t* Wo; const int32_t* bo; ivit_scale o_scale; ivit_scale res1_scale;
  ivit_scale ln2_gamma; const int32_t* ln2_beta;
  const int8_t* W1; const int32_t* b1; ivit_scale fc1_scale;
  ivit_exp_params gelu; ivit_scale gelu_post;
  const int8_t* W2; const int32_t* b2; ivit_scale fc2_scale; ivit_scale res2_scale;
  /* 0: ShiftGELU as Algorithm 2 (row maximum, a kernel of its own between FC1 and FC2).
   * 1: the static-maximum variant of ivit_shiftgelu_static, applied inside the FC1 epilogue. */
  int32_t gelu_static_max;
} ivit_block_params;

size_t ivit_block_workspace_bytes(const ivit_block_params* p);
/* X, Y: [B*T, D] int8 contiguous (ld = D); X == Y is not allowed.  workspace:
 * device memory, 256-byte aligned, at least ivit_block_workspace_bytes(p). */
int ivit_block_forward(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* X, int8_t* Y,
                       void* workspace, size_t workspace_bytes);

/* ivit_block_forward for callers that cannot allocate device memory.
 * (The paper has no counterpart; this entry point exists for deployment reasons only.)
 * Some callers are not allowed to call cudaMalloc at all: a plugin running inside a host
 * application that owns the memory pool, code that runs where allocation would synchronise the
 * device (inside a latency-critical serving loop), or a process whose allocator is locked down.
 * Such a caller cannot provide the workspace that ivit_block_forward asks for.  This variant
 * computes the same block with the same kernels, but takes its scratch from a fixed array that is
 * part of the library image: IVIT_STATIC_SCRATCH_BYTES bytes of device memory, which every GPU
 * that loads the library holds until the process exits, whether or not this call is ever used.
 *  - X, Y: [B*T, D] int8 device tensors owned by the caller, as for ivit_block_forward.
 *  - Returns IVIT_ERR_WORKSPACE, and enqueues nothing, when ivit_block_workspace_bytes(p)
 *    exceeds IVIT_STATIC_SCRATCH_BYTES (the DeiT-Tiny block of one image needs about 0.6 MiB).
 *  - The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *  - The first call on a device looks up the array's device address (one cudaGetSymbolAddress, no
 *    allocation); make that first call before any CUDA stream capture.
 *  - All calls share the one array and it keeps whatever the last call left in it.  No part of it
 *    has to start at zero: every buffer inside is fully written before it is read.  Two calls whose
 *    kernels overlap on the GPU (different streams, different contexts, different host threads)
 *    race on the array; keep them ordered on one stream. */
#define IVIT_STATIC_SCRATCH_BYTES (8u << 20)
int ivit_block_forward_static(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* X, int8_t* Y);

/* Attention core of the block alone (Sec. 3.1 MSA equation without the output
 * projection): QKV [B*T, 3D] int8 -> O [B*T, D] int8, using the attention
 * fields of p.  workspace as for ivit_block_forward. */
int ivit_attention(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O,
                   void* workspace, size_t workspace_bytes);

/* ---- full ViT-family forward (patch embedding, class token, blocks, head) ----
 * The paper does not describe these outer layers; they are Dense / LayerNorm
 * instances of the operators above:  patches -> Dense(Wpe) + rq(pos) -> rows
 * 1..T-1 of each image; row 0 = cls; depth blocks; LayerNorm of the class row;
 * Dense(Whead) -> int32 logits rq(acc + b; head_scale) (not saturated). */
typedef struct {
  int64_t B, img, patch, T, D, depth, classes;   /* T = (img/patch)^2 + 1 */
  const int8_t* Wpe; const int32_t* bpe; ivit_scale pe_scale;   /* [D, 3*patch*patch] */
  const int8_t* pos; ivit_scale pos_scale;                      /* [T-1, D] */
  const int8_t* cls;                                            /* [D] */
  const ivit_block_params* blocks;                              /* HOST array of depth entries */
  ivit_scale lnf_gamma; const int32_t* lnf_beta;
  const int8_t* Whead; const int32_t* bhead; ivit_scale head_scale; /* [classes, D] */
} ivit_vit_params;

size_t ivit_vit_workspace_bytes(const ivit_vit_params* p);
/* image [B,3,img,img] int8 -> logits [B, classes] int32 (ld = classes). */
int ivit_vit_forward(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image, int32_t* logits,
                     void* workspace, size_t workspace_bytes);

/* The same forward, additionally copying the output of the last encoder block, [B*T, D] int8 (ld = D), to
 * `tokens` (device, 16-byte aligned; NULL: no copy).  The class rows of that tensor are what the final LayerNorm
 * and the classifier read; the other rows reach no logit, so this is the call that lets a caller (or a parity
 * test) see every byte the encoder produced. */
int ivit_vit_forward_tokens(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image, int32_t* logits,
                            int8_t* tokens, void* workspace, size_t workspace_bytes);

/* Same forward with HOST buffers: copies image_host to a staging area in the workspace, runs
 * ivit_vit_forward, and copies the logits back to logits_host.  The call only enqueues work and
 * returns: the caller synchronises the context's stream before reading logits_host, and both host
 * buffers must stay valid (and the image unchanged) until then.  The input copy runs on a stream
 * of the context's own into one of two staging buffers used alternately, so the copy of one call
 * overlaps the compute of the call before it when calls are enqueued back to back (pinned host
 * memory is needed for that overlap; pageable memory works but copies synchronously).  The first
 * call on a context creates that stream and its events.  All calls on one context must use the
 * same workspace.  workspace must hold ivit_vit_host_workspace_bytes(p). */
size_t ivit_vit_host_workspace_bytes(const ivit_vit_params* p);
int ivit_vit_forward_host(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image_host,
                          int32_t* logits_host, void* workspace, size_t workspace_bytes);

/* ---- Swin-shaped forward (window attention, patch merging, token pooling) ----
 * The paper names Swin as a benchmark model without describing its outer layers; they are instances of the
 * operators above.  Token rows are WINDOW-MAJOR everywhere (windows of one image in raster order, raster order
 * inside a window), so that every window is a contiguous run of window^2 rows:
 *   patches (window-major) -> Dense(Wpe) -> LayerNorm -> for every stage [ blocks -> (not after the last stage)
 *   2x2 merge: gather_rows(merge_index) viewed as [rows / 4, 4C] -> LayerNorm -> Dense(Wmerge) ] ->
 *   LayerNorm -> token mean (rq with pool_scale, sat8) -> Dense(Whead) -> int32 logits (not saturated).
 * A block with shifted[i] != 0 is a shifted-window block: its input rows are permuted by shift_index before
 * the block and its output rows by unshift_index after it (the cyclic roll as a row gather; the attention mask
 * is part of the block's attn_bias).  Every block of stage s has B * (res / window)^2 windows of window^2
 * tokens, D = C, and the heads / MLP width the caller chose. */
typedef struct {
  int64_t C, res, depth;                      /* channels, tokens per image side, blocks */
  const ivit_block_params* blocks;            /* HOST array of depth entries */
  const uint8_t* shifted;                     /* HOST array of depth flags, or NULL (no shifted block) */
  const int32_t* shift_index;                 /* device int32 [B*res*res] or NULL */
  const int32_t* unshift_index;               /* device int32 [B*res*res] or NULL */
  const int32_t* merge_index;                 /* device int32 [B*res*res]; NULL after the last stage */
  ivit_scale merge_ln_gamma; const int32_t* merge_ln_beta;   /* 4C channels */
  const int8_t* Wmerge; ivit_scale merge_scale;              /* [2C, 4C], no bias */
} ivit_swin_stage;

typedef struct {
  int64_t B, img, patch, window, classes, n_stages;
  int32_t M_ln;
  const int8_t* Wpe; const int32_t* bpe; ivit_scale pe_scale;   /* [C0, 3*patch*patch] */
  ivit_scale pe_ln_gamma; const int32_t* pe_ln_beta;
  const ivit_swin_stage* stages;                                /* HOST array of n_stages entries */
  ivit_scale lnf_gamma; const int32_t* lnf_beta;
  ivit_scale pool_scale;                                        /* per-tensor, 1 / tokens folded in */
  const int8_t* Whead; const int32_t* bhead; ivit_scale head_scale;   /* [classes, C_last] */
} ivit_swin_params;

size_t ivit_swin_workspace_bytes(const ivit_swin_params* p);
/* image [B,3,img,img] int8 (device) -> logits [B, classes] int32 (device, ld = classes).  tokens: NULL, or a
 * device buffer [B * res_last^2, C_last] int8 that receives the output of the last block (what the final
 * LayerNorm reads).  Nothing is allocated: every intermediate lives in the workspace (device, 256-byte aligned,
 * at least ivit_swin_workspace_bytes(p)). */
int ivit_swin_forward(ivit_ctx* ctx, const ivit_swin_params* p, const int8_t* image, int32_t* logits,
                      int8_t* tokens, void* workspace, size_t workspace_bytes);
/* The same with HOST buffers: image_host is copied to one of two staging areas of the workspace (on a copy stream of
 * the context, so that the copy overlaps the previous call's compute), the forward runs, the logits are copied back
 * to logits_host; the call only enqueues (synchronise the stream
 * before reading logits_host; keep both host buffers valid until then; pinned memory makes the copies
 * asynchronous).  workspace must hold ivit_swin_host_workspace_bytes(p). */
size_t ivit_swin_host_workspace_bytes(const ivit_swin_params* p);
int ivit_swin_forward_host(ivit_ctx* ctx, const ivit_swin_params* p, const int8_t* image_host,
                           int32_t* logits_host, void* workspace, size_t workspace_bytes);

/* Graph replay for ivit_vit_forward_host and ivit_swin_forward_host (off by default).  When enabled, the third call in a row that repeats
 * the same model description (every field of p, of its stages and of its blocks), workspace and stream captures the device part
 * of the forward into a CUDA graph, and later calls launch that graph instead of about a hundred kernels; any
 * change of those arguments, a new stream, or switching the mode off drops the graph.  Needs a stream other than
 * the legacy default stream (with the default stream the kernels keep being launched one by one).  Tensors the
 * model description points to may change contents between calls; they must stay at the same addresses.
 * Results are identical in both modes: a graph is dropped, and captured again later, when another call on the
 * context has rebuilt a slot of the ShiftGELU table cache since the capture (see ivit_ctx_table_generation). */
int ivit_ctx_set_host_graph(ivit_ctx* ctx, int enable);
/* Number of graphs currently instantiated for ivit_vit_forward_host (0, 1 or 2: one per staging buffer). */
int ivit_ctx_host_graph_count(ivit_ctx* ctx);

/* ---- per-kernel timing (measurement aid; not part of the paper's method) ----
 * Between profile_start and profile_stop every kernel the context launches is bracketed by a pair
 * of CUDA events on the context's stream (at most 8192 launches per session; later ones are not
 * recorded).  profile_stop synchronises the stream and returns the number of records (or a
 * negative error).  profile_get returns record idx: the kernel class (ivit_kernel_kind_name),
 * its device time in milliseconds and its algorithmic work (int8 ops for GEMMs, bytes moved for
 * the other kernels). */
int ivit_ctx_profile_start(ivit_ctx* ctx);
int ivit_ctx_profile_stop(ivit_ctx* ctx);
int ivit_ctx_profile_get(ivit_ctx* ctx, int32_t idx, int32_t* kind, float* ms, double* work);
const char* ivit_kernel_kind_name(int32_t kind);

/* Issue-only ceiling of the int8 tensor cores (measurement aid; the paper has no counterpart): one CTA per SM
 * issues `iters` x 4 tcgen05.mma.kind::i8 instructions of shape M128 x N256 x K32 on operands that stay in
 * shared memory, with no loads and no epilogue.  Runs the kernel twice on the context's stream (the second
 * launch is timed with CUDA events), SYNCHRONISES the stream, and returns the time in milliseconds and the int8
 * operations (2 per multiply-accumulate) of the timed launch; ops / ms is the rate the Dense kernels' TOP/s are
 * measured against.  1 <= iters <= 2^20. */
int ivit_probe_int8_mma(ivit_ctx* ctx, int32_t iters, float* ms, double* ops);

/* Verification aid for Sec. 3.5: out[i] = the integer square root that the I-LayerNorm kernels compute for the
 * radicand n0 + i, i < count (device uint16 array; n0 + count <= 2^26, the largest sum of squared deviations of
 * an int8 row of 1024 channels).  The kernels take the root bit by bit instead of running Eq. (iterative); a test
 * compares this routine with the iteration over the whole range. */
int ivit_isqrt_range(ivit_ctx* ctx, uint32_t n0, uint32_t count, uint16_t* out);

/* ---- data movement helpers (not in the paper; needed by the full models) ---- */

/* img [B,C,Hi,Wi] int8 -> rows [B*(Hi/P)*(Wi/P), C*P*P], column order
 * (c, py, px).  window > 0: rows of one image are emitted window-major. */
int ivit_patchify(ivit_ctx* ctx, const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi,
                  int64_t P, int64_t window, int8_t* out, int64_t ldout);
/* dst[i, 0:width] = src[index[i], 0:width]; width % 16 == 0; index int32 on device. */
int ivit_gather_rows(ivit_ctx* ctx, const int8_t* src, int64_t ldsrc, const int32_t* index,
                     int64_t n_rows, int64_t width, int8_t* dst, int64_t lddst);
/* dst[g * group_stride + 0:width] = src_row[0:width] for g < groups (class-token rows). */
int ivit_fill_rows(ivit_ctx* ctx, const int8_t* src_row, int64_t width, int8_t* dst,
                   int64_t group_stride, int64_t groups);
/* out[g, c] = sat8( rq( sum_{t<T} in[g*T + t, c]; scale ) )  (token pooling, 1/T folded in scale) */
int ivit_token_mean(ivit_ctx* ctx, const int8_t* in, int64_t ldin, int64_t groups, int64_t T,
                    int64_t C, ivit_scale scale, int8_t* out, int64_t ldout);

/* ---- host-only helpers (offline) ---- */

/* Sec. 3.2, DN(): 0 < ratio < 1 -> mult in [2^30, 2^31), shift in [31, 62]. */
int ivit_dyadic_from_double(double ratio, int32_t* mult, int32_t* shift);
/* Checks the bounds listed at ivit_exp_params. */
int ivit_validate_exp_params(ivit_exp_params p, int64_t row_len, int32_t is_gelu);
/* Checks a HOST copy of a per-channel scale: 0 < mult, 31 <= shift <= 62. */
int ivit_validate_scale(const int32_t* mult_host, const uint8_t* shift_host, int64_t n);

#ifdef __cplusplus
}
#endif
#endif /* IVIT_H */
