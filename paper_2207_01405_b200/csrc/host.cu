// Host side of the C ABI: context, argument validation, operator entry points and the
// composition of one encoder block / one ViT forward out of the kernels (Sec. 3.1).
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

using namespace ivit;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int64_t round16(int64_t v) { return (v + 15) / 16 * 16; }

int check_exp(ivit_exp_params p, int64_t row_len, bool gelu) {
  if (p.I0 < 1 || p.I0 > (1 << 15) || p.N < 0 || p.N > 24 || p.M != 45 || p.k_out < 2 || p.k_out > 8) return IVIT_ERR_RANGE;
  const int64_t top = (int64_t)p.I0 << p.N;
  if (gelu) {
    if (2 * top > 4294967295LL) return IVIT_ERR_RANGE;
  } else {
    if (row_len * top > 4294967295LL || top < (1 << 14)) return IVIT_ERR_RANGE;
  }
  return IVIT_OK;
}

struct BlockWs {
  size_t A, QKV, S, P, O, Xh, G, total;
  int64_t ldS;
};

BlockWs block_ws(const ivit_block_params* p) {
  BlockWs w;
  const size_t M = (size_t)(p->B * p->T), D = (size_t)p->D, H = (size_t)p->H;
  w.ldS = round16(p->T);
  const size_t s_bytes = (size_t)(p->B * p->heads * p->T) * (size_t)w.ldS;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.A = take(M * D);
  w.QKV = take(M * 3 * D);
  w.S = take(s_bytes);
  w.P = take(s_bytes);
  w.O = take(M * D);
  w.Xh = take(M * D);
  w.G = take(M * H);
  w.total = off;
  return w;
}

int check_block(const ivit_block_params* p) {
  if (!p || p->B < 0 || p->T < 1 || p->D < 16 || p->heads < 1 || p->H < 16) return IVIT_ERR_INVALID_ARG;
  if (p->D % p->heads) return IVIT_ERR_INVALID_ARG;
  const int64_t d = p->D / p->heads;
  if (d % 16 || p->D % 16 || p->H % 16) return IVIT_ERR_UNSUPPORTED;
  if (!p->Wqkv || !p->Wo || !p->W1 || !p->W2) return IVIT_ERR_INVALID_ARG;
  if (p->M_ln < 8 || p->M_ln > 29) return IVIT_ERR_RANGE;
  const ivit_scale* sc[] = {&p->ln1_gamma, &p->qkv_scale, &p->qk_scale, &p->pv_scale, &p->o_scale, &p->res1_scale,
                            &p->ln2_gamma, &p->fc1_scale, &p->gelu_post, &p->fc2_scale, &p->res2_scale};
  for (const ivit_scale* s : sc)
    if (!scale_ok(*s)) return IVIT_ERR_RANGE;
  if (p->qk_scale.mult_c || p->pv_scale.mult_c || p->res1_scale.mult_c || p->res2_scale.mult_c || p->gelu_post.mult_c)
    return IVIT_ERR_INVALID_ARG;
  if (p->attn_bias && p->attn_bias_batches < 1) return IVIT_ERR_INVALID_ARG;
  int rc = check_exp(p->smax, p->T, false);
  if (rc) return rc;
  return check_exp(p->gelu, p->H, true);
}

GemmProblem linear_problem(const int8_t* A, int64_t lda, const int8_t* W, int64_t ldw, const int32_t* bias,
                           ivit_scale scale, const int8_t* res, int64_t ldres, int64_t res_rows,
                           ivit_scale res_scale, void* out, int64_t ldo, int out_dtype, int64_t group_rows,
                           int64_t group_stride, int64_t M, int64_t N, int64_t K) {
  GemmProblem g{};
  g.A = A; g.lda = lda; g.B = W; g.ldb = ldw; g.transB = 1;
  g.batches_outer = g.batches_inner = 1;
  g.M = M; g.N = N; g.K = K;
  g.epi.bias = bias;
  g.epi.bias32 = nullptr; g.epi.ldbias = 0; g.epi.bias_batches = 1;
  g.epi.scale = to_dev(scale);
  g.epi.res = res; g.epi.ldres = ldres; g.epi.res_rows = res_rows < 1 ? 1 : res_rows;
  g.epi.res_scale = to_dev(res_scale);
  g.epi.out = out; g.epi.ldo = ldo; g.epi.out_dtype = out_dtype;
  g.epi.group_rows = group_rows; g.epi.group_stride = group_stride;
  return g;
}

int attention_impl(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O, char* ws, const BlockWs& w) {
  if (ctx->gemm_engine == 0) {
    const int rc = launch_attention_fused(ctx, p, QKV, O);
    if (rc != IVIT_ERR_UNSUPPORTED) return rc;
  }
  const int64_t B = p->B, T = p->T, D = p->D, h = p->heads, d = D / h, ldq = 3 * D, ldS = w.ldS;
  int8_t* S = reinterpret_cast<int8_t*>(ws + w.S);
  int8_t* P = reinterpret_cast<int8_t*>(ws + w.P);
  // scores: Q_i K_i^T (+ bias), requantised to int8; 1/sqrt(d) lives in qk_scale
  GemmProblem qk{};
  qk.A = QKV; qk.lda = ldq; qk.sAo = T * ldq; qk.sAi = d;
  qk.B = QKV + D; qk.ldb = ldq; qk.sBo = T * ldq; qk.sBi = d; qk.transB = 1;
  qk.sCo = h * T * ldS; qk.sCi = T * ldS;
  qk.batches_outer = B; qk.batches_inner = h; qk.M = T; qk.N = T; qk.K = d;
  qk.epi.bias32 = p->attn_bias; qk.epi.ldbias = T; qk.epi.bias_batches = p->attn_bias ? p->attn_bias_batches : 1;
  qk.epi.scale = to_dev(p->qk_scale); qk.epi.res_rows = 1;
  qk.epi.out = S; qk.epi.ldo = ldS; qk.epi.out_dtype = IVIT_I8;
  int rc = launch_gemm(ctx, qk);
  if (rc) return rc;
  rc = launch_shiftmax(ctx, S, IVIT_I8, ldS, nullptr, 0, 1, ScaleDev{nullptr, nullptr, 1, 1}, p->smax, P, ldS, B * h * T, T);
  if (rc) return rc;
  // Attn_i = P_i V_i, heads concatenated along the feature dimension
  GemmProblem pv{};
  pv.A = P; pv.lda = ldS; pv.sAo = h * T * ldS; pv.sAi = T * ldS;
  pv.B = QKV + 2 * D; pv.ldb = ldq; pv.sBo = T * ldq; pv.sBi = d; pv.transB = 0;
  pv.sCo = T * D; pv.sCi = d;
  pv.batches_outer = B; pv.batches_inner = h; pv.M = T; pv.N = d; pv.K = T;
  pv.epi.bias_batches = 1; pv.epi.res_rows = 1;
  pv.epi.scale = to_dev(p->pv_scale);
  pv.epi.out = O; pv.epi.ldo = D; pv.epi.out_dtype = IVIT_I8;
  return launch_gemm(ctx, pv);
}

// Asks the Dense launch `g` to run I-LayerNorm (gamma, beta) on its finished output rows, writing `out` (ld = C).
void want_layernorm(GemmProblem& g, const ivit_scale& gamma, const int32_t* beta, int M_ln, int8_t* out, int64_t ld) {
  g.epi.rop.kind = 1;
  g.epi.rop.gs = to_dev(gamma);
  g.epi.rop.beta = beta;
  g.epi.rop.M_ln = M_ln;
  g.epi.rop.ln_out = out;
  g.epi.rop.ld_ln = ld;
}

// One encoder block.  a_ready: LayerNorm 1 of X already sits in the workspace (the previous block's last Dense
// layer produced it); next: the block that follows on Y with the same shape, or nullptr - its LayerNorm 1 is then
// run in the tail of this block's last Dense layer, where that is possible.  *a_next_ready tells the caller whether
// it was.  Row operators that a Dense kernel cannot take on run as kernels of their own, with the same result.
int block_impl(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* X, int8_t* Y, char* ws, bool a_ready = false,
               const ivit_block_params* next = nullptr, bool* a_next_ready = nullptr) {
  const BlockWs w = block_ws(p);
  const int64_t M = p->B * p->T, D = p->D, H = p->H;
  int8_t* A = reinterpret_cast<int8_t*>(ws + w.A);
  int8_t* QKV = reinterpret_cast<int8_t*>(ws + w.QKV);
  int8_t* O = reinterpret_cast<int8_t*>(ws + w.O);
  int8_t* Xh = reinterpret_cast<int8_t*>(ws + w.Xh);
  int8_t* G = reinterpret_cast<int8_t*>(ws + w.G);
  const ivit_scale none{nullptr, nullptr, 1, 1};
  int rc;
  if (a_next_ready) *a_next_ready = false;
  // X^ = MSA(LayerNorm(X)) + X
  if (!a_ready && (rc = launch_layernorm(ctx, X, IVIT_I8, D, to_dev(p->ln1_gamma), p->ln1_beta, p->M_ln, A, D, M, D))) return rc;
  if ((rc = launch_gemm(ctx, linear_problem(A, D, p->Wqkv, D, p->bqkv, p->qkv_scale, nullptr, 0, 1, none, QKV, 3 * D,
                                            IVIT_I8, 0, 0, M, 3 * D, D)))) return rc;
  if ((rc = attention_impl(ctx, p, QKV, O, ws, w))) return rc;
  // output projection + residual; LayerNorm 2 of its rows in the kernel's tail
  GemmProblem proj = linear_problem(O, D, p->Wo, D, p->bo, p->o_scale, X, D, M, p->res1_scale, Xh, D, IVIT_I8, 0, 0, M, D, D);
  want_layernorm(proj, p->ln2_gamma, p->ln2_beta, p->M_ln, A, D);
  ctx->rowop_fused = 0;
  if ((rc = launch_gemm(ctx, proj))) return rc;
  // Y = MLP(LayerNorm(X^)) + X^
  if (!ctx->rowop_fused &&
      (rc = launch_layernorm(ctx, Xh, IVIT_I8, D, to_dev(p->ln2_gamma), p->ln2_beta, p->M_ln, A, D, M, D))) return rc;
  GemmProblem fc1 = linear_problem(A, D, p->W1, D, p->b1, p->fc1_scale, nullptr, 0, 1, none, G, H, IVIT_I8, 0, 0, M, H, D);
  if (p->gelu_static_max) {
    // static-maximum ShiftGELU variant: element-wise, applied to the requantised value inside the FC1 epilogue
    if ((rc = gelu_static_row(ctx, p->gelu, p->gelu_post, &fc1.epi.act_table))) return rc;
    if ((rc = launch_gemm(ctx, fc1))) return rc;
  } else {
    // Algorithm 2 needs the maximum of a token's whole MLP row: ShiftGELU of a block of rows runs once all the
    // channel tiles of those rows are stored, in the FC1 kernel's tail
    if (ctx->row_fusion & 2) {
      if ((rc = gelu_table_for(ctx, p->gelu, p->gelu_post, &fc1.epi.rop.table))) return rc;
      fc1.epi.rop.kind = 2;
    }
    ctx->rowop_fused = 0;
    if ((rc = launch_gemm(ctx, fc1))) return rc;
    if (!ctx->rowop_fused && (rc = launch_shiftgelu(ctx, G, H, p->gelu, p->gelu_post, G, H, M, H))) return rc;
  }
  GemmProblem fc2 = linear_problem(G, H, p->W2, H, p->b2, p->fc2_scale, Xh, D, M, p->res2_scale, Y, D, IVIT_I8, 0, 0, M, D, H);
  if (next) want_layernorm(fc2, next->ln1_gamma, next->ln1_beta, next->M_ln, A, D);
  ctx->rowop_fused = 0;
  if ((rc = launch_gemm(ctx, fc2))) return rc;
  if (a_next_ready) *a_next_ready = next && ctx->rowop_fused;
  return IVIT_OK;
}

}  // namespace

namespace {

void host_graph_drop(ivit_ctx* ctx, int slot) {
  if (ctx->hg_exec[slot]) cudaGraphExecDestroy(ctx->hg_exec[slot]);
  ctx->hg_exec[slot] = nullptr;
  ctx->hg_key_bytes[slot] = 0;   // the key buffer itself is kept for the next description
  ctx->hg_seen[slot] = 0;
}

bool grow(char*& buf, size_t& cap, size_t need) {
  if (cap >= need) return true;
  char* n = new (std::nothrow) char[need];
  if (!n) return false;
  delete[] buf;
  buf = n;
  cap = need;
  return true;
}

// The device part of ivit_vit_forward_host.  With graph replay switched on, the third call that repeats the same
// model description, buffers and stream captures the forward into a CUDA graph (the first two run kernel by
// kernel, so that look-up tables exist); later calls launch the instantiated graph.  Any change of the arguments
// drops the graph.  The graph holds the addresses of cached ShiftGELU tables: it is only kept while the table
// generation of the context is the one it was captured at (another call that rebuilds a table slot makes the
// next call fall back to kernels and capture again), and a capture during which a table had to be built is thrown
// away.  A capture that fails leaves the kernel-by-kernel path in place.
// `run` enqueues the forward kernel by kernel; ctx->hg_scratch holds key_bytes bytes that describe the call (model
// description, buffers, stream, engine).
template <class Run>
int replay_or_run(ivit_ctx* ctx, int slot, size_t key_bytes, Run run) {
  const char* key = ctx->hg_scratch;
  const bool same = ctx->hg_key_bytes[slot] == key_bytes && std::memcmp(ctx->hg_key[slot], key, key_bytes) == 0;
  if (!same) {
    host_graph_drop(ctx, slot);
    if (!grow(ctx->hg_key[slot], ctx->hg_key_cap[slot], key_bytes)) return IVIT_ERR_CUDA;
    std::memcpy(ctx->hg_key[slot], key, key_bytes);
    ctx->hg_key_bytes[slot] = key_bytes;
    ctx->hg_seen[slot] = 1;
    return run();
  }
  if (ctx->hg_exec[slot]) {
    if (ctx->hg_gen[slot] == ctx->gelu_gen) {
      if (cudaGraphLaunch(ctx->hg_exec[slot], ctx->stream) != cudaSuccess) return IVIT_ERR_CUDA;
      ctx->launches += ctx->hg_launches[slot];
      return IVIT_OK;
    }
    // a table slot was rebuilt since the capture: the graph may point at another parameter set's table
    cudaGraphExecDestroy(ctx->hg_exec[slot]);
    ctx->hg_exec[slot] = nullptr;
    ctx->hg_seen[slot] = 1;
    return run();
  }
  if (ctx->hg_seen[slot] < 0 || ++ctx->hg_seen[slot] < 3) return run();
  const int64_t before = ctx->launches;
  // state of the table cache, put back if the capture is not kept (kernels recorded in a discarded capture never ran)
  GeluKey keys_before[kGeluTableSlots];
  std::memcpy(keys_before, ctx->gelu_keys, sizeof(keys_before));
  const int used_before = ctx->gelu_used, next_before = ctx->gelu_next;
  const uint64_t gen_before = ctx->gelu_gen;
  auto restore_cache = [&]() {
    if (ctx->gelu_gen == gen_before) return;
    std::memcpy(ctx->gelu_keys, keys_before, sizeof(keys_before));
    ctx->gelu_used = used_before;
    ctx->gelu_next = next_before;
    ++ctx->gelu_gen;
  };
  if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    ctx->hg_seen[slot] = -1;
    return run();
  }
  const int rc = run();
  cudaGraph_t graph = nullptr;
  const cudaError_t end = cudaStreamEndCapture(ctx->stream, &graph);
  cudaGraphExec_t exec = nullptr;
  const bool tables_stable = ctx->gelu_gen == gen_before;
  if (rc == IVIT_OK && end == cudaSuccess && graph && tables_stable && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
    cudaGraphDestroy(graph);
    ctx->hg_exec[slot] = exec;
    ctx->hg_gen[slot] = ctx->gelu_gen;
    ctx->hg_launches[slot] = ctx->launches - before;
    if (cudaGraphLaunch(exec, ctx->stream) != cudaSuccess) return IVIT_ERR_CUDA;
    return IVIT_OK;
  }
  if (graph) cudaGraphDestroy(graph);
  cudaGetLastError();
  ctx->launches = before;
  restore_cache();
  // a model with more parameter sets than table slots rebuilds tables on every call: try again later, not never
  ctx->hg_seen[slot] = tables_stable ? -1 : 1;
  if (rc) return rc;
  return run();   // nothing ran during the discarded capture
}


int forward_or_replay(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* img_dev, int32_t* lg_dev, void* workspace,
                      size_t inner, int slot) {
  auto run = [&]() { return ivit_vit_forward(ctx, p, img_dev, lg_dev, workspace, inner); };
  if (!ctx->host_graph || ctx->profiling || ctx->stream == nullptr) return run();
  const size_t nb = (size_t)p->depth * sizeof(ivit_block_params);
  const void* tail[4] = {img_dev, lg_dev, workspace, (const void*)ctx->stream};
  const size_t key_bytes = sizeof(*p) + nb + sizeof(tail) + 2 * sizeof(int);
  if (!grow(ctx->hg_scratch, ctx->hg_scratch_cap, key_bytes)) return IVIT_ERR_CUDA;
  char* key = ctx->hg_scratch;
  std::memcpy(key, p, sizeof(*p));
  std::memcpy(key + sizeof(*p), p->blocks, nb);
  std::memcpy(key + sizeof(*p) + nb, tail, sizeof(tail));
  const int modes[2] = {ctx->gemm_engine, 0};   // second word: which forward (0 = ViT)
  std::memcpy(key + sizeof(*p) + nb + sizeof(tail), modes, sizeof(modes));
  return replay_or_run(ctx, slot, key_bytes, run);
}

// The same for the Swin-shaped forward: the description also covers the stages, their blocks and shift flags.
int swin_forward_or_replay(ivit_ctx* ctx, const ivit_swin_params* p, const int8_t* img_dev, int32_t* lg_dev, void* workspace,
                           size_t inner, int slot) {
  auto run = [&]() { return ivit_swin_forward(ctx, p, img_dev, lg_dev, nullptr, workspace, inner); };
  if (!ctx->host_graph || ctx->profiling || ctx->stream == nullptr) return run();
  size_t key_bytes = sizeof(*p) + (size_t)p->n_stages * sizeof(ivit_swin_stage);
  for (int64_t i = 0; i < p->n_stages; ++i)
    key_bytes += (size_t)p->stages[i].depth * (sizeof(ivit_block_params) + 1);
  const void* tail[4] = {img_dev, lg_dev, workspace, (const void*)ctx->stream};
  key_bytes += sizeof(tail) + 2 * sizeof(int);
  if (!grow(ctx->hg_scratch, ctx->hg_scratch_cap, key_bytes)) return IVIT_ERR_CUDA;
  char* key = ctx->hg_scratch;
  size_t off = 0;
  auto put = [&](const void* src, size_t n) { std::memcpy(key + off, src, n); off += n; };
  put(p, sizeof(*p));
  put(p->stages, (size_t)p->n_stages * sizeof(ivit_swin_stage));
  for (int64_t i = 0; i < p->n_stages; ++i) {
    const ivit_swin_stage& st = p->stages[i];
    put(st.blocks, (size_t)st.depth * sizeof(ivit_block_params));
    for (int64_t b = 0; b < st.depth; ++b) {
      const uint8_t f = st.shifted ? st.shifted[b] : 0;
      put(&f, 1);
    }
  }
  put(tail, sizeof(tail));
  const int modes[2] = {ctx->gemm_engine, 1};   // 1 = Swin-shaped forward
  put(modes, sizeof(modes));
  return replay_or_run(ctx, slot, key_bytes, run);
}

// The host-buffer forwards: [inner workspace | two image staging buffers | logits].  The buffers are used alternately:
// the copy of this call's image runs on a copy stream of the context while the compute stream still works on the
// previous call; it only waits for the call before that to have finished with the buffer.  `run(img_dev, lg_dev,
// slot)` enqueues the device part on the compute stream.
template <class Run>
int host_forward(ivit_ctx* ctx, const int8_t* image_host, int32_t* logits_host, size_t img_bytes, size_t lg_bytes,
                        size_t inner, void* workspace, size_t workspace_bytes, Run run) {
  const size_t img_slot = align_up(img_bytes, 256);
  const size_t img_off = inner, lg_off = inner + 2 * img_slot;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < lg_off + align_up(lg_bytes, 256))
    return IVIT_ERR_WORKSPACE;
  if (!ctx->copy_stream) {
    // first use: a stream of its own for the input copies, and the events that order it with the compute stream
    if (cudaSetDevice(ctx->device) != cudaSuccess ||
        cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess)
      return IVIT_ERR_CUDA;
    for (int i = 0; i < 2; ++i)
      if (cudaEventCreateWithFlags(&ctx->img_ready[i], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&ctx->img_free[i], cudaEventDisableTiming) != cudaSuccess)
        return IVIT_ERR_CUDA;
    ctx->host_calls = 0;
  }
  const int slot = (int)(ctx->host_calls & 1);
  char* ws = static_cast<char*>(workspace);
  char* img_dev = ws + img_off + (size_t)slot * img_slot;
  if (ctx->host_calls >= 2 && cudaStreamWaitEvent(ctx->copy_stream, ctx->img_free[slot], 0) != cudaSuccess) return IVIT_ERR_CUDA;
  if (cudaMemcpyAsync(img_dev, image_host, img_bytes, cudaMemcpyHostToDevice, ctx->copy_stream) != cudaSuccess ||
      cudaEventRecord(ctx->img_ready[slot], ctx->copy_stream) != cudaSuccess ||
      cudaStreamWaitEvent(ctx->stream, ctx->img_ready[slot], 0) != cudaSuccess)
    return IVIT_ERR_CUDA;
  ++ctx->host_calls;
  const int rc = run(reinterpret_cast<const int8_t*>(img_dev), reinterpret_cast<int32_t*>(ws + lg_off), slot);
  // recorded even after an error: a later copy into this buffer waits for it
  if (cudaEventRecord(ctx->img_free[slot], ctx->stream) != cudaSuccess) return IVIT_ERR_CUDA;
  if (rc) return rc;
  if (cudaMemcpyAsync(logits_host, ws + lg_off, lg_bytes, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
    return IVIT_ERR_CUDA;
  return IVIT_OK;
}


}  // namespace

namespace ivit {
int launch_gemm(ivit_ctx* ctx, const GemmProblem& g) {
  if (ctx->gemm_engine == 0) {
    const int rc = launch_gemm_tc(ctx, g);
    if (rc != IVIT_ERR_UNSUPPORTED) return rc;
  }
  return launch_gemm_simt(ctx, g);
}
}  // namespace ivit

extern "C" {

const char* ivit_strerror(int code) {
  switch (code) {
    case IVIT_OK: return "ok";
    case IVIT_ERR_INVALID_ARG: return "invalid argument";
    case IVIT_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
    case IVIT_ERR_RANGE: return "quantisation constant out of range";
    case IVIT_ERR_UNSUPPORTED: return "shape or dtype combination not supported";
    case IVIT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case IVIT_ERR_CUDA: return "CUDA call failed";
    case IVIT_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown error";
  }
}

int ivit_ctx_create(ivit_ctx** out, int device, void* cuda_stream) {
  if (!out) return IVIT_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return IVIT_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return IVIT_ERR_CUDA;
  if (prop.major != 10) return IVIT_ERR_CUDA;  // kernels are built for sm_100a only
  if (cudaSetDevice(device) != cudaSuccess) return IVIT_ERR_CUDA;
  ivit_ctx* c = new (std::nothrow) ivit_ctx();
  if (!c) return IVIT_ERR_CUDA;
  std::memset(c, 0, sizeof(*c));
  c->device = device;
  c->stream = (cudaStream_t)cuda_stream;
  c->sm_count = prop.multiProcessorCount;
  if (cudaHostAlloc((void**)&c->status_host, sizeof(int), cudaHostAllocMapped) != cudaSuccess) { delete c; return IVIT_ERR_CUDA; }
  *c->status_host = 0;
  if (cudaHostGetDevicePointer((void**)&c->status_dev, c->status_host, 0) != cudaSuccess ||
      cudaMalloc((void**)&c->gelu_tables, (size_t)kGeluTableSlots * kGeluTableBytes + 128 + kRowStateBytes) != cudaSuccess ||
      cudaMemset(c->gelu_tables + (size_t)kGeluTableSlots * kGeluTableBytes, 0, 128 + kRowStateBytes) != cudaSuccess) {
    cudaFreeHost(c->status_host);
    delete c;
    return IVIT_ERR_CUDA;
  }
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    fn = nullptr;
  c->tmap_encode = fn;
  if (gemm_tc_prepare_device() != IVIT_OK || attention_prepare_device() != IVIT_OK) {
    cudaGetLastError();
    cudaFree(c->gelu_tables);
    cudaFreeHost(c->status_host);
    delete c;
    return IVIT_ERR_CUDA;
  }
  c->sched_dev = reinterpret_cast<unsigned*>(c->gelu_tables + (size_t)kGeluTableSlots * kGeluTableBytes);
  c->rowblk_dev = c->sched_dev + 32;
  c->row_fusion = 0;
  c->gemm_pairs = 1;
  *out = c;
  return IVIT_OK;
}

int ivit_ctx_destroy(ivit_ctx* ctx) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  // graphs point at the table cache: drop them and let the stream drain before the cache is freed
  for (int i = 0; i < 2; ++i) {
    host_graph_drop(ctx, i);
    delete[] ctx->hg_key[i];
  }
  delete[] ctx->hg_scratch;
  cudaStreamSynchronize(ctx->stream);
  cudaFree(ctx->gelu_tables);
  cudaFreeHost(ctx->status_host);
  tmap_cache_free(ctx);
  if (ctx->copy_stream) {
    cudaStreamSynchronize(ctx->copy_stream);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(ctx->img_ready[i]);
      cudaEventDestroy(ctx->img_free[i]);
    }
    cudaStreamDestroy(ctx->copy_stream);
  }
  if (ctx->prof_ev) {
    for (int i = 0; i < 2 * kProfMax; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
    delete[] ctx->prof_kind;
    delete[] ctx->prof_work;
  }
  delete ctx;
  return IVIT_OK;
}

int ivit_ctx_set_stream(ivit_ctx* ctx, void* cuda_stream) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  ctx->stream = (cudaStream_t)cuda_stream;
  for (int i = 0; i < 2; ++i) host_graph_drop(ctx, i);
  ctx->gelu_used = 0;  // tables were built in the order of the old stream
  ctx->gelu_next = 0;
  ++ctx->gelu_gen;
  return IVIT_OK;
}

int ivit_ctx_poll_status(ivit_ctx* ctx) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  volatile int* s = ctx->status_host;
  const int v = *s;
  if (v != 0) {
    *s = 0;
    // a kernel that gave up may have left work counters behind: zero them for the launches that follow
    cudaMemsetAsync(ctx->sched_dev, 0, 128 + kRowStateBytes, ctx->stream);
    return v;
  }
  return IVIT_OK;
}

int64_t ivit_ctx_launch_count(const ivit_ctx* ctx) { return ctx ? ctx->launches : 0; }
int64_t ivit_ctx_pair_launch_count(const ivit_ctx* ctx) { return ctx ? ctx->pair_launches : 0; }

uint64_t ivit_ctx_table_generation(const ivit_ctx* ctx) { return ctx ? ctx->gelu_gen : 0; }

int ivit_ctx_set_row_fusion(ivit_ctx* ctx, int enable) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  // 1: every row operator; 2: I-LayerNorm only, 4: ShiftGELU only (for measurements)
  ctx->row_fusion = enable == 1 ? 3 : (enable == 2 ? 1 : (enable == 4 ? 2 : 0));
  for (int i = 0; i < 2; ++i) host_graph_drop(ctx, i);
  return IVIT_OK;
}

int ivit_ctx_set_gemm_pairs(ivit_ctx* ctx, int enable) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  ctx->gemm_pairs = enable ? 1 : 0;
  for (int i = 0; i < 2; ++i) host_graph_drop(ctx, i);
  return IVIT_OK;
}

int ivit_ctx_set_gemm_engine(ivit_ctx* ctx, int engine) {
  if (!ctx || engine < 0 || engine > 1) return IVIT_ERR_INVALID_ARG;
  ctx->gemm_engine = engine;
  return IVIT_OK;
}

int ivit_linear(ivit_ctx* ctx, const int8_t* A, int64_t lda, const int8_t* W, int64_t ldw,
                const int32_t* bias, ivit_scale scale, const int8_t* res, int64_t ldres,
                int64_t res_rows, ivit_scale res_scale, void* out, int64_t ldo, int32_t out_dtype,
                int64_t out_group_rows, int64_t out_group_stride, int64_t M, int64_t N, int64_t K) {
  if (!ctx || !A || !W || !out || M < 0 || N < 1 || K < 1) return IVIT_ERR_INVALID_ARG;
  if (out_dtype != IVIT_I8 && out_dtype != IVIT_I32) return IVIT_ERR_INVALID_ARG;
  if (K > 65536) return IVIT_ERR_RANGE;
  if (K % 16) return IVIT_ERR_UNSUPPORTED;
  if (lda < K || ldw < K || ldo < N) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(A) || !aligned16(W) || !aligned16(out) || lda % 16 || ldw % 16) return IVIT_ERR_ALIGNMENT;
  if (ldo % (out_dtype == IVIT_I8 ? 16 : 4)) return IVIT_ERR_ALIGNMENT;
  if (bias && !aligned16(bias)) return IVIT_ERR_ALIGNMENT;
  if (!scale_ok(scale)) return IVIT_ERR_RANGE;
  if (res) {
    if (!scale_ok(res_scale) || res_scale.mult_c) return IVIT_ERR_RANGE;
    if (res_rows < 1 || ldres < N) return IVIT_ERR_INVALID_ARG;
    if (!aligned16(res) || ldres % 16) return IVIT_ERR_ALIGNMENT;
  }
  if (out_group_rows > 0 && out_group_stride < out_group_rows) return IVIT_ERR_INVALID_ARG;
  return launch_gemm(ctx, linear_problem(A, lda, W, ldw, bias, scale, res, ldres, res_rows, res_scale, out, ldo,
                                         out_dtype, out_group_rows, out_group_stride, M, N, K));
}

int ivit_matmul(ivit_ctx* ctx, const int8_t* A, int64_t lda, int64_t sAo, int64_t sAi,
                const int8_t* B, int64_t ldb, int64_t sBo, int64_t sBi, int32_t transB,
                const int32_t* bias32, int64_t ldbias, int64_t bias_batches, ivit_scale scale,
                int8_t* C, int64_t ldc, int64_t sCo, int64_t sCi, int64_t batches_outer,
                int64_t batches_inner, int64_t Ma, int64_t Nb, int64_t K) {
  if (!ctx || !A || !B || !C || Ma < 0 || Nb < 0 || K < 1 || batches_outer < 0 || batches_inner < 1)
    return IVIT_ERR_INVALID_ARG;
  if (K > 65536) return IVIT_ERR_RANGE;
  if (!scale_ok(scale) || scale.mult_c) return IVIT_ERR_RANGE;
  if (bias32 && (bias_batches < 1 || ldbias < Nb)) return IVIT_ERR_INVALID_ARG;
  if (!aligned4(A) || !aligned4(B) || !aligned4(C)) return IVIT_ERR_ALIGNMENT;
  const int64_t strides[] = {lda, sAo, sAi, ldb, sBo, sBi, ldc, sCo, sCi};
  for (int64_t s : strides)
    if (s % 4) return IVIT_ERR_ALIGNMENT;
  if (lda < K || ldc < Nb || ldb < (transB ? K : Nb)) return IVIT_ERR_INVALID_ARG;
  GemmProblem g{};
  g.A = A; g.lda = lda; g.sAo = sAo; g.sAi = sAi;
  g.B = B; g.ldb = ldb; g.sBo = sBo; g.sBi = sBi; g.transB = transB ? 1 : 0;
  g.sCo = sCo; g.sCi = sCi; g.batches_outer = batches_outer; g.batches_inner = batches_inner;
  g.M = Ma; g.N = Nb; g.K = K;
  g.epi.bias32 = bias32; g.epi.ldbias = ldbias; g.epi.bias_batches = bias32 ? bias_batches : 1;
  g.epi.scale = to_dev(scale); g.epi.res_rows = 1;
  g.epi.out = C; g.epi.ldo = ldc; g.epi.out_dtype = IVIT_I8;
  return launch_gemm(ctx, g);
}

int ivit_shiftmax(ivit_ctx* ctx, const void* in, int32_t in_dtype, int64_t ldin,
                  const int32_t* bias32, int64_t ldbias, int64_t bias_rows, ivit_scale pre,
                  ivit_exp_params p, int8_t* out, int64_t ldout, int64_t rows, int64_t d) {
  if (!ctx || !in || !out || rows < 0 || d < 1) return IVIT_ERR_INVALID_ARG;
  if (in_dtype != IVIT_I8 && in_dtype != IVIT_I32) return IVIT_ERR_INVALID_ARG;
  if (d > 8192) return IVIT_ERR_UNSUPPORTED;
  if (ldin < d || ldout < round16(d)) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(in) || !aligned16(out) || ldout % 16 || ldin % (in_dtype == IVIT_I8 ? 16 : 4)) return IVIT_ERR_ALIGNMENT;
  int rc = check_exp(p, d, false);
  if (rc) return rc;
  if (in_dtype == IVIT_I32) {
    if (!scale_ok(pre) || pre.mult_c) return IVIT_ERR_RANGE;
    if (bias32 && (bias_rows < 1 || ldbias < d)) return IVIT_ERR_INVALID_ARG;
    if (bias32 && (!aligned16(bias32) || ldbias % 4)) return IVIT_ERR_ALIGNMENT;
  }
  return launch_shiftmax(ctx, in, in_dtype, ldin, bias32, ldbias, bias_rows, to_dev(pre), p, out, ldout, rows, d);
}

int ivit_shiftmax_direct(ivit_ctx* ctx, const int32_t* in, int64_t ldin, ivit_exp_params p, int8_t* out,
                         int64_t ldout, int64_t rows, int64_t d) {
  if (!ctx || !in || !out || rows < 0 || d < 1) return IVIT_ERR_INVALID_ARG;
  if (d > 8192) return IVIT_ERR_UNSUPPORTED;
  if (ldin < d || ldout < round16(d)) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(in) || !aligned16(out) || ldout % 16 || ldin % 4) return IVIT_ERR_ALIGNMENT;
  if (p.I0 < 1 || p.I0 > (1 << 28) || p.N < 0 || p.N > 24 || p.k_out < 2 || p.k_out > 8 || p.M < 32 || p.M > 62)
    return IVIT_ERR_RANGE;
  // the largest possible sum d * I0 * 2^N leaves the reciprocal floor(2^M / sum) at least 13 bits
  if (((int64_t)p.I0 << p.N) > (((int64_t)1 << (p.M - 13)) / d)) return IVIT_ERR_RANGE;
  return launch_shiftmax_direct(ctx, in, ldin, p, out, ldout, rows, d);
}

int ivit_shiftgelu(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p,
                   ivit_scale post, int8_t* out, int64_t ldout, int64_t rows, int64_t cols) {
  if (!ctx || !in || !out || rows < 0 || cols < 1) return IVIT_ERR_INVALID_ARG;
  if (cols % 16 || cols > 16384) return IVIT_ERR_UNSUPPORTED;
  if (ldin < cols || ldout < cols) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(in) || !aligned16(out) || ldin % 16 || ldout % 16) return IVIT_ERR_ALIGNMENT;
  if (!scale_ok(post) || post.mult_c) return IVIT_ERR_RANGE;
  int rc = check_exp(p, cols, true);
  if (rc) return rc;
  return launch_shiftgelu(ctx, in, ldin, p, post, out, ldout, rows, cols);
}

int ivit_shiftgelu_static(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p,
                          ivit_scale post, int8_t* out, int64_t ldout, int64_t rows, int64_t cols) {
  if (!ctx || !in || !out || rows < 0 || cols < 1) return IVIT_ERR_INVALID_ARG;
  if (cols % 16 || cols > 16384) return IVIT_ERR_UNSUPPORTED;
  if (ldin < cols || ldout < cols) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(in) || !aligned16(out) || ldin % 16 || ldout % 16) return IVIT_ERR_ALIGNMENT;
  if (!scale_ok(post) || post.mult_c) return IVIT_ERR_RANGE;
  int rc = check_exp(p, cols, true);
  if (rc) return rc;
  return launch_shiftgelu_static(ctx, in, ldin, p, post, out, ldout, rows, cols);
}

int ivit_layernorm(ivit_ctx* ctx, const void* in, int32_t in_dtype, int64_t ldin,
                   ivit_scale gamma_scale, const int32_t* beta, int32_t M_ln, int8_t* out,
                   int64_t ldout, int64_t rows, int64_t C) {
  if (!ctx || !in || !out || rows < 0 || C < 1) return IVIT_ERR_INVALID_ARG;
  if (in_dtype != IVIT_I8 && in_dtype != IVIT_I32) return IVIT_ERR_INVALID_ARG;
  if (C % 4 || C > 16384) return IVIT_ERR_UNSUPPORTED;
  if (M_ln < 8 || M_ln > 29) return IVIT_ERR_RANGE;
  if (ldin < C || ldout < C) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(in) || !aligned16(out) || ldout % 16 || ldin % (in_dtype == IVIT_I8 ? 16 : 4)) return IVIT_ERR_ALIGNMENT;
  if (!scale_ok(gamma_scale)) return IVIT_ERR_RANGE;
  return launch_layernorm(ctx, in, in_dtype, ldin, to_dev(gamma_scale), beta, M_ln, out, ldout, rows, C);
}

size_t ivit_block_workspace_bytes(const ivit_block_params* p) {
  if (check_block(p) != IVIT_OK) return 0;
  return block_ws(p).total;
}

int ivit_block_forward(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* X, int8_t* Y,
                       void* workspace, size_t workspace_bytes) {
  if (!ctx || !X || !Y || X == Y) return IVIT_ERR_INVALID_ARG;
  int rc = check_block(p);
  if (rc) return rc;
  if (!aligned16(X) || !aligned16(Y)) return IVIT_ERR_ALIGNMENT;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < block_ws(p).total)
    return IVIT_ERR_WORKSPACE;
  return block_impl(ctx, p, X, Y, static_cast<char*>(workspace));
}

// Scratch of ivit_block_forward_static: part of the library image, present on every GPU that loads it.
static __device__ __align__(256) unsigned char g_static_scratch[IVIT_STATIC_SCRATCH_BYTES];

int ivit_block_forward_static(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* X, int8_t* Y) {
  if (!ctx || !X || !Y || X == Y) return IVIT_ERR_INVALID_ARG;
  int rc = check_block(p);
  if (rc) return rc;
  if (!aligned16(X) || !aligned16(Y)) return IVIT_ERR_ALIGNMENT;
  if (block_ws(p).total > (size_t)IVIT_STATIC_SCRATCH_BYTES) return IVIT_ERR_WORKSPACE;   // larger than the fixed scratch
  // In host code the array's name is only a handle; kernels need its device address, which differs per
  // device.  It is looked up once per device, with that device current, and kept.
  // (Two host threads making the first call on a device at the same time both look the address up and store the
  // same value: harmless.)
  static void* scratch_of_device[64] = {nullptr};
  if (ctx->device < 0 || ctx->device >= 64) return IVIT_ERR_UNSUPPORTED;
  if (!scratch_of_device[ctx->device]) {
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess) return IVIT_ERR_CUDA;
    if (current != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return IVIT_ERR_CUDA;
    void* ptr = nullptr;
    const cudaError_t err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (current != ctx->device) cudaSetDevice(current);
    if (err != cudaSuccess || !ptr) return IVIT_ERR_CUDA;
    scratch_of_device[ctx->device] = ptr;
  }
  return block_impl(ctx, p, X, Y, static_cast<char*>(scratch_of_device[ctx->device]));
}

int ivit_attention(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O,
                   void* workspace, size_t workspace_bytes) {
  if (!ctx || !QKV || !O) return IVIT_ERR_INVALID_ARG;
  int rc = check_block(p);
  if (rc) return rc;
  if (!aligned16(QKV) || !aligned16(O)) return IVIT_ERR_ALIGNMENT;
  const BlockWs w = block_ws(p);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < w.total) return IVIT_ERR_WORKSPACE;
  return attention_impl(ctx, p, QKV, O, static_cast<char*>(workspace), w);
}

static int check_vit(const ivit_vit_params* p) {
  if (!p || p->B < 0 || p->depth < 1 || !p->blocks || p->patch < 4 || p->patch % 4 || p->img % p->patch) return IVIT_ERR_INVALID_ARG;
  const int64_t g = p->img / p->patch;
  if (p->T != g * g + 1 || p->D % 16 || p->classes < 1) return IVIT_ERR_INVALID_ARG;
  if (!p->Wpe || !p->pos || !p->cls || !p->Whead) return IVIT_ERR_INVALID_ARG;
  if (!scale_ok(p->pe_scale) || !scale_ok(p->pos_scale) || p->pos_scale.mult_c || !scale_ok(p->lnf_gamma) || !scale_ok(p->head_scale))
    return IVIT_ERR_RANGE;
  for (int64_t l = 0; l < p->depth; ++l) {
    const ivit_block_params* b = &p->blocks[l];
    int rc = check_block(b);
    if (rc) return rc;
    if (b->B != p->B || b->T != p->T || b->D != p->D) return IVIT_ERR_INVALID_ARG;
  }
  return IVIT_OK;
}

struct VitWs { size_t patches, X, Y, Z, block, total; };
static VitWs vit_ws(const ivit_vit_params* p) {
  VitWs w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t Kpe = (size_t)(3 * p->patch * p->patch);
  w.patches = take((size_t)(p->B * (p->T - 1)) * Kpe);
  w.X = take((size_t)(p->B * p->T * p->D));
  w.Y = take((size_t)(p->B * p->T * p->D));
  w.Z = take((size_t)(p->B * p->D));
  size_t blk = 0;
  for (int64_t l = 0; l < p->depth; ++l) {
    const size_t b = block_ws(&p->blocks[l]).total;
    blk = b > blk ? b : blk;
  }
  w.block = take(blk);
  w.total = off;
  return w;
}

size_t ivit_vit_workspace_bytes(const ivit_vit_params* p) {
  if (check_vit(p) != IVIT_OK) return 0;
  return vit_ws(p).total;
}

int ivit_vit_forward(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image, int32_t* logits,
                     void* workspace, size_t workspace_bytes) {
  return ivit_vit_forward_tokens(ctx, p, image, logits, nullptr, workspace, workspace_bytes);
}

int ivit_vit_forward_tokens(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image, int32_t* logits,
                            int8_t* tokens, void* workspace, size_t workspace_bytes) {
  if (!ctx || !image || !logits) return IVIT_ERR_INVALID_ARG;
  int rc = check_vit(p);
  if (rc) return rc;
  if (!aligned16(image) || !aligned16(logits) || p->classes % 4) return IVIT_ERR_ALIGNMENT;
  if (tokens && !aligned16(tokens)) return IVIT_ERR_ALIGNMENT;
  const VitWs w = vit_ws(p);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < w.total) return IVIT_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  const int64_t B = p->B, T = p->T, D = p->D, np = T - 1, Kpe = 3 * p->patch * p->patch;
  int8_t* patches = reinterpret_cast<int8_t*>(ws + w.patches);
  int8_t* X = reinterpret_cast<int8_t*>(ws + w.X);
  int8_t* Y = reinterpret_cast<int8_t*>(ws + w.Y);
  int8_t* Z = reinterpret_cast<int8_t*>(ws + w.Z);
  const ivit_scale none{nullptr, nullptr, 1, 1};
  if ((rc = launch_patchify(ctx, image, B, 3, p->img, p->img, p->patch, 0, patches, Kpe))) return rc;
  // patch embedding as a Dense layer; the position embedding enters through the residual port;
  // patch q of image b lands in token row b*T + 1 + q
  if ((rc = launch_gemm(ctx, linear_problem(patches, Kpe, p->Wpe, Kpe, p->bpe, p->pe_scale, p->pos, D, np,
                                            p->pos_scale, X + D, D, IVIT_I8, np, T, B * np, D, Kpe)))) return rc;
  if ((rc = launch_fill_rows(ctx, p->cls, D, X, T * D, B))) return rc;
  bool a_ready = false;   // LayerNorm 1 of the next block already produced by the previous block's last Dense layer
  for (int64_t l = 0; l < p->depth; ++l) {
    const ivit_block_params* next = l + 1 < p->depth ? &p->blocks[l + 1] : nullptr;
    if ((rc = block_impl(ctx, &p->blocks[l], X, Y, ws + w.block, a_ready, next, &a_ready))) return rc;
    int8_t* t = X; X = Y; Y = t;
  }
  if (tokens && cudaMemcpyAsync(tokens, X, (size_t)(B * T * D), cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess)
    return IVIT_ERR_CUDA;
  // final LayerNorm on the class-token rows, then the classifier (int32 logits, not saturated)
  if ((rc = launch_layernorm(ctx, X, IVIT_I8, T * D, to_dev(p->lnf_gamma), p->lnf_beta, p->blocks[0].M_ln, Z, D, B, D))) return rc;
  return launch_gemm(ctx, linear_problem(Z, D, p->Whead, D, p->bhead, p->head_scale, nullptr, 0, 1, none, logits,
                                         p->classes, IVIT_I32, 0, 0, B, p->classes, D));
}

size_t ivit_vit_host_workspace_bytes(const ivit_vit_params* p) {
  if (check_vit(p) != IVIT_OK) return 0;
  const size_t img = align_up((size_t)(p->B * 3 * p->img * p->img), 256);
  const size_t lg = align_up((size_t)(p->B * p->classes) * 4, 256);
  return vit_ws(p).total + 2 * img + lg;
}

// ---- Swin-shaped forward -------------------------------------------------------------------------------

static int check_swin(const ivit_swin_params* p) {
  if (!p || p->B < 0 || p->n_stages < 1 || !p->stages || p->patch < 4 || p->patch % 4 || p->window < 1 || p->classes < 1)
    return IVIT_ERR_INVALID_ARG;
  if (p->img % p->patch || !p->Wpe || !p->Whead) return IVIT_ERR_INVALID_ARG;
  if (p->M_ln < 8 || p->M_ln > 29) return IVIT_ERR_RANGE;
  if (!scale_ok(p->pe_scale) || !scale_ok(p->pe_ln_gamma) || !scale_ok(p->lnf_gamma) || !scale_ok(p->pool_scale) ||
      p->pool_scale.mult_c || !scale_ok(p->head_scale))
    return IVIT_ERR_RANGE;
  int64_t res = p->img / p->patch;
  for (int64_t s = 0; s < p->n_stages; ++s) {
    const ivit_swin_stage* st = &p->stages[s];
    if (st->res != res || st->C < 16 || st->C % 16 || st->depth < 1 || !st->blocks || res % p->window) return IVIT_ERR_INVALID_ARG;
    const int64_t windows = p->B * (res / p->window) * (res / p->window);
    for (int64_t l = 0; l < st->depth; ++l) {
      const ivit_block_params* b = &st->blocks[l];
      int rc = check_block(b);
      if (rc) return rc;
      if (b->B != windows || b->T != p->window * p->window || b->D != st->C) return IVIT_ERR_INVALID_ARG;
      if (st->shifted && st->shifted[l] && (!st->shift_index || !st->unshift_index)) return IVIT_ERR_INVALID_ARG;
    }
    const bool last = s + 1 == p->n_stages;
    if (last != (st->merge_index == nullptr)) return IVIT_ERR_INVALID_ARG;
    if (!last) {
      if (!st->Wmerge || res % 2) return IVIT_ERR_INVALID_ARG;
      if (!scale_ok(st->merge_ln_gamma) || !scale_ok(st->merge_scale)) return IVIT_ERR_RANGE;
      if (p->stages[s + 1].C != 2 * st->C) return IVIT_ERR_INVALID_ARG;
      res /= 2;
    }
  }
  return IVIT_OK;
}

struct SwinWs { size_t patches, P[3], Z, block, total; };
static SwinWs swin_ws(const ivit_swin_params* p) {
  SwinWs w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const int64_t res0 = p->img / p->patch;
  const size_t Kpe = (size_t)(3 * p->patch * p->patch);
  w.patches = take((size_t)(p->B * res0 * res0) * Kpe);
  // the token tensor is largest in stage 0 (every merge halves its bytes); three buffers of that size
  const size_t tok = (size_t)(p->B * res0 * res0 * p->stages[0].C);
  for (int i = 0; i < 3; ++i) w.P[i] = take(tok);
  w.Z = take((size_t)(p->B * p->stages[p->n_stages - 1].C));
  size_t blk = 0;
  for (int64_t s = 0; s < p->n_stages; ++s)
    for (int64_t l = 0; l < p->stages[s].depth; ++l) {
      const size_t b = block_ws(&p->stages[s].blocks[l]).total;
      blk = b > blk ? b : blk;
    }
  w.block = take(blk);
  w.total = off;
  return w;
}

size_t ivit_swin_workspace_bytes(const ivit_swin_params* p) {
  if (check_swin(p) != IVIT_OK) return 0;
  return swin_ws(p).total;
}

// Dense layer followed by I-LayerNorm of its output rows (in the Dense kernel's tail where that is possible).
static int dense_then_layernorm(ivit_ctx* ctx, GemmProblem g, const ivit_scale& gamma, const int32_t* beta, int M_ln,
                                int8_t* ln_out) {
  const int64_t M = g.M, N = g.N;
  want_layernorm(g, gamma, beta, M_ln, ln_out, N);
  ctx->rowop_fused = 0;
  int rc = launch_gemm(ctx, g);
  if (rc) return rc;
  if (ctx->rowop_fused) return IVIT_OK;
  return launch_layernorm(ctx, g.epi.out, IVIT_I8, g.epi.ldo, to_dev(gamma), beta, M_ln, ln_out, N, M, N);
}

int ivit_swin_forward(ivit_ctx* ctx, const ivit_swin_params* p, const int8_t* image, int32_t* logits,
                      int8_t* tokens, void* workspace, size_t workspace_bytes) {
  if (!ctx || !image || !logits) return IVIT_ERR_INVALID_ARG;
  int rc = check_swin(p);
  if (rc) return rc;
  if (!aligned16(image) || !aligned16(logits) || p->classes % 4 || (tokens && !aligned16(tokens))) return IVIT_ERR_ALIGNMENT;
  const SwinWs w = swin_ws(p);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < w.total) return IVIT_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  const ivit_scale none{nullptr, nullptr, 1, 1};
  const int64_t B = p->B, Kpe = 3 * p->patch * p->patch;
  int64_t res = p->img / p->patch, rows = B * res * res;
  int8_t* patches = reinterpret_cast<int8_t*>(ws + w.patches);
  int8_t* cur = reinterpret_cast<int8_t*>(ws + w.P[0]);
  int8_t* other = reinterpret_cast<int8_t*>(ws + w.P[1]);
  int8_t* third = reinterpret_cast<int8_t*>(ws + w.P[2]);
  int8_t* Z = reinterpret_cast<int8_t*>(ws + w.Z);
  char* wsb = ws + w.block;
  if ((rc = launch_patchify(ctx, image, B, 3, p->img, p->img, p->patch, p->window, patches, Kpe))) return rc;
  const int64_t C0 = p->stages[0].C;
  if ((rc = dense_then_layernorm(ctx, linear_problem(patches, Kpe, p->Wpe, Kpe, p->bpe, p->pe_scale, nullptr, 0, 1, none, other,
                                                      C0, IVIT_I8, 0, 0, rows, C0, Kpe),
                                 p->pe_ln_gamma, p->pe_ln_beta, p->M_ln, cur))) return rc;
  // the final LayerNorm, dressed as the LayerNorm 1 of a block that follows the last one
  ivit_block_params fin{};
  fin.ln1_gamma = p->lnf_gamma; fin.ln1_beta = p->lnf_beta; fin.M_ln = p->M_ln;
  bool a_ready = false;   // the LayerNorm output that the next block (or the pooling) reads sits in the block workspace
  for (int64_t s = 0; s < p->n_stages; ++s) {
    const ivit_swin_stage* st = &p->stages[s];
    const int64_t C = st->C;
    for (int64_t l = 0; l < st->depth; ++l) {
      const bool sh = st->shifted && st->shifted[l];
      const bool sh_next = l + 1 < st->depth && st->shifted && st->shifted[l + 1];
      // LayerNorm 1 of the next block comes out of this block's last Dense layer when the next block reads this
      // block's output rows as they are (no row permutation in between)
      const ivit_block_params* next = (l + 1 < st->depth && !sh && !sh_next) ? &st->blocks[l + 1] : nullptr;
      if (l + 1 == st->depth && s + 1 == p->n_stages && !sh) next = &fin;
      if (sh) {
        if ((rc = launch_gather_rows(ctx, cur, C, st->shift_index, rows, C, third, C))) return rc;
        if ((rc = block_impl(ctx, &st->blocks[l], third, other, wsb, false, nullptr, nullptr))) return rc;
        if ((rc = launch_gather_rows(ctx, other, C, st->unshift_index, rows, C, cur, C))) return rc;
        a_ready = false;
      } else {
        if ((rc = block_impl(ctx, &st->blocks[l], cur, other, wsb, a_ready, next, &a_ready))) return rc;
        int8_t* t = cur; cur = other; other = t;
      }
    }
    if (st->merge_index) {
      // 2x2 patch merging: four C-wide slices per output row, LayerNorm over 4C, Dense to 2C
      if ((rc = launch_gather_rows(ctx, cur, C, st->merge_index, rows, C, other, C))) return rc;
      rows /= 4;
      res /= 2;
      if ((rc = launch_layernorm(ctx, other, IVIT_I8, 4 * C, to_dev(st->merge_ln_gamma), st->merge_ln_beta, p->M_ln, third,
                                 4 * C, rows, 4 * C))) return rc;
      // ... followed by LayerNorm 1 of the next stage's first block (into the block workspace, where it expects it)
      const ivit_block_params* nb = &p->stages[s + 1].blocks[0];
      if ((rc = dense_then_layernorm(ctx, linear_problem(third, 4 * C, st->Wmerge, 4 * C, nullptr, st->merge_scale, nullptr, 0, 1,
                                                          none, cur, 2 * C, IVIT_I8, 0, 0, rows, 2 * C, 4 * C),
                                     nb->ln1_gamma, nb->ln1_beta, nb->M_ln, reinterpret_cast<int8_t*>(wsb)))) return rc;
      a_ready = !(p->stages[s + 1].shifted && p->stages[s + 1].shifted[0]);
    }
  }
  const int64_t Cl = p->stages[p->n_stages - 1].C;
  if (tokens && cudaMemcpyAsync(tokens, cur, (size_t)(rows * Cl), cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess)
    return IVIT_ERR_CUDA;
  const int8_t* normed = reinterpret_cast<const int8_t*>(wsb);
  if (!a_ready) {
    if ((rc = launch_layernorm(ctx, cur, IVIT_I8, Cl, to_dev(p->lnf_gamma), p->lnf_beta, p->M_ln, other, Cl, rows, Cl))) return rc;
    normed = other;
  }
  if ((rc = launch_token_mean(ctx, normed, Cl, B, rows / (B > 0 ? B : 1), Cl, to_dev(p->pool_scale), Z, Cl))) return rc;
  return launch_gemm(ctx, linear_problem(Z, Cl, p->Whead, Cl, p->bhead, p->head_scale, nullptr, 0, 1, none, logits, p->classes,
                                         IVIT_I32, 0, 0, B, p->classes, Cl));
}

size_t ivit_swin_host_workspace_bytes(const ivit_swin_params* p) {
  if (check_swin(p) != IVIT_OK) return 0;
  return swin_ws(p).total + 2 * align_up((size_t)(p->B * 3 * p->img * p->img), 256) + align_up((size_t)(p->B * p->classes) * 4, 256);
}

int ivit_swin_forward_host(ivit_ctx* ctx, const ivit_swin_params* p, const int8_t* image_host, int32_t* logits_host,
                           void* workspace, size_t workspace_bytes) {
  if (!ctx || !image_host || !logits_host) return IVIT_ERR_INVALID_ARG;
  const int rc = check_swin(p);
  if (rc) return rc;
  const size_t inner = swin_ws(p).total;
  return host_forward(ctx, image_host, logits_host, (size_t)(p->B * 3 * p->img * p->img), (size_t)(p->B * p->classes) * 4, inner,
                      workspace, workspace_bytes, [&](const int8_t* img_dev, int32_t* lg_dev, int slot) {
                        return swin_forward_or_replay(ctx, p, img_dev, lg_dev, workspace, inner, slot);
                      });
}

int ivit_ctx_set_host_graph(ivit_ctx* ctx, int enable) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  ctx->host_graph = enable ? 1 : 0;
  if (!enable)
    for (int i = 0; i < 2; ++i) host_graph_drop(ctx, i);
  return IVIT_OK;
}

int ivit_ctx_host_graph_count(ivit_ctx* ctx) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  return (ctx->hg_exec[0] ? 1 : 0) + (ctx->hg_exec[1] ? 1 : 0);
}

int ivit_vit_forward_host(ivit_ctx* ctx, const ivit_vit_params* p, const int8_t* image_host,
                          int32_t* logits_host, void* workspace, size_t workspace_bytes) {
  if (!ctx || !image_host || !logits_host) return IVIT_ERR_INVALID_ARG;
  const int rc = check_vit(p);
  if (rc) return rc;
  const size_t inner = vit_ws(p).total;
  return host_forward(ctx, image_host, logits_host, (size_t)(p->B * 3 * p->img * p->img), (size_t)(p->B * p->classes) * 4, inner,
                      workspace, workspace_bytes, [&](const int8_t* img_dev, int32_t* lg_dev, int slot) {
                        return forward_or_replay(ctx, p, img_dev, lg_dev, workspace, inner, slot);
                      });
}

int ivit_ctx_profile_start(ivit_ctx* ctx) {
  if (!ctx) return IVIT_ERR_INVALID_ARG;
  if (!ctx->prof_ev) {
    ctx->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfMax];
    ctx->prof_kind = new (std::nothrow) int[kProfMax];
    ctx->prof_work = new (std::nothrow) double[kProfMax];
    if (!ctx->prof_ev || !ctx->prof_kind || !ctx->prof_work) return IVIT_ERR_CUDA;
    for (int i = 0; i < 2 * kProfMax; ++i)
      if (cudaEventCreate(&ctx->prof_ev[i]) != cudaSuccess) return IVIT_ERR_CUDA;
  }
  ctx->prof_count = 0;
  ctx->profiling = true;
  return IVIT_OK;
}

int ivit_ctx_profile_stop(ivit_ctx* ctx) {
  if (!ctx || !ctx->profiling) return IVIT_ERR_INVALID_ARG;
  ctx->profiling = false;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IVIT_ERR_CUDA;
  return ctx->prof_count;
}

int ivit_ctx_profile_get(ivit_ctx* ctx, int32_t idx, int32_t* kind, float* ms, double* work) {
  if (!ctx || !kind || !ms || !work || idx < 0 || idx >= ctx->prof_count || ctx->profiling) return IVIT_ERR_INVALID_ARG;
  if (cudaEventElapsedTime(ms, ctx->prof_ev[2 * idx], ctx->prof_ev[2 * idx + 1]) != cudaSuccess) return IVIT_ERR_CUDA;
  *kind = ctx->prof_kind[idx];
  *work = ctx->prof_work[idx];
  return IVIT_OK;
}

const char* ivit_kernel_kind_name(int32_t kind) {
  switch (kind) {
    case KIND_GEMM_TC: return "gemm_tcgen05";
    case KIND_GEMM_SIMT: return "gemm_dp4a";
    case KIND_LAYERNORM: return "layernorm";
    case KIND_SHIFTMAX: return "shiftmax";
    case KIND_SHIFTGELU: return "shiftgelu";
    case KIND_GELU_TABLE: return "shiftgelu_table";
    case KIND_ATTENTION: return "attention_fused";
    case KIND_MOVE: return "data_movement";
    default: return "unknown";
  }
}

int ivit_patchify(ivit_ctx* ctx, const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi,
                  int64_t P, int64_t window, int8_t* out, int64_t ldout) {
  if (!ctx || !img || !out || B < 0 || C < 1 || P < 1) return IVIT_ERR_INVALID_ARG;
  if (P % 4 || Hi % P || Wi % P) return IVIT_ERR_UNSUPPORTED;
  if (window > 0 && ((Hi / P) % window || (Wi / P) % window)) return IVIT_ERR_INVALID_ARG;
  if (ldout < C * P * P) return IVIT_ERR_INVALID_ARG;
  if (!aligned16(img) || !aligned16(out) || ldout % 4 || Wi % 4) return IVIT_ERR_ALIGNMENT;
  return launch_patchify(ctx, img, B, C, Hi, Wi, P, window, out, ldout);
}

int ivit_gather_rows(ivit_ctx* ctx, const int8_t* src, int64_t ldsrc, const int32_t* index,
                     int64_t n_rows, int64_t width, int8_t* dst, int64_t lddst) {
  if (!ctx || !src || !index || !dst || n_rows < 0 || width < 1) return IVIT_ERR_INVALID_ARG;
  if (width % 16) return IVIT_ERR_UNSUPPORTED;
  if (!aligned16(src) || !aligned16(dst) || ldsrc % 16 || lddst % 16) return IVIT_ERR_ALIGNMENT;
  return launch_gather_rows(ctx, src, ldsrc, index, n_rows, width, dst, lddst);
}

int ivit_fill_rows(ivit_ctx* ctx, const int8_t* src_row, int64_t width, int8_t* dst,
                   int64_t group_stride, int64_t groups) {
  if (!ctx || !src_row || !dst || groups < 0 || width < 1) return IVIT_ERR_INVALID_ARG;
  if (width % 16) return IVIT_ERR_UNSUPPORTED;
  if (!aligned16(src_row) || !aligned16(dst) || group_stride % 16) return IVIT_ERR_ALIGNMENT;
  return launch_fill_rows(ctx, src_row, width, dst, group_stride, groups);
}

int ivit_token_mean(ivit_ctx* ctx, const int8_t* in, int64_t ldin, int64_t groups, int64_t T,
                    int64_t C, ivit_scale scale, int8_t* out, int64_t ldout) {
  if (!ctx || !in || !out || groups < 0 || T < 1 || C < 1) return IVIT_ERR_INVALID_ARG;
  if (!scale_ok(scale) || scale.mult_c) return IVIT_ERR_RANGE;
  if (T > (1 << 23)) return IVIT_ERR_RANGE;
  return launch_token_mean(ctx, in, ldin, groups, T, C, to_dev(scale), out, ldout);
}

int ivit_dyadic_from_double(double ratio, int32_t* mult, int32_t* shift) {
  if (!mult || !shift || !(ratio > 0.0) || !std::isfinite(ratio)) return IVIT_ERR_INVALID_ARG;
  int e = 0;
  const double mant = std::frexp(ratio, &e);
  long long b = std::llround(std::ldexp(mant, 31));
  int c = 31 - e;
  if (b == (1ll << 31)) { b = 1ll << 30; c -= 1; }
  if (c < 31 || c > 62) return IVIT_ERR_RANGE;
  *mult = (int32_t)b;
  *shift = c;
  return IVIT_OK;
}

int ivit_validate_exp_params(ivit_exp_params p, int64_t row_len, int32_t is_gelu) {
  if (row_len < 1) return IVIT_ERR_INVALID_ARG;
  return check_exp(p, row_len, is_gelu != 0);
}

int ivit_validate_scale(const int32_t* mult_host, const uint8_t* shift_host, int64_t n) {
  if (!mult_host || !shift_host || n < 0) return IVIT_ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i)
    if (mult_host[i] <= 0 || shift_host[i] < 31 || shift_host[i] > 62) return IVIT_ERR_RANGE;
  return IVIT_OK;
}

}  // extern "C"
