// Shared device helpers and the context of the integer-only ViT library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ivit.h"

namespace ivit {

constexpr int kProfMax = 8192;
enum KernelKind { KIND_GEMM_TC = 0, KIND_GEMM_SIMT, KIND_LAYERNORM, KIND_SHIFTMAX, KIND_SHIFTGELU, KIND_GELU_TABLE,
                  KIND_ATTENTION, KIND_MOVE, KIND_COUNT };
constexpr int kGeluTableSlots = 16;
constexpr int kRowCounters = 4096;     // row blocks a Dense launch with a row operator may have
constexpr int kRowStateStride = 32;    // words between the counters (and between the flags) of neighbouring row blocks: one 128-byte line each
constexpr size_t kRowStateBytes = 4 * (32 + 2 * (size_t)kRowCounters * kRowStateStride);
constexpr int kGeluTailRows = 2;      // rows a warp of the Dense kernel works on together in the ShiftGELU tail
constexpr int kGeluTailSmem = 16 * kGeluTailRows * 256;
constexpr int kGeluTableBytes = 128 * 256;  // [max(0,row max of x)] [x + 128] -> int8 output

struct GeluKey {
  int32_t I0, N, M, k_out, mult, shift;
  bool operator==(const GeluKey& o) const {
    return I0 == o.I0 && N == o.N && M == o.M && k_out == o.k_out && mult == o.mult && shift == o.shift;
  }
};

}  // namespace ivit

struct ivit_ctx {
  int device;
  cudaStream_t stream;
  int* status_host;  // mapped pinned memory: kernels write the first device-side error here
  int* status_dev;   // device view of the same word
  int8_t* gelu_tables;  // kGeluTableSlots tables on the device
  unsigned* sched_dev;  // two pairs of work counters of the attention kernel (behind the tables), used alternately
  unsigned* rowblk_dev; // row-operator state of the Dense kernels: kRowStateBytes (zero between launches)
  int row_fusion;       // non-zero (bit 0 LayerNorm, bit 1 ShiftGELU; default 0): LayerNorm / ShiftGELU run in the tail of the Dense kernel that produces their rows
  int rowop_fused;      // set by the Dense launcher when the kernel it launched runs the requested row operator
  int attn_gen;         // pair of the next launch
  ivit::GeluKey gelu_keys[ivit::kGeluTableSlots];
  int gelu_used;
  int gelu_next;
  uint64_t gelu_gen;    // bumped whenever a table slot is (re)built: graphs that point at the tables check it
  int64_t launches;
  int64_t pair_launches;   // Dense launches that ran on CTA pairs (ivit_ctx_pair_launch_count)
  int gemm_engine;
  int sm_count;
  void* tmap_encode;  // cuTensorMapEncodeTiled, resolved at context creation
  int gemm_pairs;     // CTA pairs (cta_group::2) for Dense layers with a long contraction (ivit_ctx_set_gemm_pairs)
  void* tmap_cache;   // encoded tensor maps by (address, extents, strides, box, swizzle); see make_tensor_map
  // ivit_vit_forward_host: input copies run on their own stream into two staging buffers (created on first use)
  cudaStream_t copy_stream;
  cudaEvent_t img_ready[2], img_free[2];
  uint64_t host_calls;
  // ivit_ctx_set_host_graph: the forward of ivit_vit_forward_host replayed as an instantiated CUDA graph, one per
  // staging buffer, captured at the third call that repeats the same arguments
  int host_graph;
  cudaGraphExec_t hg_exec[2];
  char* hg_key[2];          // model description, workspace and stream the graph was captured with
  size_t hg_key_bytes[2];
  size_t hg_key_cap[2];     // allocated size of hg_key (the buffers are reused from call to call)
  char* hg_scratch;         // key of the current call, compared with hg_key
  size_t hg_scratch_cap;
  uint64_t hg_gen[2];       // table generation the graph was captured at
  int hg_seen[2];           // calls seen with this key (-1: capture failed, launch kernel by kernel)
  int64_t hg_launches[2];   // kernels inside the graph
  // per-kernel timing session (ivit_ctx_profile_*)
  bool profiling;
  int prof_count;
  cudaEvent_t* prof_ev;   // 2 * kProfMax events, created on first use
  int* prof_kind;
  double* prof_work;
};

namespace ivit {

__device__ __forceinline__ int sat8(int v) { return max(-128, min(127, v)); }

// Round-half-up dyadic requantisation, Sec. 3.2: floor((a*m + 2^(s-1)) / 2^s) in 64 bits.
__device__ __forceinline__ int rq(int a, int m, int s) {
  long long p = (long long)a * (long long)m + (1ll << (s - 1));
  return (int)(p >> s);
}

// Same value, for a shift known to be >= 32 (the product's low word only feeds the carry).
__device__ __forceinline__ int rq_hi(int a, int m, int s) {
  long long p = (long long)a * (long long)m + (1ll << (s - 1));
  return (int)(p >> 32) >> (s - 32);
}

// Shifts are bounded to [31, 62]: with 0 < mult < 2^31 and |a| < 2^31 the requantised value then fits 32 bits.
__host__ __device__ __forceinline__ int clamp_shift(int s) { return s < 31 ? 31 : (s > 62 ? 62 : s); }

struct ScaleDev {
  const int32_t* mult_c;
  const uint8_t* shift_c;
  int mult;
  int shift;
  __device__ __forceinline__ int m(int c) const { return mult_c ? mult_c[c] : mult; }
  __device__ __forceinline__ int s(int c) const { return clamp_shift(shift_c ? (int)shift_c[c] : shift); }
};

inline ScaleDev to_dev(const ivit_scale& s) { return ScaleDev{s.mult_c, s.shift_c, s.mult, s.shift}; }

// Integer exponential of a non-positive argument, exp(S * I) in units of S * 2^-N with I0 = round(1 / S):
// Eq. (exp_shift) turns the base into 2 with log2(e) ~ (1.0111)b, so the exponent is -n / I0 with
// n = nd + ceil(nd / 2) - ceil(nd / 16) for nd = -I >= 0 (the arithmetic shifts of the negative I round towards
// -inf, which is what the two ceilings say); n = q * I0 + r splits it into an integer power of two and a
// fraction -r / I0 in (-1, 0], on which Eq. (linear) takes 2^x ~ 1 + x / 2: mantissa I0 - ceil(r / 2), scaled by
// 2^(N - q).  32-bit: nd < 2^15, I0 <= 2^15, N <= 24.
__device__ __forceinline__ unsigned shiftexp(int I, int I0, int N) {
  const unsigned nd = (unsigned)(-I);
  const unsigned n = nd + ((nd + 1u) >> 1) - ((nd + 15u) >> 4);
  const unsigned q = n / (unsigned)I0;
  const unsigned r = n - q * (unsigned)I0;
  const unsigned mant = (unsigned)I0 - ((r + 1u) >> 1);
  if (q <= (unsigned)N) return mant << ((unsigned)N - q);
  const unsigned down = q - (unsigned)N;
  return down >= 31u ? 0u : mant >> down;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }

inline bool scale_ok(const ivit_scale& s) {
  if (s.mult_c) return s.shift_c != nullptr;
  return s.mult > 0 && s.shift >= 31 && s.shift <= 62;
}

// Brackets one kernel launch: counts it and, inside a timing session, records an event pair.
struct LaunchScope {
  ivit_ctx* ctx;
  int slot;
  LaunchScope(ivit_ctx* c, int kind, double work) : ctx(c), slot(-1) {
    if (c->profiling && c->prof_count < kProfMax) {
      slot = c->prof_count++;
      c->prof_kind[slot] = kind;
      c->prof_work[slot] = work;
      cudaEventRecord(c->prof_ev[2 * slot], c->stream);
    }
  }
  int done() {
    ctx->launches += 1;
    if (slot >= 0) cudaEventRecord(ctx->prof_ev[2 * slot + 1], ctx->stream);
    return cudaGetLastError() == cudaSuccess ? IVIT_OK : IVIT_ERR_CUDA;
  }
};

// ---- programmatic dependent launch ---------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialization: the next kernel
// of the stream may be scheduled (and run its set-up) while this one drains.  A kernel therefore
// calls pdl_wait() before it reads or writes anything another kernel may touch, and pdl_trigger()
// to let its successor be scheduled early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                            Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same for a kernel whose CTAs work in pairs: clusters of two CTAs along x.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k_pair(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// launchers implemented in the kernel files ---------------------------------------------

// What a Dense launch does with a block of output rows once all its channel tiles are stored (see rowops.cuh).
struct RowOpArgs {
  int kind;              // 0: nothing; 1: I-LayerNorm of the rows into ln_out; 2: ShiftGELU of the rows, in place
  unsigned* counters;    // [2] CTAs finished; from word 32 on one arrival counter per row block, then one ready flag per
                         // row block, each on a 128-byte line of its own; all zero between launches
  // kind 1
  ScaleDev gs;           // per-channel (or per-tensor) multiplier and shift of the affine requantisation
  const int32_t* beta;
  int M_ln;
  int8_t* ln_out;
  int64_t ld_ln;
  unsigned mean_magic;   // floor(2^32 / 2C) + 1
  int vec;               // per-channel arrays aligned for 16-byte loads
  // kind 2
  const int8_t* table;   // 128 x 256 bytes: [max(0, row maximum)][x + 128]
};

struct GemmEpilogue {
  const int32_t* bias;       // [N] (linear) or nullptr
  const int32_t* bias32;     // [bias_batches, Ma, ldbias] (matmul) or nullptr
  int64_t ldbias, bias_batches;
  ScaleDev scale;
  const int8_t* res;
  int64_t ldres, res_rows;
  ScaleDev res_scale;
  void* out;
  int64_t ldo;
  int out_dtype;
  int64_t group_rows, group_stride;
  const int8_t* act_table;   // int8 outputs only: out = act_table[sat8(value) + 128] (256 entries on the device) or nullptr
  RowOpArgs rop;             // row operator wanted on the finished output rows (kind 0: none); the launcher sets
                             // ctx->rowop_fused when the kernel it launched runs it, else the caller launches it
};

struct GemmProblem {
  const int8_t* A; int64_t lda, sAo, sAi;
  const int8_t* B; int64_t ldb, sBo, sBi;
  int transB;              // 1: B is [N,K]; 0: B is [K,N]
  int64_t sCo, sCi;        // batch offsets of out (elements)
  int64_t batches_outer, batches_inner;
  int64_t M, N, K;
  GemmEpilogue epi;
};

int launch_gemm_simt(ivit_ctx* ctx, const GemmProblem& g);
// Returns IVIT_ERR_UNSUPPORTED when the shape does not qualify for the tensor-core kernel.
int launch_gemm_tc(ivit_ctx* ctx, const GemmProblem& g);
int launch_gemm(ivit_ctx* ctx, const GemmProblem& g);
// Per-device kernel attributes (shared-memory limits) of the tensor-core kernels, for the current device.
int gemm_tc_prepare_device();
void tmap_cache_free(ivit_ctx* ctx);
int attention_prepare_device();
// Fused Q K^T -> requant -> Shiftmax -> P V -> requant; IVIT_ERR_UNSUPPORTED when the shape does not qualify.
int launch_attention_fused(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O);

int launch_layernorm(ivit_ctx* ctx, const void* in, int in_dtype, int64_t ldin, ScaleDev gs,
                     const int32_t* beta, int M_ln, int8_t* out, int64_t ldout, int64_t rows, int64_t C);
int launch_shiftmax(ivit_ctx* ctx, const void* in, int in_dtype, int64_t ldin, const int32_t* bias32,
                    int64_t ldbias, int64_t bias_rows, ScaleDev pre, ivit_exp_params p, int8_t* out,
                    int64_t ldout, int64_t rows, int64_t d);
int launch_shiftmax_direct(ivit_ctx* ctx, const int32_t* in, int64_t ldin, ivit_exp_params p, int8_t* out,
                           int64_t ldout, int64_t rows, int64_t d);
// The 128 x 256 ShiftGELU table of (p, post) on the device (built on first use, cached in the context).
int gelu_table_for(ivit_ctx* ctx, ivit_exp_params p, ivit_scale post, const int8_t** table);
// Row `127` of the ShiftGELU table of (p, post) on the device (built on first use): the static-maximum variant.
int gelu_static_row(ivit_ctx* ctx, ivit_exp_params p, ivit_scale post, const int8_t** row);
int launch_shiftgelu_static(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p, ivit_scale post,
                            int8_t* out, int64_t ldout, int64_t rows, int64_t cols);
int launch_shiftgelu(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p, ivit_scale post,
                     int8_t* out, int64_t ldout, int64_t rows, int64_t cols);
int launch_patchify(ivit_ctx* ctx, const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi,
                    int64_t P, int64_t window, int8_t* out, int64_t ldout);
int launch_gather_rows(ivit_ctx* ctx, const int8_t* src, int64_t ldsrc, const int32_t* index,
                       int64_t n_rows, int64_t width, int8_t* dst, int64_t lddst);
int launch_fill_rows(ivit_ctx* ctx, const int8_t* src_row, int64_t width, int8_t* dst,
                     int64_t group_stride, int64_t groups);
int launch_token_mean(ivit_ctx* ctx, const int8_t* in, int64_t ldin, int64_t groups, int64_t T,
                      int64_t C, ScaleDev scale, int8_t* out, int64_t ldout);

}  // namespace ivit
