// I-LayerNorm (Sec. 3.5), Shiftmax (Algorithm 1) and ShiftGELU (Algorithm 2) kernels, sm_100a.
// One warp owns one row; rows are read once from HBM as coalesced 32-bit words and
// kept in registers between the reduction and the output pass.
#include "rowops.cuh"
#include <type_traits>

namespace ivit {

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned warp_sum_u(unsigned v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ long long warp_sum_ll(long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_max(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Eq. (iterative): x_{i+1} = (x_i + floor(n / x_i)) >> 1 from x_0 = 2^floor(bit(n)/2); the first
// step is taken unconditionally, the following nine only while they decrease (leaving the loop
// at the first non-decrease gives the same value as holding it for the remaining steps).
__device__ __forceinline__ unsigned isqrt_u32(unsigned n) {
  if (n == 0) return 0;
  int bits = 32 - __clz(n);
  unsigned x = 1u << (bits >> 1);
  x = (x + n / x) >> 1;
#pragma unroll 1
  for (int i = 1; i < 10; ++i) {
    unsigned nx = (x + n / x) >> 1;
    if (nx >= x) break;
    x = nx;
  }
  return x;
}
__device__ __forceinline__ unsigned long long isqrt_u64(unsigned long long n) {
  if (n == 0) return 0;
  int bits = 64 - __clzll(n);
  unsigned long long x = 1ull << (bits >> 1);
  x = (x + n / x) >> 1;
#pragma unroll 1
  for (int i = 1; i < 10; ++i) {
    unsigned long long nx = (x + n / x) >> 1;
    if (nx >= x) break;
    x = nx;
  }
  return x;
}

// Four int32 values saturated to int8 and packed, x0 in the low byte.
__device__ __forceinline__ unsigned pack_sat8_u(int x0, int x1, int x2, int x3) {
  unsigned t, d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(x3), "r"(x2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(x1), "r"(x0), "r"(t));
  return d;
}

__device__ __forceinline__ int floordiv_pos(int a, int b) {  // b > 0
  int q = a / b;
  return (a - q * b < 0) ? q - 1 : q;
}

// ------------------------------------------------------------------ I-LayerNorm, int8 input

// WPL = 32-bit words of the row held per lane (C <= 128 * WPL).
template <int WPL>
__global__ void __launch_bounds__(256) layernorm_i8_kernel(const int8_t* __restrict__ in, int64_t ldin,
                                                           ScaleDev gs, const int32_t* __restrict__ beta,
                                                           int M_ln, int8_t* __restrict__ out, int64_t ldout,
                                                           int64_t rows, int C) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int nwords = C >> 2;
  for (int64_t r = warp; r < rows; r += nwarps) {
    const int* src = reinterpret_cast<const int*>(in + r * ldin);
    int w[WPL];
    int s1 = 0, s2 = 0;
#pragma unroll
    for (int i = 0; i < WPL; ++i) {
      const int idx = lane + 32 * i;
      w[i] = idx < nwords ? __ldg(src + idx) : 0;
      s1 = __dp4a(w[i], 0x01010101, s1);
      s2 = __dp4a(w[i], w[i], s2);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    const int mu = floordiv_pos(2 * s1 + C, 2 * C);
    // sum (x - mu)^2 = sum x^2 - 2 mu sum x + C mu^2, exactly
    const long long V = (long long)s2 - 2ll * mu * s1 + (long long)C * mu * mu;
    const unsigned sd = isqrt_u32((unsigned)V);
    const int F = sd == 0 ? 0 : (int)((1u << M_ln) / sd);
    int* dst = reinterpret_cast<int*>(out + r * ldout);
#pragma unroll
    for (int i = 0; i < WPL; ++i) {
      const int idx = lane + 32 * i;
      if (idx < nwords) {
        unsigned packed = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int c = idx * 4 + b;
          const int x = (int)(int8_t)(w[i] >> (8 * b));
          int v = rq((x - mu) * F, gs.m(c), gs.s(c));
          if (beta) v += __ldg(beta + c);
          packed |= (unsigned)(sat8(v) & 0xff) << (8 * b);
        }
        dst[idx] = (int)packed;
      }
    }
  }
}

// Rows of up to 1024 channels: a warp takes R rows at a time (layernorm_rows); the per-channel constants are
// prepared once per block in shared memory, before the wait for the previous kernel (they are parameters, not
// results).
template <int WPL, int R>
__global__ void __launch_bounds__(128) layernorm_rows_kernel(const int8_t* __restrict__ in, int64_t ldin, ScaleDev gs,
                                                             const int32_t* __restrict__ beta, int M_ln,
                                                             int8_t* __restrict__ out, int64_t ldout, int64_t rows, int C,
                                                             unsigned mean_magic, int vec) {
  extern __shared__ int4 ln_consts[];   // [3][C / 4]: multipliers, shifts, addends (or betas)
  pdl_trigger();
  const int nwords = C >> 2;
  int4* sm_m = ln_consts;
  int4* sm_s = ln_consts + nwords;
  int4* sm_b = ln_consts + 2 * nwords;
  bool fast = ln_stage_consts(gs, beta, nwords, vec, sm_m, sm_s, sm_b, threadIdx.x, blockDim.x);
  fast = __syncthreads_and(fast) != 0;
  if (fast) ln_fold_consts(nwords, sm_s, sm_b, threadIdx.x, blockDim.x);
  __syncthreads();
  const LnConsts k{sm_m, sm_s, sm_b, fast};
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t r0 = warp * R; r0 < rows; r0 += nwarps * R) {
    const int nrows = (int)(rows - r0 < R ? rows - r0 : R);
    layernorm_rows<WPL, R, false>(in + r0 * ldin, ldin, nrows, C, M_ln, mean_magic, k, out + r0 * ldout, ldout, lane);
  }
}

// Any C (multiple of 4): the row is read again from cache for the output pass.
__global__ void __launch_bounds__(256) layernorm_i8_long_kernel(const int8_t* __restrict__ in, int64_t ldin,
                                                                ScaleDev gs, const int32_t* __restrict__ beta,
                                                                int M_ln, int8_t* __restrict__ out,
                                                                int64_t ldout, int64_t rows, int C) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int nwords = C >> 2;
  for (int64_t r = warp; r < rows; r += nwarps) {
    const int* src = reinterpret_cast<const int*>(in + r * ldin);
    int s1 = 0, s2 = 0;
    for (int idx = lane; idx < nwords; idx += 32) {
      const int w = __ldg(src + idx);
      s1 = __dp4a(w, 0x01010101, s1);
      s2 = __dp4a(w, w, s2);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    const int mu = floordiv_pos(2 * s1 + C, 2 * C);
    const long long V = (long long)s2 - 2ll * mu * s1 + (long long)C * mu * mu;
    const unsigned sd = isqrt_u32((unsigned)V);
    const int F = sd == 0 ? 0 : (int)((1u << M_ln) / sd);
    int* dst = reinterpret_cast<int*>(out + r * ldout);
    for (int idx = lane; idx < nwords; idx += 32) {
      const int w = __ldg(src + idx);
      unsigned packed = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int c = idx * 4 + b;
        const int x = (int)(int8_t)(w >> (8 * b));
        int v = rq((x - mu) * F, gs.m(c), gs.s(c));
        if (beta) v += __ldg(beta + c);
        packed |= (unsigned)(sat8(v) & 0xff) << (8 * b);
      }
      dst[idx] = (int)packed;
    }
  }
}

// int32 input (|x| <= 2^20): 64-bit sums, two passes over the row.
__global__ void __launch_bounds__(256) layernorm_i32_kernel(const int32_t* __restrict__ in, int64_t ldin,
                                                            ScaleDev gs, const int32_t* __restrict__ beta,
                                                            int M_ln, int8_t* __restrict__ out, int64_t ldout,
                                                            int64_t rows, int C) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t r = warp; r < rows; r += nwarps) {
    const int32_t* src = in + r * ldin;
    long long s1 = 0;
    for (int c = lane; c < C; c += 32) s1 += __ldg(src + c);
    s1 = warp_sum_ll(s1);
    const long long num = 2 * s1 + C, den = 2ll * C;
    long long mu = num / den;
    if (num - mu * den < 0) mu -= 1;
    long long V = 0;
    for (int c = lane; c < C; c += 32) {
      const long long y = (long long)__ldg(src + c) - mu;
      V += y * y;
    }
    V = warp_sum_ll(V);
    const unsigned long long sd = isqrt_u64((unsigned long long)V);
    const long long F = sd == 0 ? 0 : (long long)((1ull << M_ln) / sd);
    for (int c = lane; c < C; c += 32) {
      const long long y = (long long)__ldg(src + c) - mu;
      int v = rq((int)(y * F), gs.m(c), gs.s(c));
      if (beta) v += __ldg(beta + c);
      out[r * ldout + c] = (int8_t)sat8(v);
    }
  }
}

int launch_layernorm(ivit_ctx* ctx, const void* in, int in_dtype, int64_t ldin, ScaleDev gs,
                     const int32_t* beta, int M_ln, int8_t* out, int64_t ldout, int64_t rows, int64_t C) {
  if (rows == 0) return IVIT_OK;
  const int threads = 256, wpb = threads / 32;
  const int64_t want = (rows + wpb - 1) / wpb;
  const int grid = (int)(want < (int64_t)ctx->sm_count * 8 ? want : (int64_t)ctx->sm_count * 8);
  cudaStream_t st = ctx->stream;
  LaunchScope ls(ctx, KIND_LAYERNORM, (double)rows * (double)C * (in_dtype == IVIT_I32 ? 5.0 : 2.0));
  if (in_dtype == IVIT_I32) {
    launch_k(layernorm_i32_kernel, dim3(grid), dim3(threads), 0, st, (const int32_t*)in, ldin, gs, beta, M_ln, out, ldout, rows, (int)C);
    return ls.done();
  }
  const int8_t* x = (const int8_t*)in;
  const int wpl = (int)((C / 4 + 31) / 32);
  if (wpl <= 8) {
    // four rows per warp (eight for rows of at most 128 channels, two above 512): short per-warp work lets the blocks of this
    // kernel slip into the tail of the kernel before it and out of the way of the one after it
    const int rpw = wpl <= 1 ? 8 : (wpl <= 4 ? 4 : 2), tb = 128;
    const int64_t warps = (rows + rpw - 1) / rpw;
    const int64_t wantb = (warps + tb / 32 - 1) / (tb / 32);
    const int gridb = (int)(wantb < (int64_t)ctx->sm_count * 12 ? wantb : (int64_t)ctx->sm_count * 12);
    const unsigned magic = (unsigned)(0x100000000ull / (unsigned long long)(2 * C)) + 1u;
    const int vec = gs.mult_c && gs.shift_c && !(reinterpret_cast<uintptr_t>(gs.mult_c) & 15) && !(reinterpret_cast<uintptr_t>(gs.shift_c) & 3) &&
                    !(reinterpret_cast<uintptr_t>(beta) & 15);
    const size_t cbytes = (size_t)(C / 4) * 3 * sizeof(int4);
    if (wpl <= 1) launch_k(layernorm_rows_kernel<1, 8>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    else if (wpl <= 2) launch_k(layernorm_rows_kernel<2, 4>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    else if (wpl <= 3) launch_k(layernorm_rows_kernel<3, 4>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    else if (wpl <= 4) launch_k(layernorm_rows_kernel<4, 4>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    else if (wpl <= 6) launch_k(layernorm_rows_kernel<6, 2>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    else launch_k(layernorm_rows_kernel<8, 2>, dim3(gridb), dim3(tb), cbytes, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C, magic, vec);
    return ls.done();
  }
  if (wpl <= 12) launch_k(layernorm_i8_kernel<12>, dim3(grid), dim3(threads), 0, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C);
  else launch_k(layernorm_i8_long_kernel, dim3(grid), dim3(threads), 0, st, x, ldin, gs, beta, M_ln, out, ldout, rows, (int)C);
  return ls.done();
}

// ------------------------------------------------------------------ Shiftmax

// Packed int8x4 word `idx` of row r.  I8: straight from memory.  I32: requantise four
// accumulators (+ bias) to int8 first, so both entry forms run the same row algorithm.
template <bool FROM_I32>
struct RowLoader {
  const void* in;
  int64_t ldin;
  const int32_t* bias32;
  int64_t ldbias, bias_rows;
  int pre_m, pre_s;
  __device__ __forceinline__ int load(int64_t r, int idx) const {
    if (!FROM_I32) {
      return __ldg(reinterpret_cast<const int*>((const int8_t*)in + r * ldin) + idx);
    } else {
      const int4 a = __ldg(reinterpret_cast<const int4*>((const int32_t*)in + r * ldin) + idx);
      int4 b = make_int4(0, 0, 0, 0);
      if (bias32) b = __ldg(reinterpret_cast<const int4*>(bias32 + (r % bias_rows) * ldbias) + idx);
      unsigned p = (unsigned)(sat8(rq(a.x + b.x, pre_m, pre_s)) & 0xff);
      p |= (unsigned)(sat8(rq(a.y + b.y, pre_m, pre_s)) & 0xff) << 8;
      p |= (unsigned)(sat8(rq(a.z + b.z, pre_m, pre_s)) & 0xff) << 16;
      p |= (unsigned)(sat8(rq(a.w + b.w, pre_m, pre_s)) & 0xff) << 24;
      return (int)p;
    }
  }
};

// WPL words per lane in registers (d <= 128 * WPL); WPL == 0: re-read the row for each pass.
// Bytes are handled as biased values u = x + 128 (x ^ 0x80), so that one byte permute yields the table index:
// ShiftExp(x - max) = tab[max - x] = tab[(max + 128) - u].  Positions past d hold u = 0 (x = -128); they never
// win the maximum and their table entries are taken out of the sum again.
template <int WPL, int ROWS, bool FROM_I32>
__global__ void __launch_bounds__(256) shiftmax_kernel(RowLoader<FROM_I32> ld, ivit_exp_params p,
                                                       int8_t* __restrict__ out, int64_t ldout,
                                                       int64_t rows, int d) {
  pdl_trigger();
  pdl_wait();
  __shared__ unsigned exp_tab[256];  // ShiftExp(-i), i = I_max - I in [0, 255]
  for (int i = threadIdx.x; i < 256; i += blockDim.x) exp_tab[i] = shiftexp(-i, p.I0, p.N);
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int nwords = (d + 3) >> 2;
  const int nwords_out = ((d + 15) >> 4) << 2;  // zero-fill up to the next multiple of 16
  const int npad = nwords * 4 - d;              // bytes past d in the last word
  constexpr int W = WPL > 0 ? WPL : 1;
  constexpr int R = WPL > 0 ? ROWS : 1;         // rows a warp works on together (their reciprocals in parallel lanes)
  const int iters = WPL > 0 ? WPL : (nwords_out + 31) / 32;
  // biased word idx of row r: bytes past d (and whole words past the row) read as 0
  auto load_biased = [&](int64_t r, int idx) -> unsigned {
    if (idx >= nwords) return 0u;
    unsigned v = (unsigned)ld.load(r, idx) ^ 0x80808080u;
    if (idx == nwords - 1 && npad) v &= 0xffffffffu >> (8 * npad);
    return v;
  };
  for (int64_t r0 = warp * R; r0 < rows; r0 += nwarps * R) {
    unsigned e[R][W][4];
    unsigned my_sum = 1, my_mxu = 0;
#pragma unroll
    for (int q = 0; q < R; ++q) {
      const int64_t r = r0 + q < rows ? r0 + q : rows - 1;   // a row past the end repeats the last one (not stored)
      unsigned w[W];
      // pass 1: row max
      unsigned mxu = 0;
#pragma unroll
      for (int i = 0; i < iters; ++i) {
        const unsigned v = load_biased(r, lane + 32 * i);
        if (WPL > 0) w[i] = v;
        mxu = max(max(mxu, __byte_perm(v, 0, 0x4440)), max(__byte_perm(v, 0, 0x4441), max(__byte_perm(v, 0, 0x4442), v >> 24)));
      }
      mxu = __reduce_max_sync(0xffffffffu, mxu);   // biased maximum = I_max + 128
      // pass 2: sum of ShiftExp(I - I_max): entry (I_max + 128) - u
      const uint8_t* tmx = reinterpret_cast<const uint8_t*>(exp_tab) + 4 * mxu;
      unsigned sum = 0;
#pragma unroll
      for (int i = 0; i < iters; ++i) {
        const unsigned v = WPL > 0 ? w[i] : load_biased(r, lane + 32 * i);
        unsigned e0 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4440));
        unsigned e1 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4441));
        unsigned e2 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4442));
        unsigned e3 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)(v >> 24));
        if (WPL > 0) { e[q][i][0] = e0; e[q][i][1] = e1; e[q][i][2] = e2; e[q][i][3] = e3; }
        sum += (e0 + e1) + (e2 + e3);
      }
      sum = __reduce_add_sync(0xffffffffu, sum);
      // every position past d of the 32 * iters words counted exp_tab[I_max + 128]: take them out
      sum -= (unsigned)(32 * iters * 4 - d) * exp_tab[mxu];
      if (lane == q) { my_sum = sum; my_mxu = mxu; }
    }
    // Eq. (IntDiv): one reciprocal per row (lane q for row q), M = 45:
    // (floor(2^45 / sum) * e) >> (45 - (k_out - 1)) == umulhi(factor, e) >> (14 - k_out) since factor <= 2^31.
    const unsigned my_factor = (unsigned)((1ull << 45) / (unsigned long long)my_sum);
    const int osh = 14 - p.k_out;
    const int omax = (1 << (p.k_out - 1)) - 1;   // the one possible 2^(k_out-1) is clamped
#pragma unroll
    for (int q = 0; q < R; ++q) {
      const unsigned factor = __shfl_sync(0xffffffffu, my_factor, q);
      const unsigned mxu = __shfl_sync(0xffffffffu, my_mxu, q);
      const int64_t r = r0 + q;
      if (r >= rows) break;
      const uint8_t* tmx = reinterpret_cast<const uint8_t*>(exp_tab) + 4 * mxu;
      int* dst = reinterpret_cast<int*>(out + r * ldout);
#pragma unroll
      for (int i = 0; i < iters; ++i) {
        const int idx = lane + 32 * i;
        if (idx < nwords_out) {
          unsigned e0, e1, e2, e3;
          if (WPL > 0) {
            e0 = e[q][i][0]; e1 = e[q][i][1]; e2 = e[q][i][2]; e3 = e[q][i][3];
          } else {
            const unsigned v = load_biased(r, idx);
            e0 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4440));
            e1 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4441));
            e2 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(v, 0, 0x4442));
            e3 = *reinterpret_cast<const unsigned*>(tmx - 4 * (int)(v >> 24));
          }
          unsigned packed = pack_sat8_u(min((int)(__umulhi(factor, e0) >> osh), omax), min((int)(__umulhi(factor, e1) >> osh), omax),
                                        min((int)(__umulhi(factor, e2) >> osh), omax), min((int)(__umulhi(factor, e3) >> osh), omax));
          // positions past d are written as zero
          if (idx >= nwords) packed = 0;
          else if (idx == nwords - 1 && npad) packed &= 0xffffffffu >> (8 * npad);
          dst[idx] = (int)packed;
        }
      }
    }
  }
}

template <bool FROM_I32>
static void shiftmax_dispatch(RowLoader<FROM_I32> ld, ivit_exp_params p, int8_t* out, int64_t ldout,
                              int64_t rows, int d, int grid, cudaStream_t st) {
  const int wpl = (((d + 15) / 16) * 4 + 31) / 32;
  if (wpl <= 2) launch_k(shiftmax_kernel<2, 4, FROM_I32>, dim3(grid), dim3(256), 0, st, ld, p, out, ldout, rows, d);
  else if (wpl <= 5) launch_k(shiftmax_kernel<5, 2, FROM_I32>, dim3(grid), dim3(256), 0, st, ld, p, out, ldout, rows, d);
  else if (wpl <= 8) launch_k(shiftmax_kernel<8, 1, FROM_I32>, dim3(grid), dim3(256), 0, st, ld, p, out, ldout, rows, d);
  else if (wpl <= 16) launch_k(shiftmax_kernel<16, 1, FROM_I32>, dim3(grid), dim3(256), 0, st, ld, p, out, ldout, rows, d);
  else launch_k(shiftmax_kernel<0, 1, FROM_I32>, dim3(grid), dim3(256), 0, st, ld, p, out, ldout, rows, d);
}

int launch_shiftmax(ivit_ctx* ctx, const void* in, int in_dtype, int64_t ldin, const int32_t* bias32,
                    int64_t ldbias, int64_t bias_rows, ScaleDev pre, ivit_exp_params p, int8_t* out,
                    int64_t ldout, int64_t rows, int64_t d) {
  if (rows == 0) return IVIT_OK;
  const int64_t want = (rows + 7) / 8;
  const int grid = (int)(want < (int64_t)ctx->sm_count * 8 ? want : (int64_t)ctx->sm_count * 8);
  LaunchScope ls(ctx, KIND_SHIFTMAX, (double)rows * (double)d * (in_dtype == IVIT_I32 ? 5.0 : 2.0));
  if (in_dtype == IVIT_I8) {
    RowLoader<false> ld{in, ldin, nullptr, 0, 1, 0, 1};
    shiftmax_dispatch<false>(ld, p, out, ldout, rows, (int)d, grid, ctx->stream);
  } else {
    RowLoader<true> ld{in, ldin, bias32, ldbias, bias_rows < 1 ? 1 : bias_rows, pre.mult, clamp_shift(pre.shift)};
    shiftmax_dispatch<true>(ld, p, out, ldout, rows, (int)d, grid, ctx->stream);
  }
  return ls.done();
}

// ------------------------------------------------------------------ Shiftmax on int32 scores (Algorithm 1, wide form)

struct DirectConsts {
  unsigned I0;
  int N;
  int osh;                       // M - (k_out - 1)
  int omax;                      // 2^(k_out-1) - 1
  int M;
  unsigned long long magic;      // reciprocal of I0 scaled by 2^64, rounded up (unused when I0 == 1)
  unsigned long long zero_from;  // I0 * (N + 29): from here on every bit of I_b < 2^29 is shifted out
  // 32-bit form (taken when exponentials, their sum and the reciprocal all fit 32 bits and zero_from <= 2^31)
  unsigned nd_cut;               // I_max - I >= nd_cut implies -I_p >= zero_from; below it -I_p fits 32 bits
  unsigned m_hi, m_lo;           // the two words of magic
};

// ShiftExp(I - I_max) for nd = I_max - I (0 .. 2^32 - 1).  The arithmetic shifts of the negative I_delta round
// towards -inf, so -I_p = nd + ceil(nd / 2) - ceil(nd / 16).  Below zero_from the quotient by I0 is < 53 and
// (-I_p) * I0 < 2^64, which makes the multiply-high by floor(2^64 / I0) + 1 the exact floor quotient.
__device__ __forceinline__ unsigned long long shiftexp_wide(unsigned nd, const DirectConsts& c) {
  const unsigned up2 = (nd >> 1) + (nd & 1u);
  const unsigned up16 = (nd >> 4) + ((nd & 15u) != 0u);
  const unsigned long long n = (unsigned long long)nd + up2 - up16;
  if (n >= c.zero_from) return 0ull;
  const unsigned q = c.I0 == 1u ? (unsigned)n : (unsigned)__umul64hi(n, c.magic);
  const unsigned r = (unsigned)(n - (unsigned long long)q * c.I0);   // 0 <= r < I0
  const unsigned Ib = c.I0 - ((r + 1) >> 1);                         // ((-r) >> 1) + I0
  return q <= (unsigned)c.N ? (unsigned long long)Ib << (c.N - q) : (unsigned long long)(Ib >> (q - c.N));
}

// The same in 32-bit arithmetic: the quotient is the high word of n * magic, taken from two 32-bit products.
__device__ __forceinline__ unsigned shiftexp_narrow(unsigned nd, const DirectConsts& c) {
  if (nd >= c.nd_cut) return 0u;
  const unsigned n = nd + ((nd >> 1) + (nd & 1u)) - ((nd >> 4) + ((nd & 15u) != 0u));
  if (n >= (unsigned)c.zero_from) return 0u;
  const unsigned q = c.I0 == 1u ? n : (unsigned)(((unsigned long long)n * c.m_hi + __umulhi(n, c.m_lo)) >> 32);
  const unsigned r = n - q * c.I0;
  const unsigned Ib = c.I0 - ((r + 1) >> 1);
  return q <= (unsigned)c.N ? Ib << (c.N - q) : Ib >> (q - c.N);
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One warp per row.  WPL groups of four scores per lane stay in registers as their exponentials
// (d <= 128 * WPL); WPL == 0 reads the row three times instead.
// NARROW: every exponential, the row sum and the reciprocal fit 32 bits (checked by the launcher).
template <int WPL, bool NARROW>
__global__ void __launch_bounds__(256) shiftmax_direct_kernel(const int32_t* __restrict__ in, int64_t ldin,
                                                              DirectConsts c, int8_t* __restrict__ out,
                                                              int64_t ldout, int64_t rows, int d) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int ngroups = (d + 3) >> 2;                // int4 groups that hold scores
  const int nwords_out = ((d + 15) >> 4) << 2;     // output words, zero-filled up to the next multiple of 16 columns
  constexpr int W = WPL > 0 ? WPL : 1;
  const int iters = WPL > 0 ? WPL : (nwords_out + 31) / 32;
  for (int64_t r = warp; r < rows; r += nwarps) {
    const int4* src = reinterpret_cast<const int4*>(in + r * ldin);
    // pass 1: row maximum (positions past d never count)
    int mx = INT_MIN;
    int4 x[W];
#pragma unroll
    for (int i = 0; i < iters; ++i) {
      const int g = lane + 32 * i;
      int4 v = make_int4(INT_MIN, INT_MIN, INT_MIN, INT_MIN);
      if (g < ngroups) {
        v = __ldg(src + g);
        if (4 * g + 1 >= d) v.y = INT_MIN;
        if (4 * g + 2 >= d) v.z = INT_MIN;
        if (4 * g + 3 >= d) v.w = INT_MIN;
      }
      if (WPL > 0) x[i] = v;
      mx = max(max(mx, max(v.x, v.y)), max(v.z, v.w));
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    // exponentials of group g (0 for positions past d)
    using E = typename std::conditional<NARROW, unsigned, unsigned long long>::type;
    auto one = [&](int v) -> E {
      if constexpr (NARROW) return shiftexp_narrow((unsigned)mx - (unsigned)v, c);
      else return shiftexp_wide((unsigned)mx - (unsigned)v, c);
    };
    auto exps = [&](int g, const int4& v, E* e) {
      e[0] = 4 * g + 0 < d ? one(v.x) : (E)0;
      e[1] = 4 * g + 1 < d ? one(v.y) : (E)0;
      e[2] = 4 * g + 2 < d ? one(v.z) : (E)0;
      e[3] = 4 * g + 3 < d ? one(v.w) : (E)0;
    };
    // pass 2: sum
    E e[W][4];
    E sum = 0;
#pragma unroll
    for (int i = 0; i < iters; ++i) {
      const int g = lane + 32 * i;
      E t[4] = {0, 0, 0, 0};
      if (g < ngroups) exps(g, WPL > 0 ? x[i] : __ldg(src + g), t);
      if (WPL > 0) { e[i][0] = t[0]; e[i][1] = t[1]; e[i][2] = t[2]; e[i][3] = t[3]; }
      sum += (t[0] + t[1]) + (t[2] + t[3]);
    }
    // the row sum is >= I0 * 2^N: the maximum contributes exactly that
    if constexpr (NARROW) sum = __reduce_add_sync(0xffffffffu, sum);
    else sum = warp_sum_u64(sum);
    // Eq. (IntDiv); factor * e <= 2^M < 2^63.  NARROW: factor < 2^32 and M - (k_out - 1) >= 32, so the product's
    // high word shifted by the rest is the same value.
    const E factor = (E)((1ull << c.M) / (unsigned long long)sum);
    auto prob = [&](E t) -> int {
      if constexpr (NARROW) return min((int)(__umulhi(factor, t) >> (c.osh - 32)), c.omax);
      else return min((int)((factor * t) >> c.osh), c.omax);
    };
    // pass 3: outputs
    int* dst = reinterpret_cast<int*>(out + r * ldout);
#pragma unroll
    for (int i = 0; i < iters; ++i) {
      const int g = lane + 32 * i;
      if (g < nwords_out) {
        E t[4] = {0, 0, 0, 0};
        if (WPL > 0) { t[0] = e[i][0]; t[1] = e[i][1]; t[2] = e[i][2]; t[3] = e[i][3]; }
        else if (g < ngroups) exps(g, __ldg(src + g), t);
        dst[g] = (int)pack_sat8_u(prob(t[0]), prob(t[1]), prob(t[2]), prob(t[3]));
      }
    }
  }
}

int launch_shiftmax_direct(ivit_ctx* ctx, const int32_t* in, int64_t ldin, ivit_exp_params p, int8_t* out,
                           int64_t ldout, int64_t rows, int64_t d) {
  if (rows == 0) return IVIT_OK;
  DirectConsts c;
  c.I0 = (unsigned)p.I0; c.N = p.N; c.M = p.M;
  c.osh = p.M - (p.k_out - 1);
  c.omax = (1 << (p.k_out - 1)) - 1;
  // floor((2^64 - 1) / I0) + 1: floor(2^64 / I0) + 1, or exactly 2^64 / I0 when I0 is a power of two (both give the floor quotient)
  c.magic = p.I0 > 1 ? ~0ull / (unsigned long long)p.I0 + 1ull : 0ull;
  c.zero_from = (unsigned long long)p.I0 * (unsigned long long)(p.N + 29);
  c.m_hi = (unsigned)(c.magic >> 32); c.m_lo = (unsigned)c.magic;
  // -I_p >= (23 / 16) nd - 1: from nd_cut on it is at least zero_from; below it -I_p <= 1.5 nd_cut + 1 < 2^32
  c.nd_cut = (unsigned)(((c.zero_from + 1) * 16 + 22) / 23);
  const unsigned long long top = (unsigned long long)p.I0 << p.N;   // the largest exponential
  const bool narrow = c.zero_from <= (1ull << 31) && top * (unsigned long long)d < (1ull << 32) && c.osh >= 32 &&
                      (p.M <= 32 || top > (1ull << (p.M - 32)));
  const int64_t want = (rows + 7) / 8;
  const int grid = (int)(want < (int64_t)ctx->sm_count * 8 ? want : (int64_t)ctx->sm_count * 8);
  LaunchScope ls(ctx, KIND_SHIFTMAX, (double)rows * (double)d * 5.0);
  const int wpl = (int)(((d + 15) / 16 * 4 + 31) / 32);
  if (narrow) {
    if (wpl <= 2) launch_k(shiftmax_direct_kernel<2, true>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
    else if (wpl <= 5) launch_k(shiftmax_direct_kernel<5, true>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
    else launch_k(shiftmax_direct_kernel<0, true>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
  } else {
    if (wpl <= 2) launch_k(shiftmax_direct_kernel<2, false>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
    else if (wpl <= 5) launch_k(shiftmax_direct_kernel<5, false>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
    else launch_k(shiftmax_direct_kernel<0, false>, dim3(grid), dim3(256), 0, ctx->stream, in, ldin, c, out, ldout, rows, (int)d);
  }
  return ls.done();
}

// ------------------------------------------------------------------ ShiftGELU

// ShiftGELU over an int8 row depends on two numbers only: the element x and m = max(0, row maximum of x)
// (the scaled value 1.702 x ~ (1.1011)b x of Eq. (GELU) is monotone in x, so its row maximum is that of m).
// The 128 x 256 results are produced once per parameter set; the row kernel then only looks values up.
// Entry (m, x): sigmoid(1.702 S x) as e / (e + e1) with both exponentials taken relative to the scaled maximum
// (Eq. (sigmoid)): e = exp of (scaled x - scaled m), e1 = exp of (-scaled m); quotient by Eq. (IntDiv) with
// M = 45 and k_out bits; the product x * quotient is requantised by `post` and saturated.
__global__ void shiftgelu_table_kernel(ivit_exp_params p, int post_m, int post_s, int8_t* __restrict__ table) {
  pdl_trigger();
  pdl_wait();
  const int m = blockIdx.x;            // 0..127
  const int x = (int)threadIdx.x - 128;
  int out = 0;
  if (x <= m) {                        // pairs with x above the row maximum cannot occur
    auto scaled = [](int v) { return v + (v >> 1) + (v >> 3) + (v >> 4); };
    const int top = scaled(m);
    const unsigned e1 = shiftexp(-top, p.I0, p.N);
    const unsigned e = shiftexp(scaled(x) - top, p.I0, p.N);
    const unsigned long long den = (unsigned long long)e + e1;
    int quot = 0;
    if (den != 0) {
      const unsigned long long recip = (1ull << 45) / den;
      quot = (int)((recip * e) >> (46 - p.k_out));       // recip * e <= 2^45
    }
    out = sat8(rq(x * quot, post_m, post_s));
  }
  table[m * 256 + threadIdx.x] = (int8_t)out;
}

// WPL > 0: rows of up to 512 * WPL values, R rows per warp at a time, kept in registers between the maximum and
// the look-ups (shiftgelu_rows).  WPL == 0: any width; the row is read twice.
template <int WPL, int R>
__global__ void __launch_bounds__(256) shiftgelu_kernel(const int8_t* __restrict__ in, int64_t ldin,
                                                        const int8_t* __restrict__ table,
                                                        int8_t* __restrict__ out, int64_t ldout,
                                                        int64_t rows, int cols, int fixed_max) {
  pdl_trigger();
  pdl_wait();
  __shared__ __align__(256) unsigned tab[8][(WPL > 0 ? R : 1) * 64];  // 256-byte table rows, per warp
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  if (WPL > 0) {
    constexpr int W = WPL > 0 ? WPL : 1;
    for (int64_t r0 = warp * R; r0 < rows; r0 += nwarps * R) {
      const int nrows = (int)(rows - r0 < R ? rows - r0 : R);
      shiftgelu_rows<W, R, false>(in + r0 * ldin, ldin, nrows, cols, table, tab[wib], out + r0 * ldout, ldout, lane, fixed_max);
      __syncwarp();
    }
    return;
  }
  const int nvec = cols >> 4;  // 16-byte vectors per row
  const int iters = (nvec + 31) / 32;
  const unsigned char* t8 = reinterpret_cast<const unsigned char*>(tab[wib]);
  for (int64_t r = warp; r < rows; r += nwarps) {
    const int4* src = reinterpret_cast<const int4*>(in + r * ldin);
    int mx4 = (int)0x80808080;
    for (int i = 0; i < iters; ++i) {
      const int idx = lane + 32 * i;
      int4 v = make_int4((int)0x80808080, (int)0x80808080, (int)0x80808080, (int)0x80808080);
      if (idx < nvec) v = __ldg(src + idx);
      mx4 = (int)__vmaxs4(__vmaxs4((unsigned)v.x, (unsigned)v.y), __vmaxs4(__vmaxs4((unsigned)v.z, (unsigned)v.w), (unsigned)mx4));
    }
    int mx = max(max((int)(int8_t)mx4, (int)(int8_t)(mx4 >> 8)), max((int)(int8_t)(mx4 >> 16), (int)(int8_t)(mx4 >> 24)));
    mx = fixed_max >= 0 ? fixed_max : max(0, warp_max(mx));   // fixed_max: the static-maximum variant
    __syncwarp();
    const unsigned* trow = reinterpret_cast<const unsigned*>(table + mx * 256);
    tab[wib][lane] = __ldg(trow + lane);
    tab[wib][lane + 32] = __ldg(trow + lane + 32);
    __syncwarp();
    int4* dst = reinterpret_cast<int4*>(out + r * ldout);
    for (int i = 0; i < iters; ++i) {
      const int idx = lane + 32 * i;
      if (idx < nvec) {
        const int4 v = __ldg(src + idx);
        const int vin[4] = {v.x, v.y, v.z, v.w};
        int vout[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const unsigned u = (unsigned)vin[k] ^ 0x80808080u;  // x + 128 per byte
          unsigned pk = t8[u & 0xff];
          pk |= (unsigned)t8[(u >> 8) & 0xff] << 8;
          pk |= (unsigned)t8[(u >> 16) & 0xff] << 16;
          pk |= (unsigned)t8[u >> 24] << 24;
          vout[k] = (int)pk;
        }
        dst[idx] = make_int4(vout[0], vout[1], vout[2], vout[3]);
      }
    }
  }
}

// Finds or builds the lookup table of a parameter set; *table = its 128 x 256 bytes on the device.
static int gelu_table(ivit_ctx* ctx, ivit_exp_params p, ivit_scale post, const int8_t** table) {
  const GeluKey key{p.I0, p.N, p.M, p.k_out, post.mult, post.shift};
  int slot = -1;
  for (int i = 0; i < ctx->gelu_used; ++i)
    if (ctx->gelu_keys[i] == key) { slot = i; break; }
  if (slot < 0) {
    if (ctx->gelu_used < kGeluTableSlots) {
      slot = ctx->gelu_used++;
    } else {
      slot = ctx->gelu_next;
      ctx->gelu_next = (ctx->gelu_next + 1) % kGeluTableSlots;
    }
    ctx->gelu_keys[slot] = key;
    ++ctx->gelu_gen;
    LaunchScope lt(ctx, KIND_GELU_TABLE, (double)kGeluTableBytes);
    launch_k(shiftgelu_table_kernel, dim3(128), dim3(256), 0, ctx->stream, p, post.mult, post.shift,
                                                          ctx->gelu_tables + (size_t)slot * kGeluTableBytes);
    int rc = lt.done();
    if (rc) return rc;
  }
  *table = ctx->gelu_tables + (size_t)slot * kGeluTableBytes;
  return IVIT_OK;
}

int gelu_table_for(ivit_ctx* ctx, ivit_exp_params p, ivit_scale post, const int8_t** table) {
  return gelu_table(ctx, p, post, table);
}

int gelu_static_row(ivit_ctx* ctx, ivit_exp_params p, ivit_scale post, const int8_t** row) {
  const int8_t* table = nullptr;
  const int rc = gelu_table(ctx, p, post, &table);
  if (rc) return rc;
  *row = table + 127 * 256;   // I_max = I_p(127)
  return IVIT_OK;
}

static int shiftgelu_rows(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p, ivit_scale post,
                          int8_t* out, int64_t ldout, int64_t rows, int64_t cols, int fixed_max) {
  if (rows == 0) return IVIT_OK;
  const int8_t* table = nullptr;
  int rc = gelu_table(ctx, p, post, &table);
  if (rc) return rc;
  const int wpl = (int)((cols / 16 + 31) / 32);
  const int rpw = wpl <= 1 ? 4 : (wpl == 2 || wpl == 4 ? 2 : 1);            // rows a warp takes at a time
  const int64_t want = ((rows + rpw - 1) / rpw + 7) / 8;
  const int grid = (int)(want < (int64_t)ctx->sm_count * 12 ? want : (int64_t)ctx->sm_count * 12);
  cudaStream_t st = ctx->stream;
  LaunchScope ls(ctx, KIND_SHIFTGELU, 2.0 * (double)rows * (double)cols);
  if (wpl <= 1) launch_k(shiftgelu_kernel<1, 4>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else if (wpl <= 2) launch_k(shiftgelu_kernel<2, 2>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else if (wpl <= 3) launch_k(shiftgelu_kernel<3, 1>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else if (wpl <= 4) launch_k(shiftgelu_kernel<4, 2>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else if (wpl <= 6) launch_k(shiftgelu_kernel<6, 1>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else if (wpl <= 8) launch_k(shiftgelu_kernel<8, 1>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  else launch_k(shiftgelu_kernel<0, 1>, dim3(grid), dim3(256), 0, st, in, ldin, table, out, ldout, rows, (int)cols, fixed_max);
  return ls.done();
}

int launch_shiftgelu(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p, ivit_scale post,
                     int8_t* out, int64_t ldout, int64_t rows, int64_t cols) {
  return shiftgelu_rows(ctx, in, ldin, p, post, out, ldout, rows, cols, -1);
}

int launch_shiftgelu_static(ivit_ctx* ctx, const int8_t* in, int64_t ldin, ivit_exp_params p, ivit_scale post,
                            int8_t* out, int64_t ldout, int64_t rows, int64_t cols) {
  return shiftgelu_rows(ctx, in, ldin, p, post, out, ldout, rows, cols, 127);
}

}  // namespace ivit

// ---- verification aid: the square-root routine of the I-LayerNorm kernels over a range of radicands ----
namespace ivit {
__global__ void isqrt_range_kernel(unsigned n0, unsigned count, uint16_t* __restrict__ out) {
  for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x)
    out[i] = (uint16_t)isqrt_bits26(n0 + i);
}
}  // namespace ivit

extern "C" int ivit_isqrt_range(ivit_ctx* ctx, uint32_t n0, uint32_t count, uint16_t* out) {
  if (!ctx || !out) return IVIT_ERR_INVALID_ARG;
  if ((uint64_t)n0 + count > (1ull << 26)) return IVIT_ERR_RANGE;
  if (count == 0) return IVIT_OK;
  ivit::isqrt_range_kernel<<<ctx->sm_count * 8, 256, 0, ctx->stream>>>(n0, count, out);
  ctx->launches += 1;
  return cudaGetLastError() == cudaSuccess ? IVIT_OK : IVIT_ERR_CUDA;
}
