// CUDA-core (dp4a) INT8 GEMM with the dyadic requantisation epilogue of Sec. 3.2.
// Handles every shape the library accepts (any K, ragged M / N, both operand orders of B,
// two-level batch strides); the tcgen05 kernel takes over where the shape qualifies.
#include "common.cuh"

namespace ivit {

constexpr int TM = 64, TN = 64, TKW = 8;  // tile: 64 x 64 outputs, 8 words (32 int8) of K per step

__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmProblem g, int64_t tiles_m, int64_t tiles_n) {
  pdl_trigger();
  pdl_wait();
  __shared__ int As[TM][TKW + 1];
  __shared__ int Bs[TN][TKW + 1];
  const int tid = threadIdx.x;
  const int64_t tile = blockIdx.x;
  const int64_t batch = tile / (tiles_m * tiles_n);
  const int64_t t2 = tile % (tiles_m * tiles_n);
  const int64_t m0 = (t2 / tiles_n) * TM, n0 = (t2 % tiles_n) * TN;
  const int64_t bo = batch / g.batches_inner, bi = batch % g.batches_inner;
  const int8_t* A = g.A + bo * g.sAo + bi * g.sAi;
  const int8_t* B = g.B + bo * g.sBo + bi * g.sBi;
  const int ty = tid >> 4, tx = tid & 15;
  int acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0;

  const int64_t K = g.K;
  for (int64_t k0 = 0; k0 < K; k0 += TKW * 4) {
    // A tile: 64 rows x 8 words; 512 words, 2 per thread
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int e = tid + i * 256, row = e >> 3, kw = e & 7;
      const int64_t r = m0 + row, k = k0 + kw * 4;
      int v = 0;
      if (r < g.M && k < K) {
        v = __ldg(reinterpret_cast<const int*>(A + r * g.lda + k));
        if (k + 4 > K) v &= (int)(0xffffffffu >> (8 * (k + 4 - K)));
      }
      As[row][kw] = v;
    }
    if (g.transB) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int e = tid + i * 256, row = e >> 3, kw = e & 7;
        const int64_t n = n0 + row, k = k0 + kw * 4;
        int v = 0;
        if (n < g.N && k < K) {
          v = __ldg(reinterpret_cast<const int*>(B + n * g.ldb + k));
          if (k + 4 > K) v &= (int)(0xffffffffu >> (8 * (k + 4 - K)));
        }
        Bs[row][kw] = v;
      }
    } else {
      // B is [K, N]: read words along n, scatter bytes so that Bs[n] holds 4 consecutive k per word
      int8_t* Bb = reinterpret_cast<int8_t*>(&Bs[0][0]);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int e = tid + i * 256, kk = e >> 4, nw = e & 15;  // 32 k rows x 16 words of n
        const int64_t k = k0 + kk, n = n0 + nw * 4;
        int v = 0;
        if (k < K && n < g.N) v = __ldg(reinterpret_cast<const int*>(B + k * g.ldb + n));
#pragma unroll
        for (int b = 0; b < 4; ++b) Bb[(nw * 4 + b) * (TKW + 1) * 4 + kk] = (int8_t)(v >> (8 * b));
      }
    }
    __syncthreads();
#pragma unroll
    for (int kw = 0; kw < TKW; ++kw) {
      int a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[ty * 4 + i][kw];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[tx * 4 + j][kw];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  const GemmEpilogue& e = g.epi;
  const int64_t out_off = bo * g.sCo + bi * g.sCi;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = m0 + ty * 4 + i;
    if (r >= g.M) continue;
    const int64_t ro = e.group_rows > 0 ? (r / e.group_rows) * e.group_stride + (r % e.group_rows) : r;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t c = n0 + tx * 4 + j;
      if (c >= g.N) continue;
      int a = acc[i][j];
      if (e.bias) a += __ldg(e.bias + c);
      if (e.bias32) a += __ldg(e.bias32 + ((batch % e.bias_batches) * g.M + r) * e.ldbias + c);
      int v = rq(a, e.scale.m((int)c), e.scale.s((int)c));
      if (e.res) v += rq((int)__ldg(e.res + (r % e.res_rows) * e.ldres + c), e.res_scale.m(0), e.res_scale.s(0));
      if (e.out_dtype == IVIT_I8)
        reinterpret_cast<int8_t*>(e.out)[out_off + ro * e.ldo + c] =
            e.act_table ? __ldg(e.act_table + sat8(v) + 128) : (int8_t)sat8(v);
      else
        reinterpret_cast<int32_t*>(e.out)[out_off + ro * e.ldo + c] = v;
    }
  }
}

int launch_gemm_simt(ivit_ctx* ctx, const GemmProblem& g) {
  const int64_t batches = g.batches_outer * g.batches_inner;
  if (batches == 0 || g.M == 0 || g.N == 0) return IVIT_OK;
  const int64_t tiles_m = (g.M + TM - 1) / TM, tiles_n = (g.N + TN - 1) / TN;
  const int64_t total = batches * tiles_m * tiles_n;
  if (total > 2147483647LL) return IVIT_ERR_UNSUPPORTED;
  LaunchScope ls(ctx, KIND_GEMM_SIMT, 2.0 * (double)batches * (double)g.M * (double)g.N * (double)g.K);
  launch_k(gemm_simt_kernel, dim3((unsigned)total), dim3(256), 0, ctx->stream, g, tiles_m, tiles_n);
  return ls.done();
}

}  // namespace ivit
