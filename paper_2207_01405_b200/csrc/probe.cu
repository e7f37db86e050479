// Measurement aid (not part of the paper's method): the rate at which this GPU's tensor cores retire
// tcgen05.mma.kind::i8 instructions when nothing else is in the way - operands fixed in shared memory, no loads,
// no epilogue.  It is the ceiling the Dense kernel's TOP/s are quoted against.
#include "tc_ptx.cuh"

namespace ivit {
namespace {

constexpr int kProbeN = 256;   // columns of one accumulator (UMMA N)

// One CTA per SM; one thread issues `iters` groups of four M128 x N256 x K32 MMAs (one 128-byte k-block of both
// operands), alternating between two accumulators in tensor memory, then waits (bounded) for the last of them.
__global__ void __launch_bounds__(128, 1) int8_mma_probe_kernel(int iters, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sa = base, sb = base + 128 * 128, bar = sb + kProbeN * 128;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + 128 * 128 + kProbeN * 128 + 16);
  for (int i = threadIdx.x; i < (128 + kProbeN) * 128 / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(gen)[i] = 0x01010101u * (uint32_t)(i & 3);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  fence_async_smem();
  if (threadIdx.x < 32) tmem_alloc(smem_u32(tmem_slot), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (threadIdx.x == 0) {
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kProbeN >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t hi = desc_hi(1024, 2);
    for (int it = 0; it < iters; ++it) {
      const uint32_t d = tmem + (uint32_t)((it & 1) * kProbeN);
      uint32_t a_lo = desc_lo(sa, 16), b_lo = desc_lo(sb, 16);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        umma_i8_lohi(d, a_lo, hi, b_lo, hi, idesc, (it > 1 || k > 0) ? 1u : 0u);
        a_lo += 2;
        b_lo += 2;
      }
    }
    umma_commit(bar);
    mbar_wait(bar, 0, status);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    tmem_dealloc(tmem, 512u);
  }
}

}  // namespace
}  // namespace ivit

extern "C" int ivit_probe_int8_mma(ivit_ctx* ctx, int32_t iters, float* ms, double* ops) {
  using namespace ivit;
  if (!ctx || !ms || !ops || iters < 1 || iters > (1 << 20)) return IVIT_ERR_INVALID_ARG;
  const size_t smem = 1024 + (128 + kProbeN) * 128 + 64;
  if (cudaFuncSetAttribute(int8_mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return IVIT_ERR_CUDA;
  cudaEvent_t a, b;
  if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return IVIT_ERR_CUDA;
  int rc = IVIT_OK;
  // one untimed launch, then the timed one
  for (int rep = 0; rep < 2 && rc == IVIT_OK; ++rep) {
    if (rep == 1) cudaEventRecord(a, ctx->stream);
    int8_mma_probe_kernel<<<ctx->sm_count, 128, smem, ctx->stream>>>(iters, ctx->status_dev);
    ctx->launches += 1;
    if (cudaGetLastError() != cudaSuccess) rc = IVIT_ERR_CUDA;
  }
  cudaEventRecord(b, ctx->stream);
  if (rc == IVIT_OK && cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = IVIT_ERR_CUDA;
  if (rc == IVIT_OK && cudaEventElapsedTime(ms, a, b) != cudaSuccess) rc = IVIT_ERR_CUDA;
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  *ops = 2.0 * 128.0 * kProbeN * 32.0 * 4.0 * (double)iters * (double)ctx->sm_count;
  return rc;
}
