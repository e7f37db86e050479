// Data-movement helpers around the encoder (patch extraction, row gathers, class-token rows,
// token pooling).  Pure permutations / sums; none of them is described in the paper.
#include "common.cuh"

namespace ivit {

// One thread per 4 output bytes (px .. px+3 of one patch row); P % 4 == 0.
__global__ void patchify_kernel(const int8_t* __restrict__ img, int64_t B, int C, int Hi, int Wi, int P,
                                int window, int8_t* __restrict__ out, int64_t ldout, int64_t total_words) {
  pdl_trigger();
  pdl_wait();
  const int gh = Hi / P, gw = Wi / P;
  const int kw = C * P * P / 4;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total_words;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int w = (int)(t % kw);
    const int64_t prow = t / kw;  // raster patch index over the batch
    const int gx = (int)(prow % gw), gy = (int)((prow / gw) % gh);
    const int64_t b = prow / ((int64_t)gw * gh);
    const int px = (w * 4) % P, py = ((w * 4) / P) % P, c = (w * 4) / (P * P);
    const int v = __ldg(reinterpret_cast<const int*>(img + ((b * C + c) * Hi + gy * P + py) * (int64_t)Wi + gx * P + px));
    int64_t row;
    if (window > 0) {
      const int wy = gy / window, wx = gx / window, iy = gy % window, ix = gx % window;
      row = (int64_t)(wy * (gw / window) + wx) * window * window + iy * window + ix;
    } else {
      row = (int64_t)gy * gw + gx;
    }
    *reinterpret_cast<int*>(out + (b * gh * gw + row) * ldout + w * 4) = v;
  }
}

// P % 16 == 0, aligned image rows: one thread moves 16 bytes (px .. px+15 of one patch row) with 32-bit index
// arithmetic; `segs` = P / 16 such pieces per patch row.
__global__ void patchify_vec_kernel(const int8_t* __restrict__ img, int C, int Hi, int Wi, int P, int window,
                                    int8_t* __restrict__ out, int64_t ldout, unsigned total_vecs) {
  pdl_trigger();
  pdl_wait();
  const unsigned gh = Hi / P, gw = Wi / P, segs = P / 16;
  const unsigned per_row = (unsigned)Wi / 16;          // 16-byte pieces per image row
  for (unsigned t = blockIdx.x * blockDim.x + threadIdx.x; t < total_vecs; t += gridDim.x * blockDim.x) {
    // t enumerates the image in memory order: consecutive threads read consecutive 16-byte pieces
    const unsigned xv = t % per_row, line = t / per_row;          // line = (b * C + c) * Hi + y
    const unsigned y = line % (unsigned)Hi, bc = line / (unsigned)Hi;
    const unsigned c = bc % (unsigned)C, b = bc / (unsigned)C;
    const unsigned gx = xv / segs, sx = xv % segs, gy = y / (unsigned)P, py = y % (unsigned)P;
    const int4 v = __ldg(reinterpret_cast<const int4*>(img) + t);
    unsigned row;
    if (window > 0) {
      const unsigned wy = gy / window, wx = gx / window, iy = gy % window, ix = gx % window;
      row = (wy * (gw / window) + wx) * window * window + iy * window + ix;
    } else {
      row = gy * gw + gx;
    }
    *reinterpret_cast<int4*>(out + ((int64_t)b * gh * gw + row) * ldout + (c * P + py) * P + sx * 16) = v;
  }
}

__global__ void gather_rows_kernel(const int8_t* __restrict__ src, int64_t ldsrc, const int32_t* __restrict__ index,
                                   int64_t n_rows, int vec_per_row, int8_t* __restrict__ dst, int64_t lddst) {
  pdl_trigger();
  pdl_wait();
  const int64_t total = n_rows * vec_per_row;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = t / vec_per_row;
    const int v = (int)(t % vec_per_row);
    const int4 x = __ldg(reinterpret_cast<const int4*>(src + (int64_t)__ldg(index + r) * ldsrc) + v);
    reinterpret_cast<int4*>(dst + r * lddst)[v] = x;
  }
}

__global__ void fill_rows_kernel(const int8_t* __restrict__ src_row, int vec_per_row, int8_t* __restrict__ dst,
                                 int64_t group_stride, int64_t groups) {
  pdl_trigger();
  pdl_wait();
  const int64_t total = groups * vec_per_row;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t g = t / vec_per_row;
    const int v = (int)(t % vec_per_row);
    reinterpret_cast<int4*>(dst + g * group_stride)[v] = __ldg(reinterpret_cast<const int4*>(src_row) + v);
  }
}

__global__ void token_mean_kernel(const int8_t* __restrict__ in, int64_t ldin, int64_t groups, int T, int C,
                                  ScaleDev scale, int8_t* __restrict__ out, int64_t ldout) {
  pdl_trigger();
  pdl_wait();
  const int64_t total = groups * C;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t g = t / C;
    const int c = (int)(t % C);
    int s = 0;
    for (int k = 0; k < T; ++k) s += __ldg(in + (g * T + k) * ldin + c);
    out[g * ldout + c] = (int8_t)sat8(rq(s, scale.mult, clamp_shift(scale.shift)));
  }
}

static int grid_for(ivit_ctx* ctx, int64_t items, int threads) {
  int64_t want = (items + threads - 1) / threads;
  const int64_t cap = (int64_t)ctx->sm_count * 16;
  return (int)(want < cap ? (want < 1 ? 1 : want) : cap);
}

int launch_patchify(ivit_ctx* ctx, const int8_t* img, int64_t B, int64_t C, int64_t Hi, int64_t Wi,
                    int64_t P, int64_t window, int8_t* out, int64_t ldout) {
  const int64_t total = B * C * Hi * Wi / 4;
  if (total == 0) return IVIT_OK;
  LaunchScope ls(ctx, KIND_MOVE, 2.0 * (double)total * 4);
  if (P % 16 == 0 && Wi % 16 == 0 && ldout % 16 == 0 && total / 4 < 0x7fffffffLL && !(reinterpret_cast<uintptr_t>(img) & 15) &&
      !(reinterpret_cast<uintptr_t>(out) & 15)) {
    launch_k(patchify_vec_kernel, dim3(grid_for(ctx, total / 4, 256)), dim3(256), 0, ctx->stream, img, (int)C, (int)Hi, (int)Wi, (int)P,
             (int)window, out, ldout, (unsigned)(total / 4));
    return ls.done();
  }
  launch_k(patchify_kernel, dim3(grid_for(ctx, total, 256)), dim3(256), 0, ctx->stream, img, B, (int)C, (int)Hi, (int)Wi, (int)P,
                                                                       (int)window, out, ldout, total);
  return ls.done();
}

int launch_gather_rows(ivit_ctx* ctx, const int8_t* src, int64_t ldsrc, const int32_t* index,
                       int64_t n_rows, int64_t width, int8_t* dst, int64_t lddst) {
  if (n_rows == 0) return IVIT_OK;
  LaunchScope ls(ctx, KIND_MOVE, 2.0 * (double)n_rows * (double)width);
  launch_k(gather_rows_kernel, dim3(grid_for(ctx, n_rows * (width / 16), 256)), dim3(256), 0, ctx->stream, 
      src, ldsrc, index, n_rows, (int)(width / 16), dst, lddst);
  return ls.done();
}

int launch_fill_rows(ivit_ctx* ctx, const int8_t* src_row, int64_t width, int8_t* dst,
                     int64_t group_stride, int64_t groups) {
  if (groups == 0) return IVIT_OK;
  LaunchScope ls(ctx, KIND_MOVE, (double)groups * (double)width);
  launch_k(fill_rows_kernel, dim3(grid_for(ctx, groups * (width / 16), 256)), dim3(256), 0, ctx->stream, 
      src_row, (int)(width / 16), dst, group_stride, groups);
  return ls.done();
}

int launch_token_mean(ivit_ctx* ctx, const int8_t* in, int64_t ldin, int64_t groups, int64_t T,
                      int64_t C, ScaleDev scale, int8_t* out, int64_t ldout) {
  if (groups == 0) return IVIT_OK;
  LaunchScope ls(ctx, KIND_MOVE, (double)groups * (double)C * (double)(T + 1));
  launch_k(token_mean_kernel, dim3(grid_for(ctx, groups * C, 256)), dim3(256), 0, ctx->stream, in, ldin, groups, (int)T, (int)C,
                                                                             scale, out, ldout);
  return ls.done();
}

}  // namespace ivit
