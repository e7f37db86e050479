// Row operators shared by the stand-alone row kernels and by the Dense kernel, whose warps run them on rows the
// kernel has just finished: I-LayerNorm (Sec. 3.5) and ShiftGELU (Algorithm 2, through its look-up table).
// One warp works on a few rows at a time; per-channel constants are prepared once per CTA in shared memory.
#pragma once

#include "common.cuh"

namespace ivit {

// Integer square root, floor(sqrt(n)) for n < 2^26, one result bit per step (no division): the value the
// guarded iteration of Eq. (iterative) converges to.  Equality with the oracle's iteration is checked
// exhaustively over the whole range by a test (ivit_isqrt_range).
__device__ __forceinline__ unsigned isqrt_bits26(unsigned n) {
  unsigned res = 0;
#pragma unroll
  for (int k = 12; k >= 0; --k) {
    const unsigned bit = 1u << (2 * k);
    const unsigned t = res + bit;
    const bool ge = n >= t;
    n = ge ? n - t : n;
    res = (res >> 1) + (ge ? bit : 0u);
  }
  return res;
}

// ---- I-LayerNorm ------------------------------------------------------------------------------------------
// out[c] = sat8( rq((x[c] - mu) * F; m_c, s_c) + beta_c ),  mu = mean rounded half up,
// F = floor(2^M_ln / isqrt(sum (x - mu)^2)).

// Per-channel constants in shared memory, one int4 per word of four channels in each of three arrays.
// fast: every channel has s >= 33 and a small beta; then the arrays hold (m, s - 32, 2^(s-33) + beta 2^(s-32)) and
//   v = (hi32(yF m) + add) >> sh   [the rounding constant 2^(s-1) is a multiple of 2^32 and beta joins it];
// otherwise they hold (m, s, beta) and the requantisation is evaluated in 64 bits.
struct LnConsts {
  const int4* m;
  const int4* s;
  const int4* b;
  bool fast;
};

// Writes the raw constants of words tid, tid + nthreads, ... and returns whether all of them allow the fast form.
__device__ __forceinline__ bool ln_stage_consts(const ScaleDev& gs, const int32_t* beta, int nwords, int vec, int4* sm_m,
                                                int4* sm_s, int4* sm_b, int tid, int nthreads) {
  bool fast = true;
  for (int idx = tid; idx < nwords; idx += nthreads) {
    int m[4], s[4], b[4];
    if (vec) {
      const int4 m4 = __ldg(reinterpret_cast<const int4*>(gs.mult_c) + idx);
      const uchar4 s4 = __ldg(reinterpret_cast<const uchar4*>(gs.shift_c) + idx);
      int4 b4 = make_int4(0, 0, 0, 0);
      if (beta) b4 = __ldg(reinterpret_cast<const int4*>(beta) + idx);
      m[0] = m4.x; m[1] = m4.y; m[2] = m4.z; m[3] = m4.w;
      s[0] = s4.x; s[1] = s4.y; s[2] = s4.z; s[3] = s4.w;
      b[0] = b4.x; b[1] = b4.y; b[2] = b4.z; b[3] = b4.w;
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        m[k] = gs.mult_c ? __ldg(gs.mult_c + idx * 4 + k) : gs.mult;
        s[k] = gs.shift_c ? (int)__ldg(gs.shift_c + idx * 4 + k) : gs.shift;
        b[k] = beta ? __ldg(beta + idx * 4 + k) : 0;
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      s[k] = clamp_shift(s[k]);
      const int sh = s[k] - 32;
      fast = fast && sh >= 1 && b[k] > -(1 << (29 - sh)) && b[k] < (1 << (29 - sh));
    }
    sm_m[idx] = make_int4(m[0], m[1], m[2], m[3]);
    sm_s[idx] = make_int4(s[0], s[1], s[2], s[3]);
    sm_b[idx] = make_int4(b[0], b[1], b[2], b[3]);
  }
  return fast;
}

// Turns this thread's own words into the fast form (after every thread agreed that it is exact).
__device__ __forceinline__ void ln_fold_consts(int nwords, int4* sm_s, int4* sm_b, int tid, int nthreads) {
  for (int idx = tid; idx < nwords; idx += nthreads) {
    int4 s = sm_s[idx], b = sm_b[idx];
    s.x -= 32; s.y -= 32; s.z -= 32; s.w -= 32;
    b.x = (1 << (s.x - 1)) + b.x * (1 << s.x);
    b.y = (1 << (s.y - 1)) + b.y * (1 << s.y);
    b.z = (1 << (s.z - 1)) + b.z * (1 << s.z);
    b.w = (1 << (s.w - 1)) + b.w * (1 << s.w);
    sm_s[idx] = s;
    sm_b[idx] = b;
  }
}

// One warp, R rows of C int8 channels (C % 4 == 0, C <= 128 * WPL <= 1024): rows in[0 .. nrows) with stride ldin
// (rows past nrows are not touched), results to out with stride ldout.  The row sums are reduced together and the
// per-row scalars (mean, sum of squared deviations, square root, reciprocal) are computed by R lanes in parallel.
// CG: read the rows with L2 loads (rows written by other CTAs of the running kernel).
template <int WPL, int R, bool CG>
__device__ __forceinline__ void layernorm_rows(const int8_t* in, int64_t ldin, int nrows, int C, int M_ln, unsigned mean_magic,
                                               const LnConsts& k, int8_t* out, int64_t ldout, int lane) {
  const int nwords = C >> 2;
  int w[R][WPL];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int* src = reinterpret_cast<const int*>(in + (int64_t)r * ldin);
#pragma unroll
    for (int i = 0; i < WPL; ++i) {
      const int idx = lane + 32 * i;
      w[r][i] = 0;
      if (r < nrows && idx < nwords) w[r][i] = CG ? __ldcg(src + idx) : __ldg(src + idx);
    }
  }
  int my_s1 = 0, my_s2 = 0;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    int s1 = 0, s2 = 0;
#pragma unroll
    for (int i = 0; i < WPL; ++i) {
      s1 = __dp4a(w[r][i], 0x01010101, s1);
      s2 = __dp4a(w[r][i], w[r][i], s2);
    }
    s1 = __reduce_add_sync(0xffffffffu, s1);
    s2 = __reduce_add_sync(0xffffffffu, s2);
    if (lane == r) { my_s1 = s1; my_s2 = s2; }
  }
  // lane r < R holds the sums of row r.  Mean, rounded half up: floor((2 S1 + C) / 2C), taken as a multiplication
  // by mean_magic = floor(2^32 / 2C) + 1 on the numerator shifted by 256 C to make it positive (exact: numerators
  // stay below 2^19 for C <= 1024).  Sum of squared deviations = sum x^2 - 2 mu sum x + C mu^2 < 2^26.
  const int mu = (int)__umulhi((unsigned)(2 * my_s1 + 257 * C), mean_magic) - 128;
  const unsigned V = (unsigned)(my_s2 - 2 * mu * my_s1 + C * mu * mu);
  const unsigned sd = isqrt_bits26(V);
  const int F = sd == 0 ? 0 : (int)((1u << M_ln) / sd);
  const int muF = (int)((unsigned)mu * (unsigned)F);
  int Fr[R], muFr[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    Fr[r] = __shfl_sync(0xffffffffu, F, r);
    muFr[r] = __shfl_sync(0xffffffffu, muF, r);
  }
#pragma unroll
  for (int i = 0; i < WPL; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nwords) {
      const int4 m4 = k.m[idx], s4 = k.s[idx], b4 = k.b[idx];
      const int cm[4] = {m4.x, m4.y, m4.z, m4.w}, cs[4] = {s4.x, s4.y, s4.z, s4.w}, cb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (r < nrows) {
          int v[4];
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            int x;   // byte b, sign-extended
            asm("prmt.b32 %0, %1, %1, %2;" : "=r"(x) : "r"(w[r][i]), "r"(0x8880 + 0x1111 * b));
            // (x - mu) * F modulo 2^32: the difference fits, |y F| <= 2^(M_ln + 1)
            const int yF = (int)((unsigned)x * (unsigned)Fr[r] - (unsigned)muFr[r]);
            if (k.fast) {
              int h;
              asm("mad.hi.s32 %0, %1, %2, %3;" : "=r"(h) : "r"(yF), "r"(cm[b]), "r"(cb[b]));
              v[b] = h >> cs[b];
            } else {
              v[b] = rq(yF, cm[b], cs[b]) + cb[b];
            }
          }
          unsigned t, d;
          asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(v[3]), "r"(v[2]), "r"(0));
          asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(v[1]), "r"(v[0]), "r"(t));
          reinterpret_cast<int*>(out + (int64_t)r * ldout)[idx] = (int)d;
        }
      }
    }
  }
}

// ---- ShiftGELU --------------------------------------------------------------------------------------------
// One warp, R rows of `cols` int8 values (cols % 16 == 0, cols <= 512 * WPL): row maximum, then one look-up per
// value in row max(0, maximum) of the 128 x 256 table; `tab` is the warp's staging space for the R table rows
// (R x 64 words of shared memory, 256-byte aligned).  in == out is allowed.
template <int WPL, int R, bool CG>
__device__ __forceinline__ void shiftgelu_rows(const int8_t* in, int64_t ldin, int nrows, int cols, const int8_t* table,
                                               unsigned* tab, int8_t* out, int64_t ldout, int lane, int fixed_max = -1) {
  const int nvec = cols >> 4;
  int4 w[R][WPL];
  int mx[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int4* src = reinterpret_cast<const int4*>(in + (int64_t)r * ldin);
    int m4 = (int)0x80808080;
#pragma unroll
    for (int i = 0; i < WPL; ++i) {
      const int idx = lane + 32 * i;
      int4 v = make_int4((int)0x80808080, (int)0x80808080, (int)0x80808080, (int)0x80808080);
      if (r < nrows && idx < nvec) v = CG ? __ldcg(src + idx) : __ldg(src + idx);
      w[r][i] = v;
      m4 = (int)__vmaxs4(__vmaxs4((unsigned)v.x, (unsigned)v.y), __vmaxs4(__vmaxs4((unsigned)v.z, (unsigned)v.w), (unsigned)m4));
    }
    mx[r] = max(max((int)(int8_t)m4, (int)(int8_t)(m4 >> 8)), max((int)(int8_t)(m4 >> 16), (int)(int8_t)(m4 >> 24)));
  }
  __syncwarp();
#pragma unroll
  for (int r = 0; r < R; ++r) {
    mx[r] = fixed_max >= 0 ? fixed_max : max(0, __reduce_max_sync(0xffffffffu, mx[r]));   // fixed_max: the static-maximum variant
    const unsigned* trow = reinterpret_cast<const unsigned*>(table + mx[r] * 256);
    tab[64 * r + lane] = __ldg(trow + lane);
    tab[64 * r + lane + 32] = __ldg(trow + lane + 32);
  }
  __syncwarp();
#pragma unroll
  for (int r = 0; r < R; ++r) {
    if (r < nrows) {
      // shared-memory address of entry 0 of this row's table: 256-byte aligned, so that one byte permute puts
      // the index x + 128 into its low byte
      const uint32_t t8 = (uint32_t)__cvta_generic_to_shared(tab + 64 * r);
      int4* dst = reinterpret_cast<int4*>(out + (int64_t)r * ldout);
#pragma unroll
      for (int i = 0; i < WPL; ++i) {
        const int idx = lane + 32 * i;
        if (idx < nvec) {
          const int vin[4] = {w[r][i].x, w[r][i].y, w[r][i].z, w[r][i].w};
          int vout[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const unsigned u = (unsigned)vin[q] ^ 0x80808080u;   // x + 128 per byte
            unsigned e[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
              const unsigned a = __byte_perm(u, t8, 0x7650 + b);
              asm volatile("ld.shared.u8 %0, [%1];" : "=r"(e[b]) : "r"(a));
            }
            vout[q] = (int)__byte_perm(__byte_perm(e[0], e[1], 0x0040), __byte_perm(e[2], e[3], 0x0040), 0x5410);
          }
          dst[idx] = make_int4(vout[0], vout[1], vout[2], vout[3]);
        }
      }
    }
  }
}

}  // namespace ivit
