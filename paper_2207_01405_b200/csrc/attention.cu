// Fused attention core of one encoder block (Sec. 3.1 MSA equation, Sec. 3.2 and Algorithm 1):
//   S = Q_i K_i^T (+ bias)  ->  requantise to int8  ->  Shiftmax  ->  P_i V_i  ->  requantise
// for one (image or window, head, 128-row tile) per CTA, rows up to 256 tokens long.
//
// The int32 score tile lives in tensor memory, never in HBM.  Two threads share one score row (one
// TMEM lane; they take alternate 32-column chunks), so the row maximum and the row sum of
// Algorithm 1 need one exchange of two words through shared memory each: no shuffles.
//   pass A  tcgen05.ld the row, requantise to int8 (kept packed in registers), running max;
//   pass B  ShiftExp by table lookup (256 entries, I_max - I in [0, 255]), row sum, and the
//           exponentials written back over the scores in tensor memory (tcgen05.st);
//   pass C  one reciprocal per row (Eq. (IntDiv)), then exp * reciprocal >> shift per value; the
//           int8 probabilities are written to shared memory in the K-major 128B-swizzled layout
//           that the second MMA consumes as its A operand.
// V is consumed as stored ([token, d] rows, MN-major B operand).  Every wait is bounded.
#include "tc_ptx.cuh"
#include <cstdlib>

namespace ivit {

namespace {

constexpr int kAttnThreads = 288;   // warp 0: TMA + MMA issue + TMEM owner; warps 1..8: two threads per score row
constexpr int UK = 32;              // K of one tcgen05.mma.kind::i8


// Eq. (IntDiv) with M = 45 for four exponentials: (floor(2^45 / sum) * e) >> (45 - (k_out - 1)) = umulhi(factor, e) >> (14 - k_out),
// clamped to 2^(k_out-1) - 1 and packed.  K8: k_out = 8, where the saturating pack does the clamp (values are <= 128).
template <bool K8>
__device__ __forceinline__ uint32_t prob_word(unsigned factor, int e0, int e1, int e2, int e3, int osh, int omax) {
  if (K8)
    return pack_sat8((int)(__umulhi(factor, (unsigned)e0) >> 6), (int)(__umulhi(factor, (unsigned)e1) >> 6),
                     (int)(__umulhi(factor, (unsigned)e2) >> 6), (int)(__umulhi(factor, (unsigned)e3) >> 6));
  return pack_sat8(min((int)(__umulhi(factor, (unsigned)e0) >> osh), omax), min((int)(__umulhi(factor, (unsigned)e1) >> osh), omax),
                   min((int)(__umulhi(factor, (unsigned)e2) >> osh), omax), min((int)(__umulhi(factor, (unsigned)e3) >> osh), omax));
}

struct AttnArgs {
  int T, d, heads, Npad;            // Npad = T rounded up to 32 (score columns and P.V contraction length)
  int64_t D;                        // heads * d
  int tiles_m;                      // ceil(T / 128)
  int bh;                           // images (or windows) x heads
  int items;                        // bh * tiles_m
  int G, R;                         // G windows of at most R = 128 / G tokens share one tile (G = 1: one image or window per tile)
  int Btot;                         // images or windows in the tensor
  int tmem_cols;
  int qk_m, qk_s, pv_m, pv_s;
  ivit_exp_params smax;
  const int32_t* bias;              // [bias_batches, T, T] or nullptr
  int64_t bias_batches;
  int8_t* O;                        // [B*T, D]
  int q_pos[3], k_pos[3], v_pos[3];
  unsigned* sched;                  // this launch's counters: [0] next work item, [1] CTAs that have finished
  unsigned* sched_other;            // the counters of the next launch
  int* status;
};

constexpr uint32_t kItemWaitRounds = 16;   // the item barrier outlasts every bounded wait of the control thread

// Persistent CTAs (two per SM) draw work items = (image or window, head, 128-row tile) from a counter, the
// full 128-row tiles first.  One control thread issues the TMA loads and the MMAs; the loads of the next item
// are issued as soon as the MMAs that read the shared-memory operands of the current one have completed, so
// they overlap the Shiftmax passes.  Barriers are used once per item: the parity of a wait is the item count.
// kPack: several windows share the tile (AttnArgs::G > 1); the plain form carries none of that index arithmetic.
template <bool kPack, bool K8>
__global__ void __launch_bounds__(kAttnThreads, 2) attention_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                 const __grid_constant__ CUtensorMap tmK,
                                                                 const __grid_constant__ CUtensorMap tmV, AttnArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // [Q 128x128B][K Npad x 128B][V Npad x d][P 128 x 128B x kblocks][exp table][row partials][item ring][barriers]
  const uint32_t q_off = 0, k_off = 128 * 128, v_off = k_off + a.Npad * 128;
  const uint32_t p_off = (v_off + a.Npad * a.d + 1023u) & ~1023u;
  const int p_kblocks = (a.Npad + 127) / 128;
  const uint32_t tab_off = p_off + p_kblocks * 128 * 128;
  const uint32_t part_off = tab_off + 1024;            // [2 halves][128 rows] partial max, then partial sum
  const uint32_t item_off = part_off + 2 * 128 * 4 * 2;   // [2] work item of even / odd iterations (-1: no more work)
  const uint32_t bar_off = item_off + 16;
  unsigned* tab = reinterpret_cast<unsigned*>(gen + tab_off);
  volatile int* item_ring = reinterpret_cast<volatile int*>(gen + item_off);
  // Q and K landed | V landed | scores ready | probabilities written | output ready | output read | item published
  const uint32_t bar_qk = base + bar_off, bar_v = bar_qk + 8, bar_s = bar_qk + 16, bar_p = bar_qk + 24,
                 bar_o = bar_qk + 32, bar_e = bar_qk + 40, bar_item = bar_qk + 48;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + bar_off + 64);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(bar_qk, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 8);
    mbar_init(bar_o, 1);
    mbar_init(bar_e, 8);
    mbar_init(bar_item, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), (uint32_t)a.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_trigger();
  // The ShiftExp table depends on parameters only: the Shiftmax threads build it before they wait for the previous
  // kernel (whose QKV tensor the control thread loads and whose successors' buffers the output overwrites).
  if (warp == 0) pdl_wait();
  // Launches alternate between two pairs of counters.  A launch leaves its own pair at zero when its last CTA
  // finishes, and also zeroes the other pair (below, after the wait), so that a launch that was cut short cannot
  // poison the next.

  // item -> (tile, image/window * heads + head): all first tiles before all second tiles
  if (warp == 0) {
    if (lane == 0) {
      auto load_qk = [&](int item) {
        const int tile = item / a.bh, bhid = item - tile * a.bh;
        const int h = bhid % a.heads, b = bhid / a.heads;
        mbar_expect_tx(bar_qk, 128 * 128 + a.Npad * 128);
        int c[4];
        c[0] = 0; c[a.q_pos[0]] = tile * 128; c[a.q_pos[1]] = h; c[a.q_pos[2]] = kPack ? b * a.G : b;
        tma_load_4d(base + q_off, &tmQ, bar_qk, c[0], c[1], c[2], c[3]);
        c[0] = 0; c[a.k_pos[0]] = 0; c[a.k_pos[1]] = h; c[a.k_pos[2]] = kPack ? b * a.G : b;
        tma_load_4d(base + k_off, &tmK, bar_qk, c[0], c[1], c[2], c[3]);
      };
      auto load_v = [&](int item) {
        const int tile = item / a.bh, bhid = item - tile * a.bh;
        const int h = bhid % a.heads, b = bhid / a.heads;
        mbar_expect_tx(bar_v, a.Npad * a.d);
        int c[4];
        c[0] = 0; c[a.v_pos[0]] = 0; c[a.v_pos[1]] = h; c[a.v_pos[2]] = kPack ? b * a.G : b;
        tma_load_4d(base + v_off, &tmV, bar_v, c[0], c[1], c[2], c[3]);
      };
      auto draw = [&]() {
        const unsigned t = atomicAdd(a.sched, 1u);
        return t < (unsigned)a.items ? (int)t : -1;
      };
      auto publish = [&](uint32_t n, int item) {
        item_ring[n & 1u] = item;
        mbar_arrive(bar_item);   // release: the item is visible to whoever sees this phase complete
      };
      // S = Q K^T: M = 128, N = Npad, both operands K-major rows of 128 bytes.  O = P V: V as stored (MN-major).
      const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.Npad >> 3) << 17) | (8u << 24);
      const uint32_t idesc2 = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(a.d >> 3) << 17) | (8u << 24);
      const uint32_t v_layout = a.d == 128 ? 2u : (a.d == 64 ? 4u : 6u);
      const int ks = (a.d + UK - 1) / UK, ks2 = a.Npad / UK;

      int item = draw();
      bool qk_flying = false, v_flying = false;   // loads issued and not yet waited for (their barrier phase = item count)
      if (item >= 0) { load_qk(item); load_v(item); qk_flying = v_flying = true; }
      bool ok = true;
      uint32_t n = 0, qk_par = 0, v_par = 0;
      for (; item >= 0; ++n) {
        const uint32_t par = n & 1u;
        publish(n, item);
        ok = mbar_wait(bar_qk, par, a.status);
        qk_flying = !ok;
        // the output of the previous item must have left tensor memory
        if (ok && n > 0) ok = mbar_wait(bar_e, par ^ 1u, a.status);
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < ks; ++k)
          umma_i8(tmem, smem_desc(base + q_off + k * UK, 16, 1024, 2), smem_desc(base + k_off + k * UK, 16, 1024, 2),
                  idesc, k != 0);
        umma_commit(bar_s);
        const int next = draw();
        // Q and K may be overwritten once the score MMAs have read them
        ok = mbar_wait(bar_s, par, a.status);
        if (!ok) break;
        if (next >= 0) { load_qk(next); qk_flying = true; qk_par = par ^ 1u; }
        // O = P V once the probabilities are in shared memory and V has landed
        ok = mbar_wait(bar_p, par, a.status);
        if (ok) { ok = mbar_wait(bar_v, par, a.status); v_flying = !ok; }
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < ks2; ++k) {
          const uint32_t pa = base + p_off + (k >> 2) * (128 * 128) + (k & 3) * UK;
          umma_i8(tmem, smem_desc(pa, 16, 1024, 2), smem_desc(base + v_off + k * UK * a.d, 16, 8 * a.d, v_layout),
                  idesc2, k != 0);
        }
        umma_commit(bar_o);
        // V may be overwritten once these MMAs have read it
        ok = mbar_wait(bar_o, par, a.status);
        if (!ok) break;
        if (next >= 0) { load_v(next); v_flying = true; v_par = par ^ 1u; }
        item = next;
      }
      // end of work (or a wait that timed out): tell the other warps; nothing may be in flight at exit
      publish(ok ? n : n + 1, -1);
      if (qk_flying) mbar_wait(bar_qk, qk_par, a.status);
      if (v_flying) mbar_wait(bar_v, v_par, a.status);
    }
  } else {
    // ---- softmax / epilogue threads: TMEM lane quarter = warp % 4; the two warps of a quarter
    //      take the even / odd 32-column chunks of the same 32 rows ----
    const int st = threadIdx.x - 32;   // 0..255
    tab[st] = shiftexp(-st, a.smax.I0, a.smax.N);
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 32) {
      a.sched_other[0] = 0;
      a.sched_other[1] = 0;
    }
    const int qd = warp & 3;
    const int half = (warp - 1) >> 2;
    const int trow = qd * 32 + lane;              // row inside the tile
    const uint32_t t_row = tmem + ((uint32_t)(qd * 32) << 16);
    const int nch = a.Npad / 16;
    const bool qk_hi = a.qk_s >= 33;              // rounding constant and shift both past the low product word
    const long long qk_c = 1ll << (a.qk_s - 1);
    const int qk_rnd = qk_hi ? 1 << (a.qk_s - 33) : 0, qk_sh = a.qk_s - 32;
    int* part_max = reinterpret_cast<int*>(gen + part_off);
    unsigned* part_sum = reinterpret_cast<unsigned*>(gen + part_off + 2 * 128 * 4);
    asm volatile("bar.sync 1, 256;" ::: "memory");   // the table is complete

    bool alive = true;   // false after a wait that timed out: no more waits, no more work, only the barriers
    for (uint32_t n = 0;; ++n) {
      const uint32_t par = n & 1u;
      // All 256 threads leave the loop together: the decision is taken on a value that every thread reads
      // after the same barrier phase.
      bool got_item = false;
      if (alive) {
        for (uint32_t w = 0; w < kItemWaitRounds && !got_item; ++w) got_item = mbar_wait(bar_item, par, a.status);
      }
      const int item = got_item ? item_ring[par] : -1;
      if (item < 0) break;
      const int tile = item / a.bh, bhid = item - tile * a.bh;
      const int h = bhid % a.heads;
      // G > 1: the tile holds G windows of R rows each (window `slot` in rows and columns slot R .. slot R + R - 1 of
      // the block-diagonal score tile); a warp's 32 rows lie inside one window
      const int slot = kPack ? trow / a.R : 0;
      const int b = kPack ? (bhid / a.heads) * a.G + slot : bhid / a.heads;   // image / window of this row
      const int m0 = tile * 128;
      const int col0 = kPack ? slot * a.R : 0;      // first row and first score column of this row's window in the tile
      const int r = m0 + trow - col0;               // token (row) inside this image / window
      const bool row_ok = r < a.T && (!kPack || b < a.Btot);
      const bool warp_ok = m0 + qd * 32 - col0 < a.T && (!kPack || b < a.Btot);   // warps whose 32 rows all lie past T only keep the barriers
      const int c_lo = col0 >> 4, c_hi = kPack ? c_lo + (a.R >> 4) : nch;   // this row's 16-column chunks
      // Plain form: the passes work on the chunks that hold columns; when the last of them holds at most eight, it is
      // taken as one 8-column piece by the second thread of the row (whose share of full chunks is never the larger
      // one), and chunks wholly past T only get their zero probabilities written.
      const int c_real = kPack ? c_hi : (a.T + 15) >> 4;
      const bool tail8 = !kPack && (a.T & 15) != 0 && (a.T & 15) <= 8;
      const int c_end = tail8 ? c_real - 1 : c_real;   // chunks worked on sixteen columns at a time
      const int ct = c_end * 16;                       // first column of the 8-column piece
      const int32_t* brow = a.bias ? a.bias + ((((int64_t)b * a.heads + h) % a.bias_batches) * a.T + (row_ok ? r : 0)) * (int64_t)a.T - col0 : nullptr;

      int mx = -128;
      bool got_s = mbar_wait(bar_s, par, a.status);
      alive = alive && got_s;
      if (got_s) tc_fence_after();
      if (got_s && warp_ok) {
        // pass A: requantise the scores to int8 (Sec. 3.2), running maximum.  The two threads of a row take
        // alternate 16-column chunks (Npad / 16 is even: equal shares).  The chunk loops are rolled (the kernel's
        // code stays within the instruction cache); what a later pass needs of a chunk waits in the chunk's own
        // tensor-memory columns.
#pragma unroll 1
        for (int c = c_lo + half; c < c_end; c += 2) {
          int v[16];
          tmem_ld16(t_row + c * 16, v);
          if (brow) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c * 16 + j - col0 < a.T) v[j] += __ldg(brow + c * 16 + j);
          }
          if (qk_hi) {          // the usual case: high product word plus 2^(s-33), shifted by s - 32
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = mad_hi(v[j], a.qk_m, qk_rnd) >> qk_sh;
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = (int)(((long long)v[j] * a.qk_m + qk_c) >> a.qk_s);
          }
          // columns past T (only in the last two chunks) never win the maximum and look up a valid table entry
          if (c >= c_end - 2) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c * 16 + j - col0 >= a.T) v[j] = -128;
          }
          // running maximum on the unsaturated values (saturation is monotone: it is applied to the result)
          int m = v[0];
#pragma unroll
          for (int j = 1; j < 16; j += 2) m = max(m, max(v[j], v[(j + 1) & 15]));
          mx = max(mx, m);
          // scores are kept as biased bytes (x + 128, i.e. x ^ 0x80) so that pass B can index with them:
          // four per word in the first four columns of the chunk
          uint32_t xs[4];
#pragma unroll
          for (int k = 0; k < 4; ++k)
            xs[k] = pack_sat8(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]) ^ 0x80808080u;
          tmem_st4(t_row + c * 16, xs);
        }
        if (tail8 && half == 1) {
          int v[8];
          tmem_ld8(t_row + ct, v);
          if (brow) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (ct + j < a.T) v[j] += __ldg(brow + ct + j);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            v[j] = qk_hi ? mad_hi(v[j], a.qk_m, qk_rnd) >> qk_sh : (int)(((long long)v[j] * a.qk_m + qk_c) >> a.qk_s);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (ct + j >= a.T) v[j] = -128;
          mx = max(mx, max(max(max(v[0], v[1]), max(v[2], v[3])), max(max(v[4], v[5]), max(v[6], v[7]))));
          const uint32_t xs2[2] = {pack_sat8(v[0], v[1], v[2], v[3]) ^ 0x80808080u, pack_sat8(v[4], v[5], v[6], v[7]) ^ 0x80808080u};
          tmem_st2(t_row + ct, xs2);
        }
        tmem_st_wait();
        mx = max(-128, min(127, mx));
        part_max[half * 128 + trow] = mx;
      }
      // only the two warps that share these 32 rows exchange partial results: a barrier of their own
      asm volatile("bar.sync %0, 64;" ::"r"(2 + qd) : "memory");
      unsigned sum = 0;
      if (got_s && warp_ok) {
        mx = max(part_max[trow], part_max[128 + trow]);
        // pass B: ShiftExp(I - I_max) by table, row sum, exponentials back into tensor memory
        // entry (I_max - I) of the table = word at tab + 4*(I_max + 128) - 4*(I + 128)
        const uint8_t* tmx = reinterpret_cast<const uint8_t*>(tab) + 4 * (mx + 128);
#pragma unroll 1
        for (int c = c_lo + half; c < c_end; c += 2) {
          int ev[16];
          uint32_t xs[4];
          tmem_ld4(t_row + c * 16, xs);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t w = xs[k];
#pragma unroll
            for (int bb = 0; bb < 4; ++bb)
              ev[4 * k + bb] = (int)*reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(w, 0, 0x4440 + bb));
          }
          if (c >= c_end - 2) {   // columns past T contribute nothing
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c * 16 + j - col0 >= a.T) ev[j] = 0;
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) sum += (unsigned)ev[j];
          tmem_st16(t_row + c * 16, ev);
        }
        if (tail8 && half == 1) {
          int ev[8];
          uint32_t xs2[2];
          tmem_ld2(t_row + ct, xs2);
#pragma unroll
          for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int bb = 0; bb < 4; ++bb)
              ev[4 * k + bb] = (int)*reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(xs2[k], 0, 0x4440 + bb));
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (ct + j >= a.T) ev[j] = 0;
            sum += (unsigned)ev[j];
          }
          tmem_st8(t_row + ct, ev);
        }
        tmem_st_wait();
        part_sum[half * 128 + trow] = sum;
      }
      asm volatile("bar.sync %0, 64;" ::"r"(2 + qd) : "memory");
      if (got_s && warp_ok) {
        sum = part_sum[trow] + part_sum[128 + trow];
        // pass C: Eq. (IntDiv) with M = 45 (prob_word)
        const unsigned factor = (unsigned)((1ull << 45) / (unsigned long long)(sum ? sum : 1u));
#pragma unroll 1
        for (int c = c_lo + half; c < c_end; c += 2) {
          int ev[16];
          tmem_ld16(t_row + c * 16, ev);
          uint32_t w[4];
#pragma unroll
          for (int k = 0; k < 4; ++k)
            w[k] = prob_word<K8>(factor, ev[4 * k], ev[4 * k + 1], ev[4 * k + 2], ev[4 * k + 3], 14 - a.smax.k_out, (1 << (a.smax.k_out - 1)) - 1);
          // A operand of P V: row = tile row, k-block = 128 columns, 16-byte pieces XOR (row & 7)
          uint8_t* prow = gen + p_off + (c >> 3) * (128 * 128) + trow * 128;
          *reinterpret_cast<uint4*>(prow + ((((c & 7)) ^ (trow & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (!kPack) {
          if (tail8 && half == 1) {   // the 8-column piece and eight zeros
            int ev[8];
            tmem_ld8(t_row + ct, ev);
            const uint32_t w0 = prob_word<K8>(factor, ev[0], ev[1], ev[2], ev[3], 14 - a.smax.k_out, (1 << (a.smax.k_out - 1)) - 1);
            const uint32_t w1 = prob_word<K8>(factor, ev[4], ev[5], ev[6], ev[7], 14 - a.smax.k_out, (1 << (a.smax.k_out - 1)) - 1);
            uint8_t* prow = gen + p_off + (c_end >> 3) * (128 * 128) + trow * 128;
            *reinterpret_cast<uint4*>(prow + ((((c_end & 7)) ^ (trow & 7)) << 4)) = make_uint4(w0, w1, 0u, 0u);
          }
          // chunks wholly past T: probability 0 (the contraction of P V runs over Npad columns)
          for (int c = c_real + half; c < nch; c += 2) {
            uint8_t* prow = gen + p_off + (c >> 3) * (128 * 128) + trow * 128;
            *reinterpret_cast<uint4*>(prow + ((((c & 7)) ^ (trow & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        if (kPack) {   // the other windows' columns of this row: probability 0, so that P V stays inside the window
          for (int c = half; c < nch; c += 2)
            if (c < c_lo || c >= c_hi)
              *reinterpret_cast<uint4*>(gen + p_off + trow * 128 + ((((c & 7)) ^ (trow & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
      // ---- output: O = sat8(rq(P V; pv_scale)), heads concatenated along the feature dimension ----
      const bool got_o = alive && mbar_wait(bar_o, par, a.status);
      alive = alive && got_o;
      if (got_o) {
        tc_fence_after();
        const long long pv_c = 1ll << (a.pv_s - 1);
        int8_t* orow = a.O + ((int64_t)b * a.T + r) * a.D + (int64_t)h * a.d;
        for (int c = half; c < a.d / 32; c += 2) {
          if (!warp_ok) break;
          int v[32];
          tmem_ld32(t_row + c * 32, v);
          if (row_ok) {
            if (a.pv_s >= 33) {   // high product word plus 2^(s-33), shifted by s - 32
              const int pv_rnd = 1 << (a.pv_s - 33), pv_sh = a.pv_s - 32;
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = mad_hi(v[j], a.pv_m, pv_rnd) >> pv_sh;
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = (int)(((long long)v[j] * a.pv_m + pv_c) >> a.pv_s);
            }
            int4 w0, w1;
            w0.x = (int)pack_sat8(v[0], v[1], v[2], v[3]);     w0.y = (int)pack_sat8(v[4], v[5], v[6], v[7]);
            w0.z = (int)pack_sat8(v[8], v[9], v[10], v[11]);   w0.w = (int)pack_sat8(v[12], v[13], v[14], v[15]);
            w1.x = (int)pack_sat8(v[16], v[17], v[18], v[19]); w1.y = (int)pack_sat8(v[20], v[21], v[22], v[23]);
            w1.z = (int)pack_sat8(v[24], v[25], v[26], v[27]); w1.w = (int)pack_sat8(v[28], v[29], v[30], v[31]);
            reinterpret_cast<int4*>(orow + c * 32)[0] = w0;
            reinterpret_cast<int4*>(orow + c * 32)[1] = w1;
          }
        }
      }
      // tensor memory may take the next item's scores
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_e);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    // the last CTA to finish leaves the counters at zero for the next launch
    __threadfence();
    if (atomicAdd(a.sched + 1, 1u) == gridDim.x - 1) {
      a.sched[0] = 0;
      a.sched[1] = 0;
      __threadfence();
    }
  }
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
  }
}

// ------------------------------------------------------------------------------------------------------------
// Rows longer than 256 tokens.  The score tile of a 128-row block no longer fits tensor memory, so the keys are
// taken in blocks of NB columns (the last block holds the remainder): S_j = Q K_j^T goes into one of two
// tensor-memory buffers, pass A requantises it and parks the int8 scores in shared memory, in the very place and
// layout (K-major, 128-byte swizzle) where the probabilities of the second MMA's A operand will stand, while the
// MMA of the next block fills the other buffer.  After the last block the row maximum is known: pass B sums the
// exponentials from the parked bytes, pass C turns the bytes into probabilities in place, and O = P V accumulates
// over the whole row in its own tensor-memory columns.  One CTA per SM; four threads share a score row (one TMEM
// lane; each takes a quarter of every key block).  The control thread runs one block ahead of the Shiftmax
// threads, also across work items.
constexpr int kLongThreads = 544;   // warp 0: TMA + MMA issue + TMEM owner; warps 1..16: four threads per score row

struct LongArgs {
  AttnArgs a;
  int NB;      // key-block width, a multiple of 32
  int nblk;    // key blocks per row (>= 2)
  int nv;      // 256-row boxes that bring V
};

__device__ __forceinline__ void tmem_ld_cols(uint32_t addr, int (&v)[16]) { tmem_ld16(addr, v); }
__device__ __forceinline__ void tmem_ld_cols(uint32_t addr, int (&v)[8]) { tmem_ld8_issue(addr, v); tmem_ld_wait8(v); }

template <bool K8>
__global__ void __launch_bounds__(kLongThreads, 1) attention_long_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                        const __grid_constant__ CUtensorMap tmK,
                                                                        const __grid_constant__ CUtensorMap tmV, LongArgs la) {
  const AttnArgs& a = la.a;
  const int NB = la.NB, nblk = la.nblk;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // [Q 128x128B][K block x 2][V 256 nv x d][P / parked scores 128 x 128B x kblocks][exp table][row partials][item ring][barriers]
  const uint32_t q_off = 0, k_off = 128 * 128, kbuf_bytes = (uint32_t)NB * 128;
  const uint32_t v_off = k_off + 2 * kbuf_bytes, v_bytes = (uint32_t)la.nv * 256 * a.d;
  const uint32_t p_off = (v_off + v_bytes + 1023u) & ~1023u;
  const uint32_t tab_off = p_off + (uint32_t)((a.Npad + 127) / 128) * 128 * 128;
  const uint32_t part_off = tab_off + 1024;              // [4 column quarters][128 rows] partial max, then partial sum
  const uint32_t item_off = part_off + 4 * 128 * 4 * 2;  // [2] work item of even / odd iterations (-1: no more work)
  const uint32_t bar_off = item_off + 16;
  unsigned* tab = reinterpret_cast<unsigned*>(gen + tab_off);
  volatile int* item_ring = reinterpret_cast<volatile int*>(gen + item_off);
  // Q landed | V landed | K block landed (x2) | scores ready (x2) | score buffer read (x2) | probabilities written |
  // output ready | output read | item published
  const uint32_t bar_q = base + bar_off, bar_v = bar_q + 8, bar_k = bar_q + 16, bar_s = bar_q + 32, bar_f = bar_q + 48,
                 bar_p = bar_q + 64, bar_o = bar_q + 72, bar_e = bar_q + 80, bar_item = bar_q + 88;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + bar_off + 128);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(bar_q, 1);
    mbar_init(bar_v, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_k + 8 * i, 1);
      mbar_init(bar_s + 8 * i, 1);
      mbar_init(bar_f + 8 * i, 16);
    }
    mbar_init(bar_p, 16);
    mbar_init(bar_o, 1);
    mbar_init(bar_e, 16);
    mbar_init(bar_item, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t o_col = 2u * (uint32_t)NB;   // output accumulator behind the two score buffers
  pdl_trigger();
  if (warp == 0) pdl_wait();   // the QKV tensor comes from the previous kernel; the other warps build their table first

  if (warp == 0) {
    if (lane == 0) {
      auto coords = [&](int item, int& tile, int& h, int& b) {
        tile = item / a.bh;
        const int bhid = item - tile * a.bh;
        h = bhid % a.heads;
        b = bhid / a.heads;
      };
      auto load_q = [&](int item) {
        int tile, h, b;
        coords(item, tile, h, b);
        mbar_expect_tx(bar_q, 128 * 128);
        int c[4];
        c[0] = 0; c[a.q_pos[0]] = tile * 128; c[a.q_pos[1]] = h; c[a.q_pos[2]] = b;
        tma_load_4d(base + q_off, &tmQ, bar_q, c[0], c[1], c[2], c[3]);
      };
      auto load_k = [&](int item, int j, uint32_t buf) {
        int tile, h, b;
        coords(item, tile, h, b);
        mbar_expect_tx(bar_k + 8 * buf, kbuf_bytes);
        int c[4];
        c[0] = 0; c[a.k_pos[0]] = j * NB; c[a.k_pos[1]] = h; c[a.k_pos[2]] = b;
        tma_load_4d(base + k_off + buf * kbuf_bytes, &tmK, bar_k + 8 * buf, c[0], c[1], c[2], c[3]);
      };
      auto load_v = [&](int item) {
        int tile, h, b;
        coords(item, tile, h, b);
        mbar_expect_tx(bar_v, v_bytes);
        for (int i = 0; i < la.nv; ++i) {
          int c[4];
          c[0] = 0; c[a.v_pos[0]] = i * 256; c[a.v_pos[1]] = h; c[a.v_pos[2]] = b;
          tma_load_4d(base + v_off + (uint32_t)i * 256u * a.d, &tmV, bar_v, c[0], c[1], c[2], c[3]);
        }
      };
      auto draw = [&]() {
        const unsigned t = atomicAdd(a.sched, 1u);
        return t < (unsigned)a.items ? (int)t : -1;
      };
      auto publish = [&](uint32_t n, int item) {
        item_ring[n & 1u] = item;
        mbar_arrive(bar_item);   // release: the item is visible to whoever sees this phase complete
      };
      const uint32_t idesc2 = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(a.d >> 3) << 17) | (8u << 24);
      const uint32_t v_layout = a.d == 128 ? 2u : (a.d == 64 ? 4u : 6u);
      const int ks = (a.d + UK - 1) / UK, ks2 = a.Npad / UK;

      uint32_t g = 0;            // key blocks issued so far, over all items of this CTA
      bool ok = true;
      bool q_fly = false, v_fly = false, k_fly[2] = {false, false};   // loads requested and not yet waited for
      uint32_t q_par = 0, v_par = 0, k_par[2] = {0, 0};
      // S_buf = Q K_j^T for key block j of `item` (the n-th item of this CTA), then the load of the key block that
      // follows it in the order of issue: block j + 1 of the same item, or block 0 of `next_item`.
      auto issue_block = [&](int item, int j, uint32_t n, int next_item) {
        const uint32_t buf = g & 1u, ph = (g >> 1) & 1u;
        ok = mbar_wait(bar_k + 8 * buf, ph, a.status);
        k_fly[buf] = !ok;
        if (ok && j == 0) { ok = mbar_wait(bar_q, n & 1u, a.status); q_fly = !ok; }
        // pass A of the block that used this score buffer two blocks ago has read it
        if (ok && g >= 2) ok = mbar_wait(bar_f + 8 * buf, ph ^ 1u, a.status);
        if (!ok) return;
        tc_fence_after();
        const int w = j == nblk - 1 ? a.Npad - j * NB : NB;
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(w >> 3) << 17) | (8u << 24);
        for (int k = 0; k < ks; ++k)
          umma_i8(tmem + buf * (uint32_t)NB, smem_desc(base + q_off + k * UK, 16, 1024, 2),
                  smem_desc(base + k_off + buf * kbuf_bytes + k * UK, 16, 1024, 2), idesc, k != 0);
        umma_commit(bar_s + 8 * buf);
        const int fj = j + 1 < nblk ? j + 1 : 0;
        const int fitem = j + 1 < nblk ? item : next_item;
        if (fitem >= 0) {
          // the other key buffer was read by the MMAs of the block before this one
          if (g >= 1) ok = mbar_wait(bar_s + 8 * (buf ^ 1u), ((g - 1) >> 1) & 1u, a.status);
          if (!ok) return;
          load_k(fitem, fj, buf ^ 1u);
          k_fly[buf ^ 1u] = true;
          k_par[buf ^ 1u] = ((g + 1) >> 1) & 1u;
        }
        ++g;
      };

      int cur = draw();
      uint32_t n = 0;
      bool first_issued = false;   // block 0 of `cur` went out at the end of the item before it
      if (cur >= 0) {
        load_q(cur); q_fly = true; q_par = 0;
        load_v(cur); v_fly = true; v_par = 0;
        load_k(cur, 0, 0); k_fly[0] = true; k_par[0] = 0;
        publish(0, cur);
      }
      while (cur >= 0) {
        int next = -1;
        for (int j = first_issued ? 1 : 0; ok && j < nblk; ++j) {
          if (j == nblk - 1) next = draw();
          issue_block(cur, j, n, next);
        }
        if (!ok) break;
        // Q may be overwritten once the score MMAs of the last block have read it
        ok = mbar_wait(bar_s + 8 * ((g - 1) & 1u), ((g - 1) >> 1) & 1u, a.status);
        if (!ok) break;
        if (next >= 0) {
          load_q(next); q_fly = true; q_par = (n + 1) & 1u;
          // The item barrier may run one phase ahead of its readers at most: every Shiftmax warp has taken item n
          // once it has handed back the score buffer of that item's last key block (the latest phase of that
          // barrier: the block that completes it next has not been issued yet).
          ok = mbar_wait(bar_f + 8 * ((g - 1) & 1u), ((g - 1) >> 1) & 1u, a.status);
          if (!ok) break;
          publish(n + 1, next);
          issue_block(next, 0, n + 1, -1);   // nblk >= 2: the block after it belongs to the same item
          if (!ok) break;
        }
        // O = P V once the probabilities are in shared memory, V has landed and the previous output has been read
        ok = mbar_wait(bar_p, n & 1u, a.status);
        if (ok) { ok = mbar_wait(bar_v, n & 1u, a.status); v_fly = !ok; }
        if (ok && n > 0) ok = mbar_wait(bar_e, (n - 1) & 1u, a.status);
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < ks2; ++k) {
          const uint32_t pa = base + p_off + (k >> 2) * (128 * 128) + (k & 3) * UK;
          umma_i8(tmem + o_col, smem_desc(pa, 16, 1024, 2), smem_desc(base + v_off + k * UK * a.d, 16, 8 * a.d, v_layout),
                  idesc2, k != 0);
        }
        umma_commit(bar_o);
        // V (and the probabilities) may be overwritten once these MMAs have read them
        ok = mbar_wait(bar_o, n & 1u, a.status);
        if (!ok) break;
        if (next >= 0) { load_v(next); v_fly = true; v_par = (n + 1) & 1u; }
        cur = next;
        ++n;
        first_issued = true;
      }
      // end of work (or a wait that timed out): tell the other warps; nothing may be in flight at exit
      publish(ok ? n : n + 1, -1);
      if (q_fly) mbar_wait(bar_q, q_par, a.status);
      if (v_fly) mbar_wait(bar_v, v_par, a.status);
      for (int i = 0; i < 2; ++i)
        if (k_fly[i]) mbar_wait(bar_k + 8 * i, k_par[i], a.status);
    }
  } else {
    // ---- Shiftmax / epilogue threads: TMEM lane quarter = warp % 4; the four warps of a quarter take the four
    //      quarters of every key block of the same 32 rows ----
    const int st = threadIdx.x - 32;   // 0..511
    if (st < 256) tab[st] = shiftexp(-st, a.smax.I0, a.smax.N);
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 32) {
      a.sched_other[0] = 0;
      a.sched_other[1] = 0;
    }
    const int qd = warp & 3;
    const int part = (warp - 1) >> 2;             // 0..3
    const int trow = qd * 32 + lane;              // row inside the tile
    const uint32_t t_row = tmem + ((uint32_t)(qd * 32) << 16);
    const bool qk_hi = a.qk_s >= 33;              // rounding constant and shift both past the low product word
    const long long qk_c = 1ll << (a.qk_s - 1);
    const int qk_rnd = qk_hi ? 1 << (a.qk_s - 33) : 0, qk_sh = a.qk_s - 32;
    int* part_max = reinterpret_cast<int*>(gen + part_off);
    unsigned* part_sum = reinterpret_cast<unsigned*>(gen + part_off + 4 * 128 * 4);
    uint8_t* p_row = gen + p_off + trow * 128;    // this row inside every 128-column block of P
    // byte address of 8 or 16 consecutive columns (col a multiple of 8 / 16) of this row in the A-operand layout
    auto p_addr = [&](int col) { return p_row + (col >> 7) * (128 * 128) + ((((col >> 4) & 7) ^ (trow & 7)) << 4) + (col & 8); };
    // this thread's pieces of key block j: whole 16-column chunks, an 8-column piece in front / behind when the
    // quarter starts / ends on an odd multiple of 8
    auto walk = [&](int j, auto&& fn) {
      const int cb = j * NB;
      const int w = j == nblk - 1 ? a.Npad - cb : NB;
      const int lo = cb + part * (w >> 2), hi = lo + (w >> 2);
      const int c16_lo = (lo + 15) & ~15, c16_hi = hi & ~15;
      if (lo & 8) { int v[8]; fn(v, lo, cb); }
#pragma unroll 1
      for (int c = c16_lo; c < c16_hi; c += 16) { int v[16]; fn(v, c, cb); }
      if (hi & 8) { int v[8]; fn(v, c16_hi, cb); }
    };
    asm volatile("bar.sync 1, 512;" ::: "memory");   // the table is complete

    bool alive = true;   // false after a wait that timed out: no more waits, no more work, only the barriers
    uint32_t g = 0;      // key blocks seen so far (same count as the control thread's)
    for (uint32_t n = 0;; ++n) {
      const uint32_t par = n & 1u;
      bool got_item = false;
      if (alive) {
        for (uint32_t w = 0; w < kItemWaitRounds && !got_item; ++w) got_item = mbar_wait(bar_item, par, a.status);
      }
      const int item = got_item ? item_ring[par] : -1;
      if (item < 0) break;
      const int tile = item / a.bh, bhid = item - tile * a.bh;
      const int h = bhid % a.heads, b = bhid / a.heads;
      const int m0 = tile * 128;
      const int r = m0 + trow;                      // token (row) inside this image
      const bool row_ok = r < a.T;
      const bool warp_ok = m0 + qd * 32 < a.T;      // warps whose 32 rows all lie past T only keep the barriers
      const int32_t* brow = a.bias ? a.bias + (((int64_t)bhid % a.bias_batches) * a.T + (row_ok ? r : 0)) * (int64_t)a.T : nullptr;

      // pass A, key block by key block: requantise the scores to int8 (Sec. 3.2), park them as biased bytes
      // (x + 128) where the probabilities will stand, running maximum
      int mx = -128;
      for (int j = 0; j < nblk; ++j, ++g) {
        const uint32_t buf = g & 1u;
        const bool got_s = alive && mbar_wait(bar_s + 8 * buf, (g >> 1) & 1u, a.status);
        alive = alive && got_s;
        if (got_s) tc_fence_after();
        if (got_s && warp_ok) {
          const uint32_t t_buf = t_row + buf * (uint32_t)NB;
          walk(j, [&](auto& v, int col, int cb) {
            constexpr int W = (int)(sizeof(v) / sizeof(v[0]));
            tmem_ld_cols(t_buf + (uint32_t)(col - cb), v);
            if (brow) {
#pragma unroll
              for (int i = 0; i < W; ++i)
                if (col + i < a.T) v[i] += __ldg(brow + col + i);
            }
            if (qk_hi) {          // the usual case: high product word plus 2^(s-33), shifted by s - 32
#pragma unroll
              for (int i = 0; i < W; ++i) v[i] = mad_hi(v[i], a.qk_m, qk_rnd) >> qk_sh;
            } else {
#pragma unroll
              for (int i = 0; i < W; ++i) v[i] = (int)(((long long)v[i] * a.qk_m + qk_c) >> a.qk_s);
            }
            if (col + W > a.T) {  // columns past T never win the maximum
#pragma unroll
              for (int i = 0; i < W; ++i)
                if (col + i >= a.T) v[i] = -128;
            }
            int m = v[0];
#pragma unroll
            for (int i = 1; i < W; i += 2) m = max(m, max(v[i], v[(i + 1) & (W - 1)]));
            mx = max(mx, m);
            uint32_t xs[W / 4];
#pragma unroll
            for (int k = 0; k < W / 4; ++k)
              xs[k] = pack_sat8(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]) ^ 0x80808080u;
            if constexpr (W == 16) *reinterpret_cast<uint4*>(p_addr(col)) = make_uint4(xs[0], xs[1], xs[2], xs[3]);
            else *reinterpret_cast<uint2*>(p_addr(col)) = make_uint2(xs[0], xs[1]);
          });
        }
        // the score buffer may take the block after the next one
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_f + 8 * buf);
      }
      if (alive && warp_ok) part_max[part * 128 + trow] = max(-128, min(127, mx));
      // only the four warps that share these 32 rows exchange partial results: a barrier of their own
      asm volatile("bar.sync %0, 128;" ::"r"(2 + qd) : "memory");
      unsigned sum = 0;
      const uint8_t* tmx = nullptr;
      if (alive && warp_ok) {
        mx = max(max(part_max[trow], part_max[128 + trow]), max(part_max[256 + trow], part_max[384 + trow]));
        // pass B: ShiftExp(I - I_max) by table, row sum.  Entry (I_max - I) = word at tab + 4 (I_max + 128) - 4 (I + 128)
        tmx = reinterpret_cast<const uint8_t*>(tab) + 4 * (mx + 128);
        for (int j = 0; j < nblk; ++j) {
          walk(j, [&](auto& ev, int col, int) {
            constexpr int W = (int)(sizeof(ev) / sizeof(ev[0]));
            uint32_t xs[W / 4];
            if constexpr (W == 16) { const uint4 q = *reinterpret_cast<const uint4*>(p_addr(col)); xs[0] = q.x; xs[1] = q.y; xs[2] = q.z; xs[3] = q.w; }
            else { const uint2 q = *reinterpret_cast<const uint2*>(p_addr(col)); xs[0] = q.x; xs[1] = q.y; }
#pragma unroll
            for (int k = 0; k < W / 4; ++k)
#pragma unroll
              for (int bb = 0; bb < 4; ++bb)
                ev[4 * k + bb] = (int)*reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(xs[k], 0, 0x4440 + bb));
            if (col + W > a.T) {   // columns past T contribute nothing
#pragma unroll
              for (int i = 0; i < W; ++i)
                if (col + i >= a.T) ev[i] = 0;
            }
#pragma unroll
            for (int i = 0; i < W; ++i) sum += (unsigned)ev[i];
          });
        }
        part_sum[part * 128 + trow] = sum;
      }
      asm volatile("bar.sync %0, 128;" ::"r"(2 + qd) : "memory");
      if (alive && warp_ok) {
        sum = (part_sum[trow] + part_sum[128 + trow]) + (part_sum[256 + trow] + part_sum[384 + trow]);
        // pass C: Eq. (IntDiv) with M = 45 (prob_word),
        // the parked score bytes turned into probabilities in place
        const unsigned factor = (unsigned)((1ull << 45) / (unsigned long long)(sum ? sum : 1u));
        for (int j = 0; j < nblk; ++j) {
          walk(j, [&](auto& ev, int col, int) {
            constexpr int W = (int)(sizeof(ev) / sizeof(ev[0]));
            uint32_t xs[W / 4];
            if constexpr (W == 16) { const uint4 q = *reinterpret_cast<const uint4*>(p_addr(col)); xs[0] = q.x; xs[1] = q.y; xs[2] = q.z; xs[3] = q.w; }
            else { const uint2 q = *reinterpret_cast<const uint2*>(p_addr(col)); xs[0] = q.x; xs[1] = q.y; }
#pragma unroll
            for (int k = 0; k < W / 4; ++k)
#pragma unroll
              for (int bb = 0; bb < 4; ++bb)
                ev[4 * k + bb] = (int)*reinterpret_cast<const unsigned*>(tmx - 4 * (int)__byte_perm(xs[k], 0, 0x4440 + bb));
            if (col + W > a.T) {
#pragma unroll
              for (int i = 0; i < W; ++i)
                if (col + i >= a.T) ev[i] = 0;
            }
#pragma unroll
            for (int k = 0; k < W / 4; ++k)
              xs[k] = prob_word<K8>(factor, ev[4 * k], ev[4 * k + 1], ev[4 * k + 2], ev[4 * k + 3], 14 - a.smax.k_out, (1 << (a.smax.k_out - 1)) - 1);
            if constexpr (W == 16) *reinterpret_cast<uint4*>(p_addr(col)) = make_uint4(xs[0], xs[1], xs[2], xs[3]);
            else *reinterpret_cast<uint2*>(p_addr(col)) = make_uint2(xs[0], xs[1]);
          });
        }
        fence_async_smem();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
      // ---- output: O = sat8(rq(P V; pv_scale)), heads concatenated along the feature dimension ----
      const bool got_o = alive && mbar_wait(bar_o, par, a.status);
      alive = alive && got_o;
      if (got_o) {
        tc_fence_after();
        const long long pv_c = 1ll << (a.pv_s - 1);
        int8_t* orow = a.O + ((int64_t)b * a.T + r) * a.D + (int64_t)h * a.d;
        for (int c = part; c < a.d / 16; c += 4) {
          if (!warp_ok) break;
          int v[16];
          tmem_ld16(t_row + 2u * (uint32_t)NB + c * 16, v);
          if (row_ok) {
            if (a.pv_s >= 33) {   // high product word plus 2^(s-33), shifted by s - 32
              const int pv_rnd = 1 << (a.pv_s - 33), pv_sh = a.pv_s - 32;
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] = mad_hi(v[i], a.pv_m, pv_rnd) >> pv_sh;
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] = (int)(((long long)v[i] * a.pv_m + pv_c) >> a.pv_s);
            }
            int4 w0;
            w0.x = (int)pack_sat8(v[0], v[1], v[2], v[3]);     w0.y = (int)pack_sat8(v[4], v[5], v[6], v[7]);
            w0.z = (int)pack_sat8(v[8], v[9], v[10], v[11]);   w0.w = (int)pack_sat8(v[12], v[13], v[14], v[15]);
            *reinterpret_cast<int4*>(orow + c * 16) = w0;
          }
        }
      }
      // the output columns of tensor memory may take the next item's P V
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_e);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    // the last CTA to finish leaves the counters at zero for the next launch
    __threadfence();
    if (atomicAdd(a.sched + 1, 1u) == gridDim.x - 1) {
      a.sched[0] = 0;
      a.sched[1] = 0;
      __threadfence();
    }
  }
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 512u);
  }
}

}  // namespace

// The shared-memory limit of a kernel is a per-device attribute: set for the current device at context creation.
int attention_prepare_device() {
  if (cudaFuncSetAttribute(attention_long_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(attention_long_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(attention_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(attention_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(attention_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(attention_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
    return IVIT_ERR_CUDA;
  return IVIT_OK;
}

// Rows longer than 256 tokens: key blocks, one CTA per SM.  IVIT_ERR_UNSUPPORTED when the row does not fit the
// kernel's shared memory (the probabilities of a 128-row tile and the whole V of a head stay resident).
static int launch_attention_long(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O) {
  const int64_t B = p->B, T = p->T, D = p->D, h = p->heads, d = D / h;
  LongArgs la{};
  AttnArgs& a = la.a;
  a.T = (int)T; a.d = (int)d; a.heads = (int)h; a.D = D;
  a.Npad = (int)((T + 31) / 32 * 32);
  a.tiles_m = (int)((T + 127) / 128);
  a.tmem_cols = 512;
  a.G = 1; a.R = 128; a.Btot = (int)B;
  int nb_max = ((512 - (int)d) / 2) / 32 * 32 > 224 ? 224 : ((512 - (int)d) / 2) / 32 * 32;   // two score buffers + d output columns
  la.nblk = (a.Npad + nb_max - 1) / nb_max;
  la.NB = ((a.Npad + la.nblk - 1) / la.nblk + 31) / 32 * 32;
  la.nv = (a.Npad + 255) / 256;
  if (la.nblk < 2 || la.NB * (la.nblk - 1) >= a.Npad) return IVIT_ERR_UNSUPPORTED;
  const uint32_t v_off = 128 * 128 + 2 * la.NB * 128;
  const uint32_t p_off = (v_off + (uint32_t)la.nv * 256 * (uint32_t)d + 1023u) & ~1023u;
  const size_t smem = 1024 + p_off + (size_t)((a.Npad + 127) / 128) * 128 * 128 + 1024 + 4096 + 16 + 128 + 16;
  if (smem > 227 * 1024) return IVIT_ERR_UNSUPPORTED;
  a.qk_m = p->qk_scale.mult; a.qk_s = clamp_shift(p->qk_scale.shift);
  a.pv_m = p->pv_scale.mult; a.pv_s = clamp_shift(p->pv_scale.shift);
  a.smax = p->smax;
  a.bias = p->attn_bias; a.bias_batches = p->attn_bias ? p->attn_bias_batches : 1;
  a.O = O;
  a.status = ctx->status_dev;
  const int64_t ldq = 3 * D;
  CUtensorMap tmQ, tmK, tmV;
  const CUtensorMapSwizzle vsw = d == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (d == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  if (!make_tensor_map(ctx, &tmQ, QKV, d, T, h, B, ldq, d, T * ldq, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B, a.q_pos) ||
      !make_tensor_map(ctx, &tmK, QKV + D, d, T, h, B, ldq, d, T * ldq, 128, la.NB, CU_TENSOR_MAP_SWIZZLE_128B, a.k_pos) ||
      !make_tensor_map(ctx, &tmV, QKV + 2 * D, d, T, h, B, ldq, d, T * ldq, (int)d, 256, vsw, a.v_pos))
    return IVIT_ERR_UNSUPPORTED;
  a.bh = (int)(B * h);
  a.items = (int)(B * h * a.tiles_m);
  a.sched = ctx->sched_dev + 2 * ctx->attn_gen;
  a.sched_other = ctx->sched_dev + 2 * (ctx->attn_gen ^ 1);
  ctx->attn_gen ^= 1;
  const int64_t grid = a.items < ctx->sm_count ? a.items : ctx->sm_count;
  LaunchScope ls(ctx, KIND_ATTENTION, 4.0 * (double)(B * h) * (double)T * (double)T * (double)d);
  if (p->smax.k_out == 8) launch_k(attention_long_kernel<true>, dim3((unsigned)grid), dim3(kLongThreads), smem, ctx->stream, tmQ, tmK, tmV, la);
  else launch_k(attention_long_kernel<false>, dim3((unsigned)grid), dim3(kLongThreads), smem, ctx->stream, tmQ, tmK, tmV, la);
  return ls.done();
}

// Returns IVIT_ERR_UNSUPPORTED when the shape is outside the fused kernels (d not 32/64/128, rows too long for
// shared memory, misaligned tensors); the caller then composes the attention from MatMul and Shiftmax kernels.
int launch_attention_fused(ivit_ctx* ctx, const ivit_block_params* p, const int8_t* QKV, int8_t* O) {
  if (!ctx->tmap_encode) return IVIT_ERR_UNSUPPORTED;
  const int64_t B = p->B, T = p->T, D = p->D, h = p->heads, d = D / h;
  if ((d != 32 && d != 64 && d != 128) || B * h > 2147483647LL / 8) return IVIT_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(QKV) & 15) || (reinterpret_cast<uintptr_t>(O) & 15)) return IVIT_ERR_UNSUPPORTED;
  if (B == 0) return IVIT_OK;
  if (T > 256) return launch_attention_long(ctx, p, QKV, O);
  AttnArgs a{};
  a.T = (int)T; a.d = (int)d; a.heads = (int)h; a.D = D;
  a.Npad = (int)((T + 31) / 32 * 32);
  a.tiles_m = (int)((T + 127) / 128);
  // Short rows (window attention): 2 windows of up to 64 tokens, or 4 of up to 32, share one 128-row tile.  The
  // score tile is then block-diagonal; the probabilities outside a row's own window are written as 0.
  a.G = 1; a.R = 128; a.Btot = (int)B;
  if (T <= 64 && B >= 2) {
    a.G = T <= 32 ? 4 : 2;
    a.R = 128 / a.G;
    a.Npad = 128;
  }
  a.tmem_cols = 32;
  while (a.tmem_cols < a.Npad) a.tmem_cols <<= 1;
  a.qk_m = p->qk_scale.mult; a.qk_s = clamp_shift(p->qk_scale.shift);
  a.pv_m = p->pv_scale.mult; a.pv_s = clamp_shift(p->pv_scale.shift);
  a.smax = p->smax;
  a.bias = p->attn_bias; a.bias_batches = p->attn_bias ? p->attn_bias_batches : 1;
  a.O = O;
  a.status = ctx->status_dev;
  const int64_t ldq = 3 * D;
  CUtensorMap tmQ, tmK, tmV;
  const CUtensorMapSwizzle vsw = d == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (d == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  // boxes: a.R rows of a.G consecutive images / windows (G = 1: 128 query rows, Npad key / value rows of one image)
  if (!make_tensor_map(ctx, &tmQ, QKV, d, T, h, B, ldq, d, T * ldq, 128, a.G > 1 ? a.R : 128, CU_TENSOR_MAP_SWIZZLE_128B, a.q_pos, a.G) ||
      !make_tensor_map(ctx, &tmK, QKV + D, d, T, h, B, ldq, d, T * ldq, 128, a.G > 1 ? a.R : a.Npad, CU_TENSOR_MAP_SWIZZLE_128B, a.k_pos, a.G) ||
      !make_tensor_map(ctx, &tmV, QKV + 2 * D, d, T, h, B, ldq, d, T * ldq, (int)d, a.G > 1 ? a.R : a.Npad, vsw, a.v_pos, a.G))
    return IVIT_ERR_UNSUPPORTED;
  const uint32_t v_off = 128 * 128 + a.Npad * 128;
  const uint32_t p_off = (v_off + a.Npad * a.d + 1023u) & ~1023u;
  const size_t smem = 1024 + p_off + (size_t)((a.Npad + 127) / 128) * 128 * 128 + 1024 + 2048 + 16 + 64 + 16;
  a.bh = (int)((B + a.G - 1) / a.G * h);
  a.items = a.bh * a.tiles_m;
  a.sched = ctx->sched_dev + 2 * ctx->attn_gen;
  a.sched_other = ctx->sched_dev + 2 * (ctx->attn_gen ^ 1);
  ctx->attn_gen ^= 1;
  const int64_t slots = 2 * (int64_t)ctx->sm_count;
  const int64_t grid = a.items < slots ? a.items : slots;
  LaunchScope ls(ctx, KIND_ATTENTION, 4.0 * (double)(B * h) * (double)T * (double)T * (double)d);
  const bool k8 = p->smax.k_out == 8;
  if (a.G > 1) {
    if (k8) launch_k(attention_kernel<true, true>, dim3((unsigned)grid), dim3(kAttnThreads), smem, ctx->stream, tmQ, tmK, tmV, a);
    else launch_k(attention_kernel<true, false>, dim3((unsigned)grid), dim3(kAttnThreads), smem, ctx->stream, tmQ, tmK, tmV, a);
  } else {
    if (k8) launch_k(attention_kernel<false, true>, dim3((unsigned)grid), dim3(kAttnThreads), smem, ctx->stream, tmQ, tmK, tmV, a);
    else launch_k(attention_kernel<false, false>, dim3((unsigned)grid), dim3(kAttnThreads), smem, ctx->stream, tmQ, tmK, tmV, a);
  }
  return ls.done();
}

}  // namespace ivit
