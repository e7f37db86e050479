// INT8 x INT8 -> INT32 GEMM on the sm_100a tensor cores with the dyadic requantisation of
// Sec. 3.2 fused into the epilogue.  Persistent and warp-specialised:
//
//   warp 0      TMA producer: streams the k-blocks of both operands of successive output tiles
//               through a ring of shared-memory stages (cp.async.bulk.tensor, hardware swizzle,
//               mbarrier transaction counts);
//   warp 1      owns tensor memory; one thread issues tcgen05.mma.kind::i8 (M = 128, N = BN,
//               K = 32 per instruction) into one of two accumulator buffers;
//   warps 2..17 epilogue (four per TMEM lane quarter): read the finished accumulator with tcgen05.ld (one
//               TMEM lane per thread), requantise, add the residual, saturate and store - while the tensor
//               core already works on the next tile in the other buffer.
//
// The 128 TMEM lanes of a tile hold the "P" operand's rows, the columns the "Q" operand's rows.
//   * Dense layers (per-channel scale / bias):  P = weight rows (output channels), Q = activation
//     rows.  A thread then owns ONE output channel: its multiplier, shift and bias stay in registers
//     for the whole tile (no shared-memory traffic per value).  A warp turns its 32 channels x 32 rows
//     into row-major bytes with 4x4 byte transposes (shuffles), stages them in a shared-memory slot
//     of its own and stores the slot with a TMA store of its own; the residual bytes of the same
//     32 x 32 piece arrive by TMA two chunks ahead.  No warp waits for another.
//   * Batched MatMul (per-tensor scale): P = rows of A, Q = rows of B (K-major, Q K^T) or B is
//     MN-major ([K, N] rows, P V; the V tile is consumed as stored, without a transpose).  A thread
//     owns one output row and stores 32 consecutive int8 values per chunk.
//
// One CTA per SM walks a contiguous range of tiles (channel blocks fastest, so that consecutive tiles
// share their activation rows; for short K those rows stay resident in shared memory).  Every
// device-side wait is bounded: when one runs out the thread records IVIT_ERR_DEVICE_TIMEOUT in the
// context's status word, carries on without further waits, drains its outstanding copies, and the
// CTA frees its tensor memory and returns.
#include "tc_ptx.cuh"
#include <cstring>
#include <new>
#include "rowops.cuh"

namespace ivit {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 4-D int8 tensor map over {inner, rows, batch_inner, batch_outer}.  The three outer dimensions are
// ordered by ascending byte stride (a head inside a token row has a smaller stride than the row);
// pos[0..2] receive the tensor-map dimension that holds the row, inner-batch and outer-batch
// coordinate.  Byte strides must be multiples of 16.
namespace {
struct TmapKey {
  const void* ptr;
  uint64_t dims[4], strides[3];
  uint32_t box[4];
  int64_t swz;   // (64 bits: the key has no padding, it is compared bytewise)
};
struct TmapSlot {
  TmapKey key;
  CUtensorMap map;
  bool used;
};
constexpr int kTmapSlots = 512;
}  // namespace

bool make_tensor_map(ivit_ctx* ctx, CUtensorMap* map, const int8_t* ptr, int64_t inner, int64_t rows, int64_t bi, int64_t bo,
              int64_t row_stride, int64_t si, int64_t so, int box_inner, int box_rows, CUtensorMapSwizzle swz,
              int pos[3], int box_bo) {
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || row_stride % 16) return false;
  struct Dim { int64_t size, stride; int box, which; };
  Dim d[3] = {{rows, row_stride, box_rows, 0}, {bi, si, 1, 1}, {bo, so, box_bo, 2}};
  // size-1 dimensions never contribute to an address: give them the largest stride so they sort last
  int64_t big = row_stride;
  for (int i = 1; i < 3; ++i)
    if (d[i].size > 1 && d[i].stride > big) big = d[i].stride;
  for (int i = 1; i < 3; ++i)
    if (d[i].size <= 1) d[i].stride = big;
  for (int i = 0; i < 3; ++i)
    for (int j = i + 1; j < 3; ++j)
      if (d[j].stride < d[i].stride) { Dim t = d[i]; d[i] = d[j]; d[j] = t; }
  cuuint64_t dims[4] = {(cuuint64_t)inner, 0, 0, 0}, strides[3];
  cuuint32_t box[4] = {(cuuint32_t)box_inner, 1, 1, 1};
  for (int i = 0; i < 3; ++i) {
    if (d[i].stride % 16 || d[i].stride <= 0 || d[i].stride >= (1ll << 40)) return false;
    dims[i + 1] = (cuuint64_t)d[i].size;
    strides[i] = (cuuint64_t)d[i].stride;
    box[i + 1] = (cuuint32_t)d[i].box;
    pos[d[i].which] = i + 1;
  }
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  // An encoded map depends on nothing but these values: a forward pass asks for the same few dozen maps again and
  // again, so they are kept (direct-mapped, the newer entry wins a slot).
  TmapKey key{};
  key.ptr = ptr;
  for (int i = 0; i < 4; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  for (int i = 0; i < 3; ++i) key.strides[i] = strides[i];
  key.swz = (int64_t)swz;
  if (!ctx->tmap_cache) ctx->tmap_cache = new (std::nothrow) TmapSlot[kTmapSlots]();
  TmapSlot* slot = nullptr;
  if (ctx->tmap_cache) {
    uint64_t h = reinterpret_cast<uintptr_t>(ptr) * 0x9E3779B97F4A7C15ull;
    h ^= (dims[1] + 31 * dims[2] + 131 * box[1] + 1031 * box[0] + 7 * (uint64_t)swz + 17 * strides[0]) * 0xC2B2AE3D27D4EB4Full;
    slot = static_cast<TmapSlot*>(ctx->tmap_cache) + (h >> 40) % kTmapSlots;
    if (slot->used && std::memcmp(&slot->key, &key, sizeof(key)) == 0) {
      *map = slot->map;
      return true;
    }
  }
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode);
  if (fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(ptr), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (slot) {
    slot->key = key;
    slot->map = *map;
    slot->used = true;
  }
  return true;
}

void tmap_cache_free(ivit_ctx* ctx) {
  delete[] static_cast<TmapSlot*>(ctx->tmap_cache);
  ctx->tmap_cache = nullptr;
}

namespace {

constexpr int BM = 128;          // TMEM lanes of a tile (UMMA M, cta_group::1)
constexpr int BK = 128;          // bytes (= int8 elements) of K per pipeline stage
constexpr int UMMA_K = 32;       // K of one tcgen05.mma.kind::i8
constexpr int kMaxStages = 8;
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kFirstEpiWarp = 2;   // warp 0: TMA loads, warp 1: MMA
constexpr int kThreads = 32 * kFirstEpiWarp + kEpiThreads;

struct TcArgs {
  GemmEpilogue epi;
  int P, Q, K;       // extents along TMEM lanes / TMEM columns / contraction (32-bit: the launcher checks the sizes)
  int64_t sCo, sCi;
  int batches_inner;
  int total_tiles;
  int tiles_each, tiles_extra;   // every CTA walks tiles_each tiles, tiles_extra CTAs one more: the first ones, or
  int long_last;                 // (long_last) the last ones, when the short tiles of a ragged last row block, which
                                 // end the tile order, can make up for the extra tile
  int tiles_p, tiles_q;
  int BN;            // columns of the tile (multiple of 32, <= 256)
  int stages;
  int tmem_cols;     // power of two >= 2 * BN (two accumulator buffers)
  int lanes_are_channels;  // 1: Dense orientation (lane = output channel, column = output row)
  int q_mn;          // 1: the Q operand tile is MN-major ([k, n] rows of q_row_bytes)
  int q_row_bytes;
  int q_stage_bytes;
  int p_pos[3], q_pos[3];  // tensor-map dimension (1..3) that holds the row / inner-batch / outer-batch coordinate
  int tma_out;       // Dense orientation, int8: the output tile is staged in shared memory and stored by TMA
  int tma_res;       // ... and the residual tile of the same shape is fetched by TMA into shared memory
  int pair;          // two CTAs (a cluster) per tile of 256 channels: cta_group::2 MMAs, each CTA loads its own 128
                     // weight rows and half of the activation rows; tiles_p then counts channel PAIRS of tiles
  int q_resident;    // Dense orientation, short K: all k-blocks of the Q (activation row) tile stay in shared
                     // memory while the CTA walks the channel blocks; only weight tiles stream through the ring
  RowOpArgs rop;     // row operator on finished blocks of output rows (Dense orientation, staged int8 output)
  int* status;
};


struct TileCoord {
  int batch;
  int bo, bi, p0, q0;
};

// Tiles are ordered p-block fastest and every CTA owns a contiguous range of them, so that the tiles a
// CTA works on in a row share their Q operand (the activation rows of a Dense layer).
__device__ __forceinline__ TileCoord tile_coord(const TcArgs& a, int t) {
  TileCoord c;
  const uint32_t per_batch = (uint32_t)a.tiles_p * (uint32_t)a.tiles_q;
  c.batch = (uint32_t)t < per_batch ? 0 : (int)((uint32_t)t / per_batch);     // a Dense layer is one batch
  const uint32_t t2 = (uint32_t)t - (uint32_t)c.batch * per_batch;
  c.q0 = (int)(t2 / (uint32_t)a.tiles_p) * a.BN;
  c.p0 = (int)(t2 % (uint32_t)a.tiles_p) * BM;
  c.bo = c.batch == 0 ? 0 : c.batch / a.batches_inner;
  c.bi = c.batch - c.bo * a.batches_inner;
  return c;
}

// Walks a contiguous range of tiles without divisions: p-block fastest, then q-block, then batch.
struct TileIter {
  int p, q, bi, bo;       // block indices
  int batch;
  int pstep, poff;        // lanes between consecutive p-blocks (two tiles when a CTA pair shares them) and this CTA's offset
  __device__ __forceinline__ void init(const TcArgs& a, int t, int poff_ = 0) {
    const TileCoord c = tile_coord(a, t);
    p = c.p0 / BM; q = c.q0 / a.BN; bi = c.bi; bo = c.bo; batch = c.batch;
    pstep = a.pair ? 2 * BM : BM;
    poff = poff_;
  }
  __device__ __forceinline__ void next(const TcArgs& a) {
    if (++p == a.tiles_p) {
      p = 0;
      if (++q == a.tiles_q) {
        q = 0;
        ++batch;
        if (++bi == a.batches_inner) { bi = 0; ++bo; }
      }
    }
  }
  __device__ __forceinline__ int p0() const { return p * pstep + poff; }
  __device__ __forceinline__ int q0(const TcArgs& a) const { return q * a.BN; }
};

// MODE fixes the run-time choices of the epilogue at compile time for the shapes of an encoder block, so that
// the per-chunk code carries no branches on kernel arguments: 0 = everything decided at run time (any
// orientation, output type and residual port), 1 = Dense orientation, int8 output staged for TMA stores, no
// residual, 2 = the same with the residual tile fetched by TMA, 3 = as 1 with an activation table applied to the
// saturated value (the element-wise ShiftGELU variant inside FC1).
// ROP != 0 (MODE 1 or 2 only): a row operator on the output, run by this same kernel: 1 = I-LayerNorm into a second
// tensor (the input of the next Dense layer), 2 = ShiftGELU in place (Algorithm 2 with its row maximum).  Both need
// whole output rows, i.e. every channel tile of a block of rows, and those tiles may belong to several CTAs.  So
// every epilogue warp, once its stores of a row block are complete, adds its tiles to the block's arrival counter;
// the warp that completes the count raises the block's ready flag.  The rows are cut into slices (one batch of the
// row routine each) that are dealt to all epilogue warps of the grid in a fixed order; a warp works on its slices
// after its CTA's last tile, straight out of L2, waiting (bounded) only for the ready flag of the slice's block.
// The last CTA to finish leaves counters and flags at zero for the next launch.
template <int MODE, int ROP, bool PAIR = false>
__global__ void __launch_bounds__(kThreads, 1) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmP,
                                                              const __grid_constant__ CUtensorMap tmQ,
                                                              const __grid_constant__ CUtensorMap tmO,
                                                              const __grid_constant__ CUtensorMap tmR, TcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve: [stages x (P tile | Q tile)] [barriers] [tmem address, issued count]
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t stage_bytes = BM * BK + (a.q_resident ? 0 : a.q_stage_bytes);
  const int kblocks = (a.K + BK - 1) / BK;
  const uint32_t qres_bytes = a.q_resident ? kblocks * a.q_stage_bytes : 0;
  const uint32_t qres = base + a.stages * stage_bytes;         // resident Q tile: kblocks x [BN rows x 128 B]
  const uint32_t stage_out = qres + qres_bytes;                // output slots: 2 x [32 rows][32 channels] int8 per epilogue warp
  const uint32_t stage_res = stage_out + (a.tma_out ? kEpiWarps * 2048 : 0);   // residual slots, same layout
  const uint32_t bars_off = a.stages * stage_bytes + qres_bytes + (a.tma_out ? kEpiWarps * 2048 : 0) + (a.tma_res ? kEpiWarps * 2048 : 0);
  const uint32_t full0 = base + bars_off, empty0 = full0 + 8 * kMaxStages;
  const uint32_t accf0 = empty0 + 8 * kMaxStages, acce0 = accf0 + 16, resf = acce0 + 16, qrese = resf + 16 * kEpiWarps;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + bars_off + 8 * (2 * kMaxStages + 5 + 2 * kEpiWarps));
  volatile int* issued_slot = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // residual port: the requantised value of every int8 residual byte (256 entries, built below), followed by the
  // 256 entries of the optional activation table
  int8_t* res_tab = reinterpret_cast<int8_t*>(tmem_slot) + 32;
  volatile uint32_t* rop_flag = tmem_slot + 2;                                // row operator: a flag the CTA agrees on
  uint8_t* rop_smem = gen_base + bars_off + 1024;   // ROP == 1: LayerNorm constants; ROP == 2: table rows, per warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's (with PAIR: this CTA pair's) contiguous range of tiles
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;      // PAIR: 0 = the CTA that issues the MMAs of the pair
  const int poff = (int)rank * BM;                          // this CTA's 128 channels inside the pair's 256
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int first_long = a.long_last ? workers - a.tiles_extra : 0;   // first worker with one tile more
  const int n_long = worker - first_long;                              // long workers before this one
  const int t_begin = worker * a.tiles_each + min(max(n_long, 0), a.tiles_extra);
  const int t_end = t_begin + a.tiles_each + ((n_long >= 0 && n_long < a.tiles_extra) ? 1 : 0);

  // set-up, spread over the epilogue threads: one barrier (or descriptor prefetch) each
  {
    const int i = (int)threadIdx.x - 64;
    if (i >= 0 && i < kMaxStages) {
      mbar_init(full0 + 8 * i, 1);
    } else if (i < 2 * kMaxStages) {
      mbar_init(empty0 + 8 * (i - kMaxStages), 1);
    } else if (i < 2 * kMaxStages + 2) {
      mbar_init(accf0 + 8 * (i - 2 * kMaxStages), 1);
    } else if (i < 2 * kMaxStages + 4) {
      mbar_init(acce0 + 8 * (i - 2 * kMaxStages - 2), PAIR ? 2 * kEpiWarps : kEpiWarps);   // PAIR: both CTAs' warps
    } else if (i < 2 * kMaxStages + 4 + 2 * kEpiWarps) {
      mbar_init(resf + 8 * (i - 2 * kMaxStages - 4), 1);   // residual slots: 2 per epilogue warp
    } else if (i == 2 * kMaxStages + 4 + 2 * kEpiWarps) {
      mbar_init(qrese, 1);
      *issued_slot = 0;
      *rop_flag = 1u;
    } else if (i == 2 * kMaxStages + 5 + 2 * kEpiWarps) {
      prefetch_tmap(&tmP);
    } else if (i == 2 * kMaxStages + 6 + 2 * kEpiWarps) {
      prefetch_tmap(&tmQ);
    } else if (i == 2 * kMaxStages + 7 + 2 * kEpiWarps) {
      if (a.tma_out) prefetch_tmap(&tmO);
    } else if (i == 2 * kMaxStages + 8 + 2 * kEpiWarps) {
      if (a.tma_res) prefetch_tmap(&tmR);
    }
    if (i >= 0 && i < 2 * kMaxStages + 5 + 2 * kEpiWarps) {
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    if (i >= 0 && i < 256 && a.epi.res) res_tab[i] = (int8_t)rq(i - 128, a.epi.res_scale.mult, clamp_shift(a.epi.res_scale.shift));
  }
  if (warp == 1) {
    if (PAIR) tmem_alloc_pair(smem_u32(tmem_slot), (uint32_t)a.tmem_cols);
    else tmem_alloc(smem_u32(tmem_slot), (uint32_t)a.tmem_cols);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the other CTA's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done (barriers, tensor memory, descriptor prefetch): let the next kernel be scheduled, then wait
  // for the previous kernel's results before touching global memory
  pdl_trigger();
  if (ROP == 1 && warp >= kFirstEpiWarp) {
    // I-LayerNorm constants of all channels into shared memory: parameters, read before the wait for the previous
    // kernel.  The form (fast / general, see LnConsts) is agreed on by all epilogue threads.
    const int et0 = (int)threadIdx.x - 32 * kFirstEpiWarp, nwords = a.P >> 2;
    int4* sm_m = reinterpret_cast<int4*>(rop_smem);
    if (!ln_stage_consts(a.rop.gs, a.rop.beta, nwords, a.rop.vec, sm_m, sm_m + nwords, sm_m + 2 * nwords, et0, kEpiThreads))
      atomicAnd(const_cast<uint32_t*>(rop_flag), 0u);
    asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
    if (*rop_flag) ln_fold_consts(nwords, sm_m + nwords, sm_m + 2 * nwords, et0, kEpiThreads);
    asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
  }
  if (warp != 0) pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0;            // k-blocks issued so far, over all tiles of this CTA
      int s = 0, wrap = 0;       // ring slot of the next k-block and how often the ring has wrapped
      bool ok = true;
      int pit = 0, qi = 0, cur_q = -1;
      TileIter ti;
      ti.init(a, t_begin, poff);
      // which tensor-map coordinate (1..3) carries the row / inner batch / outer batch index
      const int pr = a.p_pos[0], pbi = a.p_pos[1], qr = a.q_pos[0], qbi = a.q_pos[1];
      // PAIR: both CTAs load (their 128 weight rows, their half of the activation rows); the bytes of both are
      // counted by the stage barrier of CTA rank 0, which alone arms it
      auto arm = [&](uint32_t bar, uint32_t bytes) {
        if (!PAIR) mbar_expect_tx(bar, bytes);
        else if (rank == 0) mbar_expect_tx(bar, 2u * bytes);
      };
      auto load = [&](uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
        if (PAIR) tma_load_4d_pair(dst, map, mapa_rank0(bar), c0, c1, c2, c3);
        else tma_load_4d(dst, map, bar, c0, c1, c2, c3);
      };
      // Dense orientation: the P operand is the weight matrix, which no kernel writes.  The weight k-blocks of the
      // first tile are requested before the wait for the previous kernel (whose last CTAs may still be running
      // elsewhere); the activation k-blocks that complete the same stage barriers follow after the wait.
      int pre = 0;
      if (a.lanes_are_channels && t_begin < t_end) {
        pre = kblocks < a.stages ? kblocks : a.stages;
        for (int kb = 0; kb < pre; ++kb) {
          arm(full0 + 8 * kb, BM * BK + a.q_stage_bytes);
          load(base + kb * stage_bytes, &tmP, full0 + 8 * kb, kb * BK, pr == 1 ? ti.p0() : 0, pr == 2 ? ti.p0() : 0,
               pr == 3 ? ti.p0() : 0);
        }
      }
      pdl_wait();
      for (int t = t_begin; ok && t < t_end; ++t, ++pit, ti.next(a)) {
        const int p0 = ti.p0(), q0 = ti.q0(a) + (PAIR ? (int)rank * (a.BN >> 1) : 0);   // PAIR: this CTA's half of the rows
        const int pc1 = pr == 1 ? p0 : (pbi == 1 ? ti.bi : ti.bo), pc2 = pr == 2 ? p0 : (pbi == 2 ? ti.bi : ti.bo),
                  pc3 = pr == 3 ? p0 : (pbi == 3 ? ti.bi : ti.bo);
        bool bring_q = false;
        if (a.q_resident && q0 != cur_q) {
          // new activation row block: its k-blocks come in beside this tile's weight k-blocks, once every MMA
          // on the old block is done
          if (qi > 0 && !mbar_wait(qrese, (qi - 1) & 1, a.status)) { ok = false; break; }
          bring_q = true;
          cur_q = q0;
          ++qi;
        }
        for (int kb = 0; kb < kblocks; ++kb) {
          if (wrap > 0 && !mbar_wait(empty0 + 8 * s, (wrap & 1) ^ 1, a.status)) { ok = false; break; }
          const uint32_t sp = base + s * stage_bytes, sq = sp + BM * BK;
          const bool early = t == t_begin && kb < pre;   // barrier armed and weights requested before the wait
          if (!early) arm(full0 + 8 * s, stage_bytes + (bring_q ? a.q_stage_bytes : 0));
          if (bring_q)
            load(qres + kb * a.q_stage_bytes, &tmQ, full0 + 8 * s, kb * BK, qr == 1 ? q0 : 0, qr == 2 ? q0 : 0,
                 qr == 3 ? q0 : 0);
          if (!early) load(sp, &tmP, full0 + 8 * s, kb * BK, pc1, pc2, pc3);
          if (!a.q_resident) {
            const int qrow = a.q_mn ? kb * BK : q0;     // MN-major: rows of the map are k, the inner index is n
            const int qc0 = a.q_mn ? q0 : kb * BK;
            load(sq, &tmQ, full0 + 8 * s, qc0, qr == 1 ? qrow : (qbi == 1 ? ti.bi : ti.bo),
                 qr == 2 ? qrow : (qbi == 2 ? ti.bi : ti.bo), qr == 3 ? qrow : (qbi == 3 ? ti.bi : ti.bo));
          }
          *issued_slot = ++issued;
          if (++s == a.stages) { s = 0; ++wrap; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && rank == 0) {   // PAIR: CTA rank 0 issues for both CTAs
      // instruction descriptor: D = S32, A = B = signed 8 bit, A K-major, M = 128 (PAIR: 256 over both CTAs), N = BN,
      // no saturation
      const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a.q_mn << 16) |
                             ((uint32_t)(a.BN >> 3) << 17) | ((uint32_t)((PAIR ? 2 * BM : BM) >> 4) << 24);
      // P descriptors: K-major rows of 128 bytes (128B swizzle, 1024 bytes per 8 rows).  Q: the same,
      // or MN-major rows of q_row_bytes (swizzle = row width, 8 rows per group).  Along K a descriptor
      // advances by 32 bytes (K-major) or 32 rows (MN-major): an add on the low word.
      const uint32_t p_hi = desc_hi(1024, 2);
      const uint32_t q_hi = !a.q_mn ? desc_hi(1024, 2)
                                    : desc_hi(8u * a.q_row_bytes, a.q_row_bytes == 128 ? 2u : (a.q_row_bytes == 64 ? 4u : 6u));
      const uint32_t q_kstep16 = (!a.q_mn ? UMMA_K : UMMA_K * a.q_row_bytes) >> 4;
      const int k_tail = (int)(a.K - (int64_t)(kblocks - 1) * BK);            // bytes of K in the last k-block
      const int tail_steps = k_tail >= BK ? BK / UMMA_K : (k_tail + UMMA_K - 1) / UMMA_K;
      // descriptor low words: the start-address field counts 16-byte units, so stages and k-blocks are plain adds
      const uint32_t p_lo0 = desc_lo(base, 16), q_lo0 = desc_lo(qres, 16);
      const uint32_t stage16 = stage_bytes >> 4, qstage16 = (uint32_t)a.q_stage_bytes >> 4;
      int consumed = 0, s = 0, wrap = 0, it = 0;
      bool ok = true;
      int cur_q = -1;
      TileIter ti;
      ti.init(a, t_begin, poff);
      for (int t = t_begin; ok && t < t_end; ++t, ++it) {
        const int buf = it & 1;
        bool last_of_q = false;
        if (a.q_resident) {
          // a new activation row block arrives k-block by k-block on the stage barriers of this tile
          cur_q = ti.q0(a);
          ti.next(a);
          last_of_q = t + 1 >= t_end || ti.q0(a) != cur_q;
        }
        // the epilogue must have drained this buffer (its use two tiles ago)
        if (it >= 2 && !mbar_wait(acce0 + 8 * buf, ((it >> 1) & 1) ^ 1, a.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full0 + 8 * s, wrap & 1, a.status)) { ok = false; break; }
          tc_fence_after();
          // low descriptor words of this stage's P tile and of the Q tile (resident, or behind P in the stage)
          const uint32_t p_lo = p_lo0 + (uint32_t)s * stage16;
          const uint32_t q_lo = a.q_resident ? q_lo0 + (uint32_t)kb * qstage16 : p_lo + ((BM * BK) >> 4);
          if (kb != kblocks - 1 || tail_steps == BK / UMMA_K) {
            if (PAIR) umma_i8_x4_pair(d_tmem, p_lo, p_hi, q_lo, q_hi, idesc, kb != 0, UMMA_K >> 4, q_kstep16);
            else umma_i8_x4(d_tmem, p_lo, p_hi, q_lo, q_hi, idesc, kb != 0, UMMA_K >> 4, q_kstep16);
          } else {
            uint32_t pl = p_lo, ql = q_lo;
            for (int k = 0; k < tail_steps; ++k) {
              if (PAIR) umma_i8_pair(d_tmem, pl, p_hi, ql, q_hi, idesc, (kb | k) != 0);
              else umma_i8_lohi(d_tmem, pl, p_hi, ql, q_hi, idesc, (kb | k) != 0);
              pl += UMMA_K >> 4;
              ql += q_kstep16;
            }
          }
          // the stage may be refilled once these MMAs have read it (PAIR: in both CTAs)
          if (PAIR) umma_commit_pair(empty0 + 8 * s);
          else umma_commit(empty0 + 8 * s);
          ++consumed;
          if (++s == a.stages) { s = 0; ++wrap; }
        }
        if (ok) {   // accumulator of this tile complete (PAIR: told to the epilogue warps of both CTAs)
          if (PAIR) umma_commit_pair(accf0 + 8 * buf);
          else umma_commit(accf0 + 8 * buf);
        }
        if (ok && last_of_q) umma_commit(qrese);   // the resident tile may be replaced once these MMAs are done
      }
      if (!ok) {
        // drain: copies that were issued but never consumed (only after a timeout)
        const int issued = *issued_slot;
        for (int j = consumed; j < issued; ++j) {
          mbar_wait(full0 + 8 * s, wrap & 1, a.status);
          if (++s == a.stages) { s = 0; ++wrap; }
        }
      }
    }
  } else {
    // ---------------- epilogue warps; TMEM lane quarter = warp % 4, 32-column chunks dealt round-robin ----------------
    // The groups of four warps ("parts") work independently.  A wait that times out is recorded and the
    // warp carries on without further waits (its results are then meaningless and the status word says so).
    const int et = threadIdx.x - 32 * kFirstEpiWarp;
    const int ew = warp - kFirstEpiWarp;
    const int qd = warp & 3;
    const int part = ew >> 2;
    constexpr int kParts = kEpiWarps / 4;
    static_assert((kParts & (kParts - 1)) == 0, "chunk rotation");
    const GemmEpilogue& e = a.epi;
    const bool dense = MODE ? true : a.lanes_are_channels != 0;
    const bool tma_out = MODE ? true : a.tma_out != 0;
    const bool tma_res = MODE ? MODE == 2 : a.tma_res != 0;   // MODE 3 = MODE 1 + activation table
    const bool ldg_res = MODE ? false : (e.res != nullptr && !a.tma_res);
    const bool out_i32 = MODE ? false : e.out_dtype == IVIT_I32;
    const int8_t* res_tab0 = res_tab + 128;   // entry of residual byte 0
    const int8_t* act_tab0 = res_tab + 256 + 128;   // entry of value 0 of the activation table
    const bool act = MODE == 3 ? true : (MODE ? false : e.act_table != nullptr);
    constexpr bool kFrag = MODE == 1 || MODE == 3;
    if (act) {
      // the table may come from an earlier kernel of the stream: read it after the dependency wait above
      if (et < 256) res_tab[256 + et] = e.act_table[et];
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
    }
    bool ok = true;

    // Dense orientation: constants of this thread's channel; fetched one tile ahead
    int nm = 1, ns = 32, nb = 0;
    auto fetch_channel = [&](int p0) {
      const int c = p0 + qd * 32 + lane;
      nm = 1; ns = 32; nb = 0;
      if (c < a.P) {
        nm = e.scale.m(c);
        ns = e.scale.s(c);
        if (e.bias) nb = __ldg(e.bias + c);
      }
    };
    // the first tile's coordinates, computed once (they cost integer divisions)
    TileIter ti_first;
    ti_first.init(a, t_begin, poff);
    if (dense && t_begin < t_end) fetch_channel(ti_first.p0());
    // MatMul orientation: one per-tensor constant set
    const int um = e.scale.mult, us = clamp_shift(e.scale.shift);
    const long long uc = 1ll << (us - 1);

    // Staged output (and residual input) of the Dense orientation: every warp owns two slots of
    // [32 rows][32 channels] bytes for each direction and needs no other warp to move them.  Its lane 0 stores a
    // filled output slot by TMA (a box of 32 channels x 32 rows) and fetches the residual bytes two chunks
    // ahead of the arithmetic into the slot whose bytes have just been used.
    const uint32_t my_out = stage_out + (uint32_t)ew * 2048u, my_res = stage_res + (uint32_t)ew * 2048u;
    const uint32_t my_resf = resf + 16u * (uint32_t)ew;
    const int c_first = qd * 32;        // first channel of this warp inside the tile
    uint32_t g = 0;                     // chunks this warp has worked on
    uint32_t rpar = 0, rpend = 0;       // per residual slot (bit 0 / 1): parity of its next arrival; a fetch in flight
    // Chunks are dealt to the parts round-robin ACROSS tiles (chunk j of a tile goes to part (rot + j) % kParts,
    // rot = chunks of this CTA's earlier tiles), so that a tile whose chunk count is no multiple of kParts
    // does not leave the same part idle every time.
    // The warp's chunk sequence two chunks ahead (residual fetches):
    TileIter pf_ti;
    int pf_t = t_begin;
    int pf_ck = part;
    int pf_rot = 0;
    uint32_t pf_g = 0;
    auto pf_settle = [&]() {
      while (pf_t < t_end) {
        const int left = a.Q - pf_ti.q0(a);
        const int nck = ((left < a.BN ? left : a.BN) + 31) >> 5;
        if (pf_ck < nck) break;
        pf_ti.next(a);
        ++pf_t;
        pf_rot = (pf_rot + nck) & (kParts - 1);
        pf_ck = (part - pf_rot) & (kParts - 1);
      }
    };
    // residual bytes of the next chunk of the look-ahead into slot pf_g & 1 (a box wholly past the last channel
    // is not fetched: the arithmetic does not wait for it either)
    auto pf_fetch = [&]() {
      if (pf_t < t_end) {
        if (pf_ti.p0() + c_first < a.P) {
          const uint32_t sl = pf_g & 1u;
          if (lane == 0) {
            mbar_expect_tx(my_resf + 8u * sl, 1024u);
            tma_load_4d(my_res + 1024u * sl, &tmR, my_resf + 8u * sl, pf_ti.p0() + c_first, pf_ti.q0(a) + 32 * pf_ck, 0, 0);
          }
          rpend |= 1u << sl;
        }
        ++pf_g;
        pf_ck += kParts;
        pf_settle();
      }
    };
    if (tma_res && t_begin < t_end) {
      pf_ti = ti_first;
      pf_settle();
      pf_fetch();
      pf_fetch();
    }

    int it = 0;
    int rot = 0;          // chunks of this CTA's earlier tiles, modulo kParts
    int tiles_in_q = 0;   // ROP: tiles of the current block of output rows that this CTA has finished
    TileIter ti = ti_first;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      TileCoord tc;
      tc.batch = ti.batch; tc.bo = ti.bo; tc.bi = ti.bi; tc.p0 = ti.p0(); tc.q0 = ti.q0(a);
      ti.next(a);   // ti now describes the next tile
      const int buf = it & 1;
      const int cm = nm, cs = ns;
      const long long cc = (long long)nb * nm + (1ll << (ns - 1));   // bias * m + 2^(s-1)
      const bool hi_ok = __all_sync(0xffffffffu, cs >= 32);    // the usual case: the shift is past the low word
      // ... and when the rounding constant is past it too and acc + bias cannot leave 32 bits (|acc| <= 2^30
      // since K <= 65536), only the high word of (acc + bias) * m is needed
      const int cbias = nb;
      const bool hi_only = __all_sync(0xffffffffu, cs >= 33 && nb > -(1 << 30) && nb < (1 << 30));
      const int rnd_hi = cs >= 33 ? 1 << (cs - 33) : 0;
      // The kernels without a residual port (MODE 1, 3) read the accumulators as fragments (tmem_ld_frag16): thread l
      // then works on the four channels (l >> 2) + 8 j of its warp, whose constants it takes from the lanes that
      // fetched them.  (With the residual port the fragment form is slower: its byte look-ups lose more to bank
      // conflicts than the transposes cost.)
      int km[4], ks[4], kb[4];
      if (kFrag) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int src = (lane >> 2) + 8 * j;
          km[j] = __shfl_sync(0xffffffffu, cm, src);
          ks[j] = __shfl_sync(0xffffffffu, cs, src);
          kb[j] = __shfl_sync(0xffffffffu, cbias, src);
        }
      }
      if (dense && t + 1 < t_end) fetch_channel(ti.p0());

      if (ok) ok = mbar_wait(accf0 + 8 * buf, (it >> 1) & 1, a.status);
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(buf * a.BN);
      const int cols_left = a.Q - tc.q0;
      const int nck = ((cols_left < a.BN ? cols_left : a.BN) + 31) >> 5;   // chunks that hold output

      if (dense) {
        // lane = output channel c, TMEM column = output row
        const int c = tc.p0 + qd * 32 + lane;
        const bool c_ok = c < a.P;
        const int sh_lo = min(cs, 32), sh_hi = max(cs - 32, 0);
        const int li = lane & 3;
        const uint32_t sel1 = (li & 1) ? 0x3715u : 0x6240u;
        const uint32_t sel2 = (li & 2) ? 0x3276u : 0x5410u;
        const int cb = qd * 32 + lane;          // channel within the tile

        // One chunk = 32 output rows x this warp's 32 channels, worked through in two halves of 16 rows to keep
        // the register footprint small: the SM holds four epilogue warps per scheduler, and it is their number
        // that hides the latencies of the shuffles, the shared-memory traffic and the barrier operations.
        auto half = [&](int (&v)[16], int ck, int h, uint8_t* pe) {
          const int j0 = ck * 32 + h * 16;
          const int r0 = tc.q0 + j0;
          const int nrow = min(16, a.Q - r0);
          if (hi_only) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = mad_hi(v[j] + cbias, cm, rnd_hi) >> sh_hi;
          } else if (hi_ok) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = mad_wide_hi(v[j], cm, cc) >> sh_hi;
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const long long tt = mad_wide(v[j], cm, cc);
              v[j] = (int)__funnelshift_rc((unsigned)tt, (unsigned)(tt >> 32), sh_lo) >> sh_hi;
            }
          }
          // residual port
          if (tma_res) {
            // residual bytes of this chunk in shared memory: [row][32 channels]
            const uint8_t* rt = gen_base + (my_res - base) + (g & 1u) * 1024 + h * 512 + lane;
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += (int)res_tab0[(int)*reinterpret_cast<const int8_t*>(rt + j * 32)];
          } else if (ldg_res) {
            int64_t rr = (int64_t)((uint64_t)r0 % (uint64_t)e.res_rows);
#pragma unroll
            for (int g = 0; g < 16; g += 8) {
              int xr[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                xr[j] = (c_ok && g + j < nrow) ? (int)__ldg(e.res + rr * e.ldres + c) : 0;
                if (++rr == e.res_rows) rr = 0;
              }
#pragma unroll
              for (int j = 0; j < 8; ++j) v[g + j] += (int)res_tab0[xr[j]];
            }
          }
          if (out_i32) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (j < nrow && c_ok) reinterpret_cast<int32_t*>(e.out)[(int64_t)(r0 + j) * e.ldo + c] = v[j];
            return;
          }
          if (act) {
            // element-wise activation of the saturated value (the static-maximum ShiftGELU variant)
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = (int)act_tab0[max(-128, min(127, v[j]))];
          }
          // int8: pack four rows per word, transpose 4x4 bytes inside each group of four lanes so that a lane
          // ends up with four consecutive channels of one row, then store 4 bytes per lane and word
          uint32_t w[4], o[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) w[k] = pack_sat8(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
#pragma unroll
          for (int k = 0; k < 4; ++k) o[k] = __shfl_xor_sync(0xffffffffu, w[k], 1);
#pragma unroll
          for (int k = 0; k < 4; ++k) w[k] = __byte_perm(w[k], o[k], sel1);
#pragma unroll
          for (int k = 0; k < 4; ++k) o[k] = __shfl_xor_sync(0xffffffffu, w[k], 2);
#pragma unroll
          for (int k = 0; k < 4; ++k) w[k] = __byte_perm(w[k], o[k], sel2);
          if (tma_out) {
            // word k belongs to slot row 16h + li + 4k: rows of 32 bytes, one bank per lane
#pragma unroll
            for (int k = 0; k < 4; ++k) *reinterpret_cast<uint32_t*>(pe + 512 * h + 128 * k) = w[k];
          } else {
            // direct stores (grouped output rows): this lane's first word is row r0 + li, then + 4 per word
            int64_t row = (int64_t)r0 + li, ro = row, grem = 0;
            if (e.group_rows > 0) {
              grem = (int64_t)((uint64_t)row % (uint64_t)e.group_rows);
              ro = (int64_t)((uint64_t)row / (uint64_t)e.group_rows) * e.group_stride + grem;
            }
            const int cbase = tc.p0 + qd * 32 + (lane & ~3);
            const bool cg_ok = cbase < a.P;   // P % 4 == 0: a group of four channels is valid as a whole
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (cg_ok && 4 * k + li < nrow)
                *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(e.out) + ro * e.ldo + cbase) = w[k];
              ro += 4;
              if (e.group_rows > 0) {
                grem += 4;
                while (grem >= e.group_rows) { grem -= e.group_rows; ro += e.group_stride - e.group_rows; }
              }
            }
          }
        };

        const bool c_any = tc.p0 + c_first < a.P;   // else the warp's box lies wholly past the last channel
        for (int ck = (part - rot) & (kParts - 1); ck < nck; ck += kParts) {
          uint8_t* pe = nullptr;
          if (tma_out) {
            const uint32_t sl = g & 1u;
            // the store that used this slot two chunks ago must have read it; the residual bytes must be here
            if (lane == 0) tma_store_wait_read1();
            if (tma_res && c_any) {
              if (ok) ok = mbar_wait(my_resf + 8u * sl, (rpar >> sl) & 1u, a.status);
              if (ok) { rpar ^= 1u << sl; rpend &= ~(1u << sl); }
            }
            __syncwarp();
            // after the transposes a lane holds 4 consecutive channels (lane >> 2) of slot row li + 4k
            pe = gen_base + (my_out - base) + sl * 1024 + li * 32 + (lane >> 2) * 4;
          }
          if constexpr (kFrag) {
            // fragment form: 16 channels x 32 rows per step; the packed words are the fragment that one stmatrix
            // stores transposed, i.e. as rows of 16 consecutive channels, into the [32 rows][32 channels] slot
            const uint32_t out_slot = my_out + 1024u * (g & 1u) + (uint32_t)lane * 32u;
            const uint8_t* res_slot = gen_base + (my_res - base) + (g & 1u) * 1024 + (2 * (lane & 3)) * 32 + (lane >> 2);
            // both halves are requested before the arithmetic on the first begins
            int vv[32];
            tmem_ld_frag16_issue<0>(t_row + (uint32_t)(32 * ck), vv);
            tmem_ld_frag16_issue<16>(t_row + (16u << 16) + (uint32_t)(32 * ck), vv);
            tmem_ld_wait(vv);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              int (&v)[16] = *reinterpret_cast<int (*)[16]>(&vv[16 * h]);
#pragma unroll
              for (int u = 0; u < 2; ++u) {       // u = 0: channel (l >> 2) + 16 h, u = 1: eight channels on
                const int m = km[2 * h + u], sft = ks[2 * h + u], bia = kb[2 * h + u];
                if (hi_only) {
                  const int add = 1 << (sft - 33), sh = sft - 32;
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    v[4 * i + 2 * u] = mad_hi(v[4 * i + 2 * u] + bia, m, add) >> sh;
                    v[4 * i + 2 * u + 1] = mad_hi(v[4 * i + 2 * u + 1] + bia, m, add) >> sh;
                  }
                } else {
                  const long long c64 = (long long)bia * m + (1ll << (sft - 1));
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    v[4 * i + 2 * u] = (int)(mad_wide(v[4 * i + 2 * u], m, c64) >> sft);
                    v[4 * i + 2 * u + 1] = (int)(mad_wide(v[4 * i + 2 * u + 1], m, c64) >> sft);
                  }
                }
              }
              if (tma_res) {
                // residual bytes [row][32 channels]: rows 8 i + 2 (l & 3) + {0, 1}, channels 16 h + (l >> 2) + {0, 8}
                const uint8_t* rt = res_slot + 16 * h;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  v[4 * i] += (int)res_tab0[(int)*reinterpret_cast<const int8_t*>(rt + i * 256)];
                  v[4 * i + 1] += (int)res_tab0[(int)*reinterpret_cast<const int8_t*>(rt + i * 256 + 32)];
                  v[4 * i + 2] += (int)res_tab0[(int)*reinterpret_cast<const int8_t*>(rt + i * 256 + 8)];
                  v[4 * i + 3] += (int)res_tab0[(int)*reinterpret_cast<const int8_t*>(rt + i * 256 + 40)];
                }
              }
              if (act) {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = (int)act_tab0[max(-128, min(127, v[j]))];
              }
              uint32_t w[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) w[i] = pack_sat8(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
              stmatrix_x4_trans_b8(out_slot + 16u * (uint32_t)h, w[0], w[1], w[2], w[3]);
            }
          } else {
            int v[16];
            tmem_ld16(t_row + (uint32_t)(32 * ck), v);
            half(v, ck, 0, pe);
            tmem_ld16(t_row + (uint32_t)(32 * ck + 16), v);
            half(v, ck, 1, pe);
          }
          if (tma_out) {
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && c_any) tma_store_4d(&tmO, my_out + 1024u * (g & 1u), tc.p0 + c_first, tc.q0 + 32 * ck, 0, 0);
            // every lane is past its reads of this slot's residual bytes: fetch those of two chunks on
            if (tma_res) pf_fetch();
            ++g;
          }
        }
      } else {
        // lane = output row, TMEM column = output column
        const int r = tc.p0 + qd * 32 + lane;
        const bool row_ok = r < a.P;
        const int64_t out_row = tc.bo * a.sCo + tc.bi * a.sCi + (int64_t)r * e.ldo;
        const int32_t* bias_row = e.bias32 ? e.bias32 + ((tc.batch % e.bias_batches) * (int64_t)a.P + r) * e.ldbias : nullptr;
        for (int ck = (part - rot) & (kParts - 1); ck < nck; ck += kParts) {
          const int j0 = ck * 32;
          const int c0 = tc.q0 + j0;
          int v[32];
          tmem_ld32(t_row + (uint32_t)j0, v);
          if (!row_ok) continue;
          const int ncol = min(32, a.Q - c0);
          if (bias_row) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (j < ncol) v[j] += __ldg(bias_row + c0 + j);
          }
          if (us >= 33) {   // the usual case: high product word plus 2^(s-33), shifted by s - 32
            const int u_rnd = 1 << (us - 33), u_sh = us - 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = mad_hi(v[j], um, u_rnd) >> u_sh;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (int)(((long long)v[j] * um + uc) >> us);
          }
          int8_t* o = reinterpret_cast<int8_t*>(e.out) + out_row + c0;
          if (ncol == 32) {
            int4 w0, w1;
            w0.x = (int)pack_sat8(v[0], v[1], v[2], v[3]);     w0.y = (int)pack_sat8(v[4], v[5], v[6], v[7]);
            w0.z = (int)pack_sat8(v[8], v[9], v[10], v[11]);   w0.w = (int)pack_sat8(v[12], v[13], v[14], v[15]);
            w1.x = (int)pack_sat8(v[16], v[17], v[18], v[19]); w1.y = (int)pack_sat8(v[20], v[21], v[22], v[23]);
            w1.z = (int)pack_sat8(v[24], v[25], v[26], v[27]); w1.w = (int)pack_sat8(v[28], v[29], v[30], v[31]);
            reinterpret_cast<int4*>(o)[0] = w0;
            reinterpret_cast<int4*>(o)[1] = w1;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (j < ncol) o[j] = (int8_t)sat8(v[j]);
          }
        }
      }
      rot = (rot + nck) & (kParts - 1);
      // this warp has read everything it needs from the buffer: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(mapa_rank0(acce0 + 8 * buf));   // the issuing CTA waits for both CTAs' warps
        else mbar_arrive(acce0 + 8 * buf);
      }
      if (ROP) {
        ++tiles_in_q;
        if (t + 1 >= t_end || ti.q0(a) != tc.q0) {
          // this warp's last tile of the row block: see the stores complete, release them, count the tiles
          if (lane == 0) {
            unsigned* q_state = a.rop.counters;
            const unsigned qblk = (unsigned)tc.q0 / (unsigned)a.BN;
            tma_store_wait_all();
            asm volatile("fence.proxy.async;" ::: "memory");
            __threadfence();
            unsigned* cnt = q_state + 32 + qblk * kRowStateStride;
            const unsigned old = atomicAdd(cnt, (unsigned)tiles_in_q);
            if (old + (unsigned)tiles_in_q == (unsigned)(a.tiles_p * kEpiWarps)) {
              *cnt = 0u;
              __threadfence();
              asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(cnt + kRowCounters * kRowStateStride), "r"(1u) : "memory");
            }
          }
          tiles_in_q = 0;
        }
      }
    }
    if (ROP && ok) {
      // ---- row operator on this warp's slices ----
      unsigned* q_state = a.rop.counters;
      constexpr int kSlice = ROP == 1 ? 8 : 2;                       // rows of a slice: one batch of the row routine
      const unsigned spb = (unsigned)(a.BN + kSlice - 1) / kSlice;   // slices per row block
      const unsigned total = (unsigned)a.tiles_q * spb;
      const unsigned nwarps = gridDim.x * kEpiWarps;
      const int C = a.P;
      const int nwords = C >> 2;
      const int4* sm_m = reinterpret_cast<const int4*>(rop_smem);
      const LnConsts lk{sm_m, sm_m + nwords, sm_m + 2 * nwords, *rop_flag != 0u};
      unsigned* tab = reinterpret_cast<unsigned*>(rop_smem) + ew * (kGeluTailRows * 64);
      for (unsigned sl = (unsigned)ew * gridDim.x + blockIdx.x; sl < total; sl += nwarps) {
        const unsigned blk = sl / spb, j = sl - blk * spb;
        const int q0 = (int)blk * a.BN;
        const int left = a.Q - q0;
        const int in_blk = left < a.BN ? left : a.BN;
        const int r0 = (int)j * kSlice;
        if (r0 >= in_blk) continue;
        unsigned rdy = 0;
        if (lane == 0) {
          // polls back off: thousands of warps may wait for a handful of flags
          const unsigned* flag = q_state + 32 + (kRowCounters + blk) * kRowStateStride;
          unsigned pause = 64;
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(rdy) : "l"(flag) : "memory");
            if (rdy) break;
            __nanosleep(pause);
            if (pause < 2048) pause <<= 1;
          }
          if (!rdy) {
            *reinterpret_cast<volatile int*>(a.status) = IVIT_ERR_DEVICE_TIMEOUT;
            __threadfence_system();
          }
        }
        rdy = __shfl_sync(0xffffffffu, rdy, 0);
        if (!rdy) break;
        const int nrows = in_blk - r0 < kSlice ? in_blk - r0 : kSlice;
        int8_t* rows0 = reinterpret_cast<int8_t*>(e.out) + (int64_t)(q0 + r0) * e.ldo;
        if (ROP == 1) {
          int8_t* dst = a.rop.ln_out + (int64_t)(q0 + r0) * a.rop.ld_ln;
          if (C <= 384) {
            layernorm_rows<3, 8, true>(rows0, e.ldo, nrows, C, a.rop.M_ln, a.rop.mean_magic, lk, dst, a.rop.ld_ln, lane);
          } else if (C <= 512) {
            layernorm_rows<4, 8, true>(rows0, e.ldo, nrows, C, a.rop.M_ln, a.rop.mean_magic, lk, dst, a.rop.ld_ln, lane);
          } else {
            for (int h = 0; h < nrows; h += 4)
              layernorm_rows<8, 4, true>(rows0 + (int64_t)h * e.ldo, e.ldo, nrows - h < 4 ? nrows - h : 4, C, a.rop.M_ln,
                                         a.rop.mean_magic, lk, dst + (int64_t)h * a.rop.ld_ln, a.rop.ld_ln, lane);
          }
        } else {
          if (C <= 1536) {
            shiftgelu_rows<3, 2, true>(rows0, e.ldo, nrows, C, a.rop.table, tab, rows0, e.ldo, lane);
          } else {
            for (int h = 0; h < nrows; ++h) {
              shiftgelu_rows<8, 1, true>(rows0 + (int64_t)h * e.ldo, e.ldo, 1, C, a.rop.table, tab, rows0 + (int64_t)h * e.ldo,
                                         e.ldo, lane);
              __syncwarp();
            }
          }
          __syncwarp();
        }
      }
    }
    if (tma_out && lane == 0) tma_store_wait_all();
    // only after a timeout: residual bytes fetched for chunks that were never worked on may be in flight
    if (tma_res && !ok && lane == 0)
      for (uint32_t sl = 0; sl < 2; ++sl)
        if ((rpend >> sl) & 1u) mbar_wait(my_resf + 8u * sl, (rpar >> sl) & 1u, a.status);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still use it
  if (warp == 1) {
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)a.tmem_cols);
    else tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
  }
  if (ROP) {
    // the last CTA to get here finds every other CTA out of the queue: it leaves the queue state at zero
    unsigned* q_state = a.rop.counters;
    if (threadIdx.x == 0) {
      __threadfence();
      *rop_flag = atomicAdd(q_state + 2, 1u) == gridDim.x - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (*rop_flag) {
      for (int i = threadIdx.x; i < a.tiles_q; i += kThreads) q_state[32 + (kRowCounters + i) * kRowStateStride] = 0u;
      if (threadIdx.x == 0) q_state[2] = 0u;
      __threadfence();
    }
  }
}

// ---- host side ------------------------------------------------------------------------------

int pow2_at_least(int v) {
  int p = 32;
  while (p < v) p <<= 1;
  return p;
}

constexpr size_t kSmemBudget = 227 * 1024;
constexpr int64_t kPairMinK = 1024;   // contraction length from which a CTA pair per tile pays (measured)
// alignment slack + one KB of barriers, tensor-memory slot, flags and the two 256-entry tables of the residual /
// activation port; a row operator's shared memory follows it
constexpr size_t kSmemFixed = 1024 + 1024;
static_assert(8 * (2 * kMaxStages + 5 + 2 * kEpiWarps) + 32 + 512 <= 1024, "barrier block");


// Tile width along the TMEM columns: the candidate with the least (rounds of tiles per CTA) x (time of a tile).
// Model of a tile's time: the larger of its operand traffic, (128 + bn) x K bytes at about 60 bytes per clock into
// an SM's shared memory, and its epilogue, which grows with the tile's width now that chunks are dealt to the
// epilogue parts across tiles, plus a fixed cost per tile.  The constants are fitted to measured launch times of the
// DeiT-S / ViT-B / ViT-L layer shapes at widths 128 ... 256 (the pick is within 4 % of the best width on each).
int pick_bn(int64_t extent, int64_t tiles_other, int64_t K, int sm_count, bool single_batch) {
  if (extent <= 256) return (int)((extent + 31) / 32 * 32);
  int best = 0;
  double best_cost = 0;
  for (int bn : {256, 224, 192, 160, 128}) {
    const int64_t tiles = tiles_other * ((extent + bn - 1) / bn);
    double rounds = (double)((tiles + sm_count - 1) / sm_count);
    // a ragged last block of at most half a tile: if every CTA that needs an extra tile gets one of its short tiles
    // (long_last in the launcher), the extra tile costs about half a round
    const int64_t ragged = extent % bn, extra = tiles % sm_count, each = tiles / sm_count;
    // (only from two full rounds on: measured inside an encoder block, a launch of one round and a half
    // of wide tiles loses to two rounds of narrow ones although it wins when timed alone)
    if (single_batch && each >= 2 && ragged != 0 && ragged <= bn / 2 && extra != 0 && (extra - 1) * (each + 1) < tiles_other) rounds -= 0.5;
    const double feed = (double)K * (128.0 + bn) / 60.0;
    const double epilogue = 8.0 * bn;
    // ties go to the narrower tile (its MMAs, loads and stores are shorter): the loop runs from wide to narrow
    const double cost = rounds * ((feed > epilogue ? feed : epilogue) + 900.0);
    if (!best || cost <= best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

}  // namespace

// The shared-memory limit of a kernel is a per-device attribute: set for the current device at context creation.
int gemm_tc_prepare_device() {
  if (cudaFuncSetAttribute(gemm_tc_kernel<0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<3, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<1, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel<2, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess)
    return IVIT_ERR_CUDA;
  return IVIT_OK;
}

int launch_gemm_tc(ivit_ctx* ctx, const GemmProblem& g) {
  if (!ctx->tmap_encode) return IVIT_ERR_UNSUPPORTED;
  const int64_t batches = g.batches_outer * g.batches_inner;
  if (batches == 0 || g.M == 0 || g.N == 0) return IVIT_OK;
  if (g.M > 2147483647LL - 512 || g.N > 2147483647LL - 512 || g.K > 65536 || batches > 2147483647LL) return IVIT_ERR_UNSUPPORTED;
  const GemmEpilogue& e = g.epi;
  if (g.lda % 16 || g.ldb % 16 || g.sAo % 16 || g.sAi % 16 || g.sBo % 16 || g.sBi % 16) return IVIT_ERR_UNSUPPORTED;

  TcArgs a{};
  a.epi = e;
  a.K = (int)g.K; a.sCo = g.sCo; a.sCi = g.sCi; a.batches_inner = (int)g.batches_inner;
  a.status = ctx->status_dev;
  CUtensorMap tmP, tmQ;
  const bool dense = g.transB && batches == 1 && !e.bias32;
  if (dense) {
    if (g.N % 4 || e.ldo % 4 || (reinterpret_cast<uintptr_t>(e.out) & 3)) return IVIT_ERR_UNSUPPORTED;
    // Dense orientation: lanes = output channels (rows of W), columns = output rows (rows of A)
    a.lanes_are_channels = 1;
    a.P = (int)g.N; a.Q = (int)g.M;
    a.tiles_p = (int)((a.P + BM - 1) / BM);
    // Long contractions are bound by the operand feed from L2 and by the issuing thread's loop: a pair of CTAs per
    // tile of 256 channels (cta_group::2) halves the activation bytes per SM and the MMAs issued per SM.  Taken
    // when the layer has whole pairs of channel tiles and the epilogue is one of the specialised forms.
    a.pair = (ctx->gemm_pairs && g.K >= kPairMinK && g.N % (2 * BM) == 0 && ctx->sm_count % 2 == 0 &&
              (g.N / (2 * BM)) * ((g.M + 255) / 256) >= ctx->sm_count / 2 &&   // a pair-tile for every pair of SMs
             
              e.out_dtype == IVIT_I8 && e.group_rows <= 0 && !(reinterpret_cast<uintptr_t>(e.out) & 15) && e.ldo % 16 == 0 &&
              (!e.res || (e.res_rows >= g.M && !(reinterpret_cast<uintptr_t>(e.res) & 15) && e.ldres % 16 == 0)) &&
              !e.act_table && !(e.rop.kind && ctx->row_fusion)) ? 1 : 0;
    if (a.pair) {
      a.tiles_p = (int)(g.N / (2 * BM));   // pairs of channel tiles
      a.BN = 256;
      a.q_stage_bytes = (a.BN / 2) * BK;   // every CTA of a pair loads half of the activation rows
    } else {
      a.BN = pick_bn(a.Q, a.tiles_p, g.K, ctx->sm_count, batches == 1);
      a.q_stage_bytes = a.BN * BK;
    }
    if (!make_tensor_map(ctx, &tmP, g.B, g.K, g.N, 1, 1, g.ldb, 0, 0, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B, a.p_pos) ||
        !make_tensor_map(ctx, &tmQ, g.A, g.K, g.M, 1, 1, g.lda, 0, 0, BK, a.pair ? a.BN / 2 : a.BN, CU_TENSOR_MAP_SWIZZLE_128B,
                         a.q_pos))
      return IVIT_ERR_UNSUPPORTED;
  } else {
    // MatMul orientation: lanes = rows of A; the epilogue's 16-byte stores need aligned output rows
    if (e.out_dtype != IVIT_I8 || e.bias || e.res || e.scale.mult_c || e.group_rows > 0 || e.act_table) return IVIT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(e.out) & 15) || e.ldo % 16 || g.sCo % 16 || g.sCi % 16) return IVIT_ERR_UNSUPPORTED;
    a.P = (int)g.M; a.Q = (int)g.N;
    a.tiles_p = (int)((a.P + BM - 1) / BM);
    a.q_mn = g.transB ? 0 : 1;
    if (!make_tensor_map(ctx, &tmP, g.A, g.K, g.M, g.batches_inner, g.batches_outer, g.lda, g.sAi, g.sAo, BK, BM,
                  CU_TENSOR_MAP_SWIZZLE_128B, a.p_pos))
      return IVIT_ERR_UNSUPPORTED;
    if (a.q_mn) {
      // the whole N extent is one tile whose k rows are N bytes wide: 32, 64 or 128
      if (g.N != 32 && g.N != 64 && g.N != 128) return IVIT_ERR_UNSUPPORTED;
      a.BN = (int)g.N;
      a.q_row_bytes = (int)g.N;
      a.q_stage_bytes = BK * a.q_row_bytes;
      const CUtensorMapSwizzle swz = a.q_row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                     : (a.q_row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
      if (!make_tensor_map(ctx, &tmQ, g.B, g.N, g.K, g.batches_inner, g.batches_outer, g.ldb, g.sBi, g.sBo, a.q_row_bytes, BK,
                    swz, a.q_pos))
        return IVIT_ERR_UNSUPPORTED;
    } else {
      a.BN = pick_bn(a.Q, (int64_t)a.tiles_p * batches, g.K, ctx->sm_count, false);
      a.q_stage_bytes = a.BN * BK;
      if (!make_tensor_map(ctx, &tmQ, g.B, g.K, g.N, g.batches_inner, g.batches_outer, g.ldb, g.sBi, g.sBo, BK, a.BN,
                    CU_TENSOR_MAP_SWIZZLE_128B, a.q_pos))
        return IVIT_ERR_UNSUPPORTED;
    }
  }
  CUtensorMap tmO = tmP;
  if (dense && e.out_dtype == IVIT_I8 && e.group_rows <= 0 && !(reinterpret_cast<uintptr_t>(e.out) & 15) && e.ldo % 16 == 0) {
    int opos[3];
    a.tma_out = make_tensor_map(ctx, &tmO, reinterpret_cast<const int8_t*>(e.out), g.N, g.M, 1, 1, e.ldo, 0, 0, 32, 32,
                         CU_TENSOR_MAP_SWIZZLE_NONE, opos) ? 1 : 0;
  }
  CUtensorMap tmR = tmP;
  if (a.tma_out && e.res && e.res_rows >= g.M && !(reinterpret_cast<uintptr_t>(e.res) & 15) && e.ldres % 16 == 0) {
    int rpos[3];
    a.tma_res = make_tensor_map(ctx, &tmR, e.res, g.N, g.M, 1, 1, e.ldres, 0, 0, 32, 32, CU_TENSOR_MAP_SWIZZLE_NONE,
                                rpos) ? 1 : 0;
  }
  // The row operator runs in this kernel when the epilogue is one of the specialised forms (staged int8 output,
  // residual absent or fetched by TMA), the rows fit the tail routines and there is a counter per row block.
  int rop = 0;
  if (e.rop.kind && a.lanes_are_channels && a.tma_out && (!e.res || a.tma_res) && !e.act_table && ctx->row_fusion) {
    const int64_t blocks_q = (a.Q + a.BN - 1) / a.BN;
    if (blocks_q <= kRowCounters && e.rop.kind == 1 && g.N <= 1024 && (ctx->row_fusion & 1)) rop = 1;
    if (blocks_q <= kRowCounters && e.rop.kind == 2 && g.N % 16 == 0 && g.N <= 4096 && !e.res && (ctx->row_fusion & 2)) rop = 2;
  }
  a.rop = e.rop;
  a.rop.kind = rop;
  a.rop.counters = ctx->rowblk_dev;
  a.rop.mean_magic = (unsigned)(0x100000000ull / (unsigned long long)(2 * g.N)) + 1u;
  a.rop.vec = e.rop.gs.mult_c && e.rop.gs.shift_c && !(reinterpret_cast<uintptr_t>(e.rop.gs.mult_c) & 15) &&
              !(reinterpret_cast<uintptr_t>(e.rop.gs.shift_c) & 3) && !(reinterpret_cast<uintptr_t>(e.rop.beta) & 15);
  const size_t rop_bytes = rop == 1 ? ((size_t)g.N * 12 + 1023) / 1024 * 1024 : (rop == 2 ? (size_t)kGeluTailSmem : 0);
  const size_t out_stage = (a.tma_out ? (size_t)kEpiWarps * 2048 : 0) + (a.tma_res ? (size_t)kEpiWarps * 2048 : 0);
  // short K: keep the activation tile resident if that still leaves four weight stages
  const size_t kblocks = (size_t)((g.K + BK - 1) / BK);
  const size_t qres_bytes = kblocks * a.q_stage_bytes;
  a.q_resident = (dense && !a.pair && kSmemFixed + rop_bytes + out_stage + qres_bytes + 4 * (size_t)BM * BK <= kSmemBudget) ? 1 : 0;
  const size_t stage = (size_t)BM * BK + (a.q_resident ? 0 : a.q_stage_bytes);
  const size_t fixed = out_stage + (a.q_resident ? qres_bytes : 0);
  int stages = (int)((kSmemBudget - kSmemFixed - rop_bytes - fixed) / stage);
  a.stages = stages > kMaxStages ? kMaxStages : stages;
  if (a.stages < 2) return IVIT_ERR_UNSUPPORTED;
  a.tmem_cols = pow2_at_least(2 * a.BN);
  a.tiles_q = (int)((a.Q + a.BN - 1) / a.BN);
  const int64_t total_tiles = (int64_t)a.tiles_p * a.tiles_q * batches;
  if (total_tiles > 2147483647LL) return IVIT_ERR_UNSUPPORTED;
  a.total_tiles = (int)total_tiles;

  const size_t smem = kSmemFixed + rop_bytes + (size_t)a.stages * stage + fixed;
  const int workers_max = a.pair ? ctx->sm_count / 2 : ctx->sm_count;   // CTAs, or CTA pairs
  const int workers = a.total_tiles < workers_max ? a.total_tiles : workers_max;
  const unsigned grid = (unsigned)(a.pair ? 2 * workers : workers);
  a.tiles_each = a.total_tiles / workers;
  a.tiles_extra = a.total_tiles % workers;
  // ... which needs a short tile in the range of every long CTA
  a.long_last = (a.Q % a.BN != 0 && a.Q % a.BN <= a.BN / 2 && batches == 1 && a.tiles_extra > 0 &&
                 (int64_t)(a.tiles_extra - 1) * (a.tiles_each + 1) < a.tiles_p) ? 1 : 0;
  LaunchScope ls(ctx, KIND_GEMM_TC, 2.0 * (double)batches * (double)g.M * (double)g.N * (double)g.K);
  // the encoder block's Dense layers take the specialised instantiations
  int mode = (a.lanes_are_channels && a.tma_out && (!e.res || a.tma_res)) ? (a.tma_res ? 2 : 1) : 0;
  if (e.act_table) mode = mode == 1 ? 3 : 0;
  if (a.pair && (mode != 1 && mode != 2)) return IVIT_ERR_UNSUPPORTED;   // (the conditions above imply mode 1 or 2)
  if (a.pair) ++ctx->pair_launches;
  if (a.pair && mode == 2) launch_k_pair(gemm_tc_kernel<2, 0, true>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (a.pair) launch_k_pair(gemm_tc_kernel<1, 0, true>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (rop == 1 && mode == 2) launch_k(gemm_tc_kernel<2, 1>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (rop == 1 && mode == 1) launch_k(gemm_tc_kernel<1, 1>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (rop == 2 && mode == 1) launch_k(gemm_tc_kernel<1, 2>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (mode == 3) launch_k(gemm_tc_kernel<3, 0>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (mode == 2) launch_k(gemm_tc_kernel<2, 0>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else if (mode == 1) launch_k(gemm_tc_kernel<1, 0>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  else launch_k(gemm_tc_kernel<0, 0>, dim3(grid), dim3(kThreads), smem, ctx->stream, tmP, tmQ, tmO, tmR, a);
  ctx->rowop_fused = (rop != 0 && (mode == 1 || mode == 2)) ? 1 : 0;
  return ls.done();
}

}  // namespace ivit
