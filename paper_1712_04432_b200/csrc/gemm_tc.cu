// Dense bf16 contraction on the 5th-generation tensor cores (tcgen05) for the three
// products of a layer: forward Y = W X, backward-data dX = W^T dY, backward-weight
// dW = dY X^T (Section 1 of the paper), with the K range optionally cut into the
// partial sums a P_r x P_c grid would form (Appendix A.2).
//
// One persistent CTA per SM, 320 threads, warp-specialised:
//   warp 0      TMA producer: operand tiles -> 128B-swizzled shared-memory ring
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma (128 x BN x 16 per
//               instruction, fp32 accumulator in TMEM) and commits to mbarriers
//   warps 2..9  epilogue: tcgen05.ld the accumulator (lane = row; each warp owns 32 rows and
//               half of the columns), apply the epilogue operation and store; operands the
//               operation reads are prefetched under the MMAs; two accumulators alternate so
//               the epilogue of one tile runs under the MMAs of the next
// Transposed operands are not copied: an operand whose contiguous dimension is M or N is
// loaded as 64-wide column chunks and described to the MMA as "MN-major".
// Tile shapes: 128 x 128, 128 x 256, 256 x 256 per CTA, or 256 x 256 per CTA pair
// (cta_group::2); tc_gemm_prepare picks one per contraction with a small cost model.  With a
// bf16 result on 128-row tiles the epilogue moves all its global data by TMA through per-warp
// staging boxes.  Tuning knobs (environment): MBD_TC_MH, MBD_TC_BN, MBD_TC_PAIR, MBD_TC_GROUP_M, MBD_TC_DEBUG, MBD_TC_X_POW2, MBD_TC_NO_TE_RING,
// MBD_TC_NO_TE.
// Every mbarrier wait is bounded; on time-out the kernel records a code and leaves.
#include <stdio.h>
#include <stdlib.h>

#include "epi.cuh"
#include "tc_common.cuh"

namespace mbd {

namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row
constexpr int NUM_THREADS = 320;      // TMA warp, MMA warp, 8 epilogue warps
// Dynamic shared memory of every instantiation: seven 32 KB stages (or any of the other rings),
// nothing more.  With the kernel's static variables (padded to 1 KB by the alignment of the ring)
// and the 1 KB the system keeps per CTA, that leaves 2 KB of an SM's 228 KB: CTAs of kernels that
// use no shared memory (a reduction, a column sum on the side stream) can be resident next to a
// GEMM CTA.  The ring must start on a 1024-byte boundary (128B swizzle); the declaration asks for
// that, and the kernel checks it and gives up cleanly otherwise.
constexpr int SMEM_DYN_BYTES = 224 * 1024;
constexpr int RING_MAX_BYTES = SMEM_DYN_BYTES;

// ---- CTA-pair (cta_group::2) helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {   // same variable in CTA `rank` of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load issued by either CTA of a pair; the transaction bytes are counted on `bar`, which may
// live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}

struct Params {
  int M, N, K;
  int tiles_m, tiles_n, kb_total, S, group_m;
  float* partials;
  Epi epi;
  int* status;
  int te;                 // epilogue moves its global data with TMA through shared memory
  int te_prefetch;        // TMA epilogue requests its boxes one tile ahead
  int te_ring;            // every CTA has one work unit: the epilogue's staging boxes lie in the operand ring, which is idle by then
  int fix;                // running sum: piece s adds its accumulator to the sum pieces 0..s-1 left in `partials`
                          // (1: the pieces of a raster group follow one another; 2: all tiles piece by piece)
  int* flags;             // fix: one word per (tile, CTA of the pair, 128-row half, epilogue warp); zero between launches
  int join;               // > 1: a tile's `join` K pieces are accumulators of their own in tensor memory, added in the epilogue
  ConvShift cv;           // cv.mode != 0: operand tiles are shifted views (see ConvShift)
};

struct Work {
  int tm, tn, s, kb0, kb1;
};

// Joined pieces: r (piece 0's 32 columns of this lane's row) += the same columns of pieces 1 .. join-1, in
// ascending order, each from the accumulator `stride` TMEM columns further on.
__device__ __forceinline__ void add_joined_pieces(uint32_t taddr, int join, int stride, uint32_t* r) {
  for (int s = 1; s < join; ++s) {
#pragma unroll
    for (int o = 0; o < 32; o += 8) {          // eight columns at a time: the caller's registers are nearly all taken
      uint32_t t[8];
      tc::tc_ld8(taddr + s * stride + o, t);
      tc::tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 8; ++i) r[o + i] = __float_as_uint(__uint_as_float(r[o + i]) + __uint_as_float(t[i]));
    }
  }
}

template <int FIX>
__device__ __forceinline__ Work decode_work(const Params& p, int w) {
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int per_group = p.group_m * p.tiles_n;
  Work o;
  if (FIX == 1 && p.fix == 1) {
    // Running sum: the pieces of a raster group follow one another (all tiles of the group for piece 0,
    // then for piece 1, ...), so that piece s of a tile finds the sum of pieces 0..s-1 still in L2 and
    // the unit it depends on always has a smaller index than itself.
    const int span = per_group * p.S;
    int g = w / span;
    const int full = p.tiles_m / p.group_m;
    if (g > full) g = full;                    // the last, shorter group
    const int first_m = g * p.group_m;
    const int gsize = min(p.tiles_m - first_m, p.group_m);
    const int gtiles = gsize * p.tiles_n;
    int r = w - g * span;
    o.s = r / gtiles;
    r -= o.s * gtiles;
    o.tm = first_m + r % gsize;
    o.tn = r / gsize;
  } else {
    o.s = w / num_tiles;
    const int t = w - o.s * num_tiles;
    const int g = t / per_group;
    const int first_m = g * p.group_m;
    const int gsize = min(p.tiles_m - first_m, p.group_m);
    const int r = t - g * per_group;
    o.tm = first_m + r % gsize;
    o.tn = r / gsize;
  }
  o.kb0 = static_cast<int>((static_cast<long long>(o.s) * p.kb_total) / p.S);
  o.kb1 = static_cast<int>((static_cast<long long>(o.s + 1) * p.kb_total) / p.S);
  return o;
}

// Running-sum hand-over between the pieces of one tile (different CTAs, same launch): the warp that wrote
// its part of the sum publishes `value` with release semantics; the warp of the next piece that owns the
// same rows and columns waits for it (bounded, like every wait here) before it reads them.
__device__ __forceinline__ void flag_publish(int* flag, int value) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(value) : "memory");
}
__device__ __forceinline__ int flag_read(const int* flag) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
  return v;
}
static __device__ __noinline__ bool flag_wait(const int* flag, int value, volatile int* abort_flag, int* status) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (flag_read(flag) == value) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
      *abort_flag = 1;
      atomicCAS(status, 0, DEV_TIMEOUT_RUNNING_SUM);
      return false;
    }
    __nanosleep(200);
  }
}

// MH = number of 128-row halves of the CTA tile (1: 128 x BN, 2: 256 x BN).  The 256-row tile
// issues two MMAs per k-step against the same B tile, which cuts the shared-memory fill per
// flop by a third (64 instead of 96 bytes per clock at BN = 256); with BN = 256 it fills all of
// TMEM, so the epilogue of a tile no longer overlaps the next tile's MMAs.
//
// PAIR = 1: two CTAs of a cluster work on one 256 x BN tile with cta_group::2 MMAs issued by the
// even CTA.  Each CTA loads its own 128 rows of A and its own half of the B tile (the tensor core
// reads both halves), keeps its 128 rows of the accumulator in its own TMEM and runs its own
// epilogue: 64 B/clk of operand fill like the 256 x 256 tile, but with two accumulators (the
// epilogue overlaps the next tile), 32 KB stages and the TMA epilogue.
// FIX = 1: the instantiation that can add a product's K pieces as a running sum in its epilogue (CTA pairs only).
// FIX = 2: the instantiation that keeps a tile's K pieces as accumulators of their own in tensor memory (p.join).
// Both are kept apart so that the FIX = 0 instantiations compile to the code they had (a run-time branch in the
// shared epilogue cost 3 - 4 % of a cfg2 / cfg3 step).
template <int A_MN, int B_MN, int BN, int MH, int PAIR, int FIX>
// 136 registers per thread at most (a few bytes of spill in three instantiations): the register file
// is split over the SM's four sub-partitions, the busiest of which holds three of this CTA's ten
// warps; at 136 registers it keeps room for two warps of a side-stream kernel (a reduction, a
// column sum), whose CTAs could not be placed on the SM otherwise.
__global__ void __maxnreg__(136)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmAux, const Params p) {
  constexpr int BMT = BM * MH;                                // rows owned by this CTA
  constexpr int TILE_M = BMT * (PAIR ? 2 : 1);                // rows of the (pair's) tile
  constexpr int BNL = PAIR ? BN / 2 : BN;                     // B rows (tile columns) loaded by this CTA
  constexpr int A_BYTES = BMT * BK * 2;
  constexpr int B_BYTES = BNL * BK * 2;
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int STAGES = RING_MAX_BYTES / STAGE_BYTES;
  // TMA epilogue (128-row tiles only): every epilogue warp owns BN/128 staging boxes of
  // [32 rows][64 columns] bf16 (4 KB, 128B-swizzled) behind a shorter ring.
  constexpr int TE_BOXES = BN / 128;
  constexpr int TE_BYTES = 8 * TE_BOXES * 4096;
  constexpr int STAGES_TE = (RING_MAX_BYTES - TE_BYTES) / STAGE_BYTES;
  // fp32 planes by TMA (p.te == 2): two boxes of [32 rows][32 columns] fp32 per epilogue warp
  constexpr int STAGES_TEP = (RING_MAX_BYTES - 8 * 2 * 4096) / STAGE_BYTES;
  constexpr int ACC_COLS = MH * BN;                           // TMEM columns of one tile
  constexpr int ACC_BUFS = ACC_COLS * 2 <= 512 ? 2 : 1;
  constexpr int TMEM_COLS = ACC_COLS * ACC_BUFS;
  constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(A_MN) << 15) | (uint32_t(B_MN) << 16) |
                             (uint32_t(BN >> 3) << 17) | (uint32_t((PAIR ? 2 * BM : BM) >> 4) << 24);

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ __align__(8) uint64_t te_bar[16];        // TMA epilogue: one per epilogue warp and staging box
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  // 1024-byte alignment of the ring (needed by the 128B swizzle pattern)
  const uint32_t ring = smem_u32(smem_raw);
  if (ring & 1023u) {                      // same answer in every CTA: all of them leave before any barrier exists
    if (threadIdx.x == 0) atomicCAS(p.status, 0, DEV_SMEM_MISALIGNED);
    return;
  }
  const bool te = FIX != 1 && MH == 1 && p.te != 0;
  // Joined pieces (p.join = 2 or 4): the K range of a tile is cut into p.join pieces, each accumulated in TMEM
  // columns of its own; the epilogue adds them in ascending order -- the sum the reduction kernel would form over
  // p.join planes, without the planes.  The accumulators of one tile then take p.join * ACC_COLS columns.
  constexpr bool JOIN = FIX == 2 && ACC_COLS <= 256;           // (a tile that fills tensor memory has no room for a second piece)
  const int join = JOIN ? p.join : 1;
  const int acc_stride = join * ACC_COLS;
  const int acc_bufs = JOIN && join > 1 ? (2 * acc_stride <= 512 ? 2 : 1) : ACC_BUFS;
  const int tmem_cols = JOIN && join > 1 ? 512 : TMEM_COLS;
  // One work unit per CTA (p.te_ring): nothing is loaded after the unit's last k-block, so the staging boxes of the
  // TMA epilogue take the ring's first bytes once the accumulator is complete and the ring keeps all its stages.
  const bool te_ring = te && p.te_ring != 0;
  const int stages = te && !te_ring ? (p.te == 2 ? STAGES_TEP : STAGES_TE) : STAGES;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;        // 0 = the CTA that issues the MMAs
  const int w_first = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int w_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&tmem_full_bar[i]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[i]), PAIR ? 16 : 8);
    }
    for (int i = 0; i < 16; ++i) mbar_init(smem_u32(&te_bar[i]), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                   "r"(tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                   "r"(tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();            // both CTAs' barriers exist before anything remote touches them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  // Set-up is done: the kernel after this one may be scheduled; and from here on this one touches
  // global memory, so whatever ran before it must have finished.
  pdl_trigger();
  pdl_wait();

  const int total_work = p.tiles_m * p.tiles_n * p.S;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step) {
        const Work wk = decode_work<FIX>(p, w);
        const int row0 = wk.tm * TILE_M + static_cast<int>(rank) * BMT;       // this CTA's rows of A
        const int col0 = wk.tn * BN + static_cast<int>(rank) * BNL;           // this CTA's part of the B tile
        for (int kb = wk.kb0; kb < wk.kb1; ++kb) {
          ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abortp, p.status, DEV_TIMEOUT_PRODUCER);
          if (!ok) break;
          const uint32_t sa = ring + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          // pair: the bytes of both CTAs are counted on the full barrier of CTA 0, which expects them
          const uint32_t fb = PAIR ? map_to_cta(smem_u32(&full_bar[stage]), 0) : smem_u32(&full_bar[stage]);
          if (!PAIR) mbar_expect_tx(fb, STAGE_BYTES);
          else if (rank == 0) mbar_expect_tx(smem_u32(&full_bar[stage]), 2 * STAGE_BYTES);
          auto load = [&](uint32_t dst, const CUtensorMap* tm, int x, int y) {
            if (PAIR) tma_load_2d_pair(dst, tm, x, y, fb);
            else tma_load_2d(dst, tm, x, y, fb);
          };
          if (p.cv.mode == 0) {
            if (A_MN == 0) {
              load(sa, &tmA, kb * BK, row0);
            } else {
#pragma unroll
              for (int c = 0; c < BMT / 64; ++c) load(sa + c * (64 * BK * 2), &tmA, row0 + c * 64, kb * BK);
            }
            if (B_MN == 0) {
              load(sb, &tmB, kb * BK, col0);
            } else {
#pragma unroll
              for (int c = 0; c < BNL / 64; ++c) load(sb + c * (64 * BK * 2), &tmB, col0 + c * 64, kb * BK);
            }
          } else if (A_MN == 0) {
            // convolution, forward (B K-major) or backward-data (B MN-major): k-block = (tap, 64-channel block)
            int t, cb;
            if (p.cv.chan_major) { cb = kb / p.cv.taps; t = kb - cb * p.cv.taps; }
            else { t = kb / p.cv.blocks; cb = kb - t * p.cv.blocks; }
            load(sa, &tmA, cb * 64, B_MN == 0 ? row0 + p.cv.off[t] : row0 - p.cv.off[t]);
            if (B_MN == 0) {
              load(sb, &tmB, kb * BK, col0);
            } else {
#pragma unroll
              for (int c = 0; c < BNL / 64; ++c) load(sb + c * (64 * BK * 2), &tmB, p.cv.tap[t] * p.cv.Cp + col0 + c * 64, cb * 64);
            }
          } else {
            // convolution, backward-weight: K = pixels; an output column chunk = (tap, 64 input channels)
#pragma unroll
            for (int c = 0; c < BMT / 64; ++c) load(sa + c * (64 * BK * 2), &tmA, row0 + c * 64, kb * BK);
#pragma unroll
            for (int c = 0; c < BNL / 64; ++c) {
              const int n0 = col0 + c * 64;
              int t = n0 / p.cv.Cp;
              if (t >= p.cv.taps) t = p.cv.taps - 1;        // columns beyond N: loaded from somewhere valid, never stored
              load(sb + c * (64 * BK * 2), &tmB, n0 - t * p.cv.Cp, kb * BK + p.cv.off[t]);
            }
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
        const Work wk = decode_work<FIX>(p, w);
        const int acc = it % acc_bufs;
        const uint32_t acc_phase = (it / acc_bufs) & 1u;
        ok = mbar_wait(smem_u32(&tmem_empty_bar[acc]), acc_phase ^ 1u, abortp, p.status, DEV_TIMEOUT_MMA_TMEM);
        if (!ok) break;
        tc_fence_after();
        uint32_t d_tmem = tmem_base + acc * acc_stride;
        int piece = 0, piece_kb0 = wk.kb0;                 // joined pieces: the balanced ranges of the K blocks
        for (int kb = wk.kb0; kb < wk.kb1; ++kb) {
          if (JOIN && join > 1 && kb == static_cast<int>((static_cast<long long>(piece + 1) * p.kb_total) / join)) {
            ++piece;
            piece_kb0 = kb;
            d_tmem += ACC_COLS;
          }
          ok = mbar_wait(smem_u32(&full_bar[stage]), phase, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = ring + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const uint64_t adesc = A_MN ? make_desc(sa, 64 * BK * 2, 1024) : make_desc(sa, 16, 1024);
          const uint64_t bdesc = B_MN ? make_desc(sb, 64 * BK * 2, 1024) : make_desc(sb, 16, 1024);
          constexpr uint64_t A_STEP = (A_MN ? (UMMA_K * 128) : (UMMA_K * 2)) >> 4;
          constexpr uint64_t B_STEP = (B_MN ? (UMMA_K * 128) : (UMMA_K * 2)) >> 4;
          constexpr uint64_t A_HALF = (128 * BK * 2) >> 4;        // rows 128..255 of the A tile, either layout
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
#pragma unroll
            for (int h = 0; h < MH; ++h) {
              if (PAIR) tc_mma_bf16_pair(d_tmem + h * BN, adesc + h * A_HALF + k * A_STEP, bdesc + k * B_STEP, IDESC,
                                         (kb > piece_kb0 || k > 0) ? 1u : 0u);
              else tc_mma_bf16(d_tmem + h * BN, adesc + h * A_HALF + k * A_STEP, bdesc + k * B_STEP, IDESC,
                               (kb > piece_kb0 || k > 0) ? 1u : 0u);
            }
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) tc_commit_pair(smem_u32(&empty_bar[stage]));
          else tc_commit(smem_u32(&empty_bar[stage]));
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (PAIR) tc_commit_pair(smem_u32(&tmem_full_bar[acc]));   // accumulator complete (both CTAs' halves)
        else tc_commit(smem_u32(&tmem_full_bar[acc]));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // Eight warps: warp & 3 = TMEM lane quarter (32 rows), (warp - 2) >> 2 = column half.
    // What the tail operation has to READ (old weights for the SGD update, stored activations
    // for the ReLU mask) is requested before the accumulator is waited for, so that its HBM
    // latency hides under the MMAs of this tile.
    constexpr int HC = BN / 2;                    // columns per warp
    constexpr int NV = HC / 8;                    // 16-byte vectors per thread and tile
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    if (te && p.te == 2) {
      // ---- One piece of a sum over K, kept as an fp32 plane of its own (Appendix A.2: the partial result a
      // process holds before the all-reduce): the accumulator leaves through two 128B-swizzled staging boxes of
      // [32 rows][32 columns] per warp and TMA stores into partials[s][M][N] (a 3-D map, so a tile's rows
      // beyond M are clipped instead of landing in the next plane).  With a K range of a few k-blocks per
      // piece the epilogue is most of a tile's time, and row-per-lane stores of 16 bytes keep the LSU busy
      // for 32 cycles each; the bulk store takes the LSU out of the path.
      const int e = warp - 2;
      const uint32_t stg = ring + (te_ring ? 0 : STAGES_TEP * STAGE_BYTES) + e * (2 * 4096);
      uint8_t* stg_gen = smem_raw + (stg - smem_u32(smem_raw));
      int it = 0, nb = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
        const Work wk = decode_work<FIX>(p, w);
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1u;
        const int row0 = wk.tm * TILE_M + static_cast<int>(rank) * BMT + q * 32;
        const int col0 = wk.tn * BN + half * HC;
        ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_phase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * ACC_COLS + half * HC;
#pragma unroll
        for (int c = 0; c < HC / 32; ++c, ++nb) {
          uint32_t r[32];
          tc_ld32(taddr + c * 32, r);
          // the store that used this box two chunks ago has read it
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          __syncwarp();
          tc_wait_ld();
          if (c == HC / 32 - 1) {                    // accumulator fully in registers: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
              else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
            }
          }
          uint8_t* box = stg_gen + (nb & 1) * 4096 + lane * 128;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(box + ((j ^ (lane & 7)) << 4)) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic writes -> visible to TMA
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                         ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(col0 + c * 32), "r"(row0), "r"(wk.s),
                           "r"(stg + (nb & 1) * 4096)
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
        }
      }
      if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores done before the CTA exits
      __syncwarp();
    } else if (te) {
      // ---- TMA epilogue: the tile's old weights / mask source arrive in this warp's staging boxes by
      // TMA, are combined in place with the accumulator, and leave by TMA store; the LSU never touches
      // global memory.  A box ([32 rows][64 columns] bf16) is requested for the NEXT tile as soon as its
      // store for this tile has read it, so the HBM latency of that load passes under the rest of this
      // tile's epilogue and the next tile's main loop instead of standing between two tiles (with K = B
      // of a few hundred, a tile's main loop is only a few microseconds long).
      const int e = warp - 2;
      const uint32_t stg = ring + (te_ring ? 0 : STAGES_TE * STAGE_BYTES) + e * (TE_BOXES * 4096);
      uint8_t* stg_gen = smem_raw + (stg - smem_u32(smem_raw));
      uint32_t lphase = 0;
      const bool need_load = p.epi.op == EPI_SGD || (p.epi.op == EPI_MASK && p.epi.mask != nullptr);
      const CUtensorMap* src_map = p.epi.op == EPI_SGD ? &tmOut : &tmAux;
      auto request = [&](const Work& wk, int b) {        // lane 0: box b of tile wk
        const int row0 = wk.tm * TILE_M + static_cast<int>(rank) * BMT + q * 32;
        const int col0 = wk.tn * BN + half * HC;
        const uint32_t lb = smem_u32(&te_bar[e * 2 + b]);
        mbar_expect_tx(lb, 4096);
        tma_load_2d(stg + b * 4096, src_map, col0 + b * 64, row0, lb);
      };
      const bool ahead = p.te_prefetch != 0;
      if (need_load && ahead && lane == 0 && w_first < total_work) {
        const Work wk0 = decode_work<FIX>(p, w_first);
#pragma unroll
        for (int b = 0; b < TE_BOXES; ++b) request(wk0, b);
      }
      int it = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
        const Work wk = decode_work<FIX>(p, w);
        const bool has_next = w + w_step < total_work;
        Work wk_next = wk;
        if (need_load && ahead && has_next && lane == 0) wk_next = decode_work<FIX>(p, w + w_step);
        if (need_load && !ahead && lane == 0) {            // tuning knob: request the boxes when the tile starts
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
#pragma unroll
          for (int b = 0; b < TE_BOXES; ++b) request(wk, b);
        }
        const int acc = it % acc_bufs;
        const uint32_t acc_phase = (it / acc_bufs) & 1u;
        const int row0 = wk.tm * TILE_M + static_cast<int>(rank) * BMT + q * 32;
        const int col0 = wk.tn * BN + half * HC;
        ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_phase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * acc_stride + half * HC;
#pragma unroll
        for (int b = 0; b < TE_BOXES; ++b) {
          if (need_load) {
            ok = mbar_wait(smem_u32(&te_bar[e * 2 + b]), lphase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
          } else if (lane == 0) {
            // nothing is loaded into the box: its store for the previous tile must have read it before it is refilled
            if (TE_BOXES == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          }
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int c = b * 2 + cc;
            uint32_t r[32];
            tc_ld32(taddr + c * 32, r);
            tc_wait_ld();
            if (JOIN && join > 1) add_joined_pieces(taddr + c * 32, join, ACC_COLS, r);
            if (c == HC / 32 - 1) {                  // accumulator fully in registers: hand it back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
                else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
              }
            }
            uint8_t* box = stg_gen + b * 4096 + lane * 128;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint4* cell = reinterpret_cast<uint4*>(box + (((cc * 4 + j) ^ (lane & 7)) << 4));
              float v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[j * 8 + i]);
              if (need_load) {
                const uint4 qv = *cell;
                const uint32_t wv[4] = {qv.x, qv.y, qv.z, qv.w};
                if (p.epi.op == EPI_SGD) {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    v[2 * i] = fmaf(p.epi.scale, v[2 * i], bf16_bits_to_f32(wv[i] & 0xFFFFu));
                    v[2 * i + 1] = fmaf(p.epi.scale, v[2 * i + 1], bf16_bits_to_f32(wv[i] >> 16));
                  }
                } else {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    if (!(bf16_bits_to_f32(wv[i] & 0xFFFFu) > 0.f)) v[2 * i] = 0.f;
                    if (!(bf16_bits_to_f32(wv[i] >> 16) > 0.f)) v[2 * i + 1] = 0.f;
                  }
                }
              } else if (p.epi.op == EPI_ACT) {
                const int n = col0 + c * 32 + j * 8;
                if (p.epi.bias && n < p.N) {
                  const float4 b0 = *reinterpret_cast<const float4*>(p.epi.bias + n);
                  const float4 b1 = *reinterpret_cast<const float4*>(p.epi.bias + n + 4);
                  v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
                  v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
                }
                if (p.epi.relu) {
#pragma unroll
                  for (int i = 0; i < 8; ++i) v[i] = fmaxf(v[i], 0.f);
                }
              }
              uint4 o;
              o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
              o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
              *cell = o;
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic writes -> visible to TMA
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(col0 + b * 64), "r"(row0), "r"(stg + b * 4096)
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (need_load && ahead && has_next) {
              asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the store has read the box: refill it
              request(wk_next, b);
            }
          }
        }
        if (!ok) break;
        lphase ^= 1u;
      }
      if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores done before the CTA exits
      __syncwarp();
    } else if (FIX == 1 && p.fix != 0) {
      // ---- Running sum of a product's K pieces (Appendix A.2: the sum over the blocks of a process group,
      // taken in ascending block order).  Piece s of a tile adds its accumulator to the sum of pieces
      // 0..s-1, which the CTA that finished piece s-1 left in ONE fp32 plane, and writes the new sum back;
      // the last piece applies the tail operation instead.  Same additions in the same order as the
      // reduction kernel over S planes, so the results agree bit for bit.  All loads of a 32-column chunk
      // (the sum so far and, for the last piece, the bf16 operand of its tail operation) are issued together
      // under the TMEM load, so a chunk costs one memory round trip.
      // Measured on the 8192^3 products (two pieces): 0.5 ms less per training step than S planes plus the
      // reduction kernel -- and no more, because these reads share the L2 -> SM path with the operand ring,
      // which the main loop already keeps close to its limit; a variant that transposed each chunk through
      // shared memory for fully coalesced accesses was slower still (24.2 against 21.2 ms per step).
      const int e = warp - 2;
      const bool src_bf16 = p.epi.out_bf16 && ((p.epi.op == EPI_SGD && p.epi.master == nullptr) ||
                                               (p.epi.op == EPI_MASK && p.epi.mask != nullptr));
      const __nv_bfloat16* tsrc = p.epi.op == EPI_SGD ? reinterpret_cast<const __nv_bfloat16*>(p.epi.out)
                                                      : reinterpret_cast<const __nv_bfloat16*>(p.epi.mask);
      const int64_t tsrc_ld = p.epi.op == EPI_SGD ? p.epi.ldo : p.epi.ldmask;
      int it = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
        const Work wk = decode_work<FIX>(p, w);
        const int acc = it % ACC_BUFS;
        const uint32_t acc_phase = (it / ACC_BUFS) & 1u;
        const bool first = wk.s == 0, last = wk.s == p.S - 1;
        const bool tail_src = last && src_bf16;
        const int64_t nbase = static_cast<int64_t>(wk.tn) * BN + half * HC;
#pragma unroll 1
        for (int h = 0; h < MH; ++h) {
          const int64_t m = static_cast<int64_t>(wk.tm) * TILE_M + rank * BMT + h * 128 + q * 32 + lane;
          const bool row_ok = m < p.M;
          int* flag = p.flags + (((static_cast<int64_t>(wk.tm) * p.tiles_n + wk.tn) * 2 + rank) * 2 + h) * 8 + e;
          if (h == 0) {
            ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_phase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
          }
          if (!first) {                          // the sum of pieces 0..s-1 of these rows and columns is complete
            if (lane == 0) ok = flag_wait(flag, wk.s, abortp, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * ACC_COLS + h * BN + half * HC;
#pragma unroll
          for (int c = 0; c < HC / 32; ++c) {
            uint32_t r[32];
            tc_ld32(taddr + c * 32, r);
            uint4 run[8], src[4];
            if (!first && row_ok) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int64_t n = nbase + c * 32 + j * 8;
                if (n < p.N) {
                  run[2 * j] = __ldcg(reinterpret_cast<const uint4*>(p.partials + m * p.N + n));
                  run[2 * j + 1] = __ldcg(reinterpret_cast<const uint4*>(p.partials + m * p.N + n + 4));
                  if (tail_src) src[j] = *reinterpret_cast<const uint4*>(tsrc + m * tsrc_ld + n);
                }
              }
            }
            tc_wait_ld();
            if (h == MH - 1 && c == HC / 32 - 1) {     // accumulator fully in registers: hand it back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
                else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
              }
            }
            if (row_ok) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int64_t n = nbase + c * 32 + j * 8;
                if (n < p.N) {
                  float v[8];
#pragma unroll
                  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[j * 8 + i]);
                  if (!first) {                   // ascending order: (sum of the earlier pieces) + this piece
                    const uint4 r0 = run[2 * j], r1 = run[2 * j + 1];
                    v[0] = __uint_as_float(r0.x) + v[0]; v[1] = __uint_as_float(r0.y) + v[1];
                    v[2] = __uint_as_float(r0.z) + v[2]; v[3] = __uint_as_float(r0.w) + v[3];
                    v[4] = __uint_as_float(r1.x) + v[4]; v[5] = __uint_as_float(r1.y) + v[5];
                    v[6] = __uint_as_float(r1.z) + v[6]; v[7] = __uint_as_float(r1.w) + v[7];
                  }
                  if (!last) {
                    float* dst = p.partials + m * p.N + n;
                    __stcg(reinterpret_cast<float4*>(dst), make_float4(v[0], v[1], v[2], v[3]));
                    __stcg(reinterpret_cast<float4*>(dst + 4), make_float4(v[4], v[5], v[6], v[7]));
                  } else if (tail_src) {            // the arithmetic of epi_apply8, operand already in registers
                    const uint4 qv = src[j];
                    const uint32_t wv[4] = {qv.x, qv.y, qv.z, qv.w};
                    if (p.epi.op == EPI_SGD) {
#pragma unroll
                      for (int i = 0; i < 4; ++i) {
                        v[2 * i] = fmaf(p.epi.scale, v[2 * i], bf16_bits_to_f32(wv[i] & 0xFFFFu));
                        v[2 * i + 1] = fmaf(p.epi.scale, v[2 * i + 1], bf16_bits_to_f32(wv[i] >> 16));
                      }
                    } else {
#pragma unroll
                      for (int i = 0; i < 4; ++i) {
                        if (!(bf16_bits_to_f32(wv[i] & 0xFFFFu) > 0.f)) v[2 * i] = 0.f;
                        if (!(bf16_bits_to_f32(wv[i] >> 16) > 0.f)) v[2 * i + 1] = 0.f;
                      }
                    }
                    uint4 o;
                    o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
                    o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
                    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.epi.out) + m * p.epi.ldo + n) = o;
                  } else {
                    epi_apply8(p.epi, m, n, v);
                  }
                }
              }
            }
          }
          if (!last) {
            __threadfence();                       // this lane's part of the sum is visible device-wide ...
            __syncwarp();
            if (lane == 0) flag_publish(flag, wk.s + 1);      // ... before the next piece is told so
          } else if (lane == 0) {
            *flag = 0;                             // consumed: the word is zero again for the next launch
          }
        }   // h
      }
    } else if (JOIN && join > 1) {
      // ---- Joined pieces without the TMA epilogue (fp32 results, ragged leading dimensions, 256-row tiles): each
      // 32-column chunk is the ascending sum of the tile's accumulators, then the tail operation from registers.
      int it = 0;
      bool ok = true;
      for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
        const Work wk = decode_work<FIX>(p, w);
        const int acc = it % acc_bufs;
        const uint32_t acc_phase = (it / acc_bufs) & 1u;
        const int64_t nbase = static_cast<int64_t>(wk.tn) * BN + half * HC;
        ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_phase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int h = 0; h < MH; ++h) {
          const int64_t m = static_cast<int64_t>(wk.tm) * TILE_M + rank * BMT + h * 128 + q * 32 + lane;
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * acc_stride + h * BN + half * HC;
#pragma unroll 1
          for (int c = 0; c < HC / 32; ++c) {
            uint32_t r[32];
            tc_ld32(taddr + c * 32, r);
            tc_wait_ld();
            add_joined_pieces(taddr + c * 32, join, ACC_COLS, r);
            if (h == MH - 1 && c == HC / 32 - 1) {     // accumulators fully in registers: hand them back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
                else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
              }
            }
            if (m < p.M) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int64_t n = nbase + c * 32 + j * 8;
                if (n < p.N) {
                  float v[8];
#pragma unroll
                  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[j * 8 + i]);
                  epi_apply8(p.epi, m, n, v);
                }
              }
            }
          }
        }
      }
    } else {
    const bool prefetch = p.S == 1 && p.epi.out_bf16 &&
                          ((p.epi.op == EPI_SGD && p.epi.master == nullptr) ||      // master weights: shared tail, no prefetch
                           (p.epi.op == EPI_MASK && p.epi.mask != nullptr));
    const __nv_bfloat16* pre_src = p.epi.op == EPI_SGD ? reinterpret_cast<const __nv_bfloat16*>(p.epi.out)
                                                       : reinterpret_cast<const __nv_bfloat16*>(p.epi.mask);
    const int64_t pre_ld = p.epi.op == EPI_SGD ? p.epi.ldo : p.epi.ldmask;
    int it = 0;
    bool ok = true;
    for (int w = w_first; w < total_work && ok; w += w_step, ++it) {
      const Work wk = decode_work<FIX>(p, w);
      const int acc = it % ACC_BUFS;
      const uint32_t acc_phase = (it / ACC_BUFS) & 1u;
      const int64_t nbase = static_cast<int64_t>(wk.tn) * BN + half * HC;
      float* part = p.S > 1 ? p.partials + static_cast<int64_t>(wk.s) * p.M * p.N : nullptr;
#pragma unroll 1
      for (int h = 0; h < MH; ++h) {
      const int64_t m = static_cast<int64_t>(wk.tm) * TILE_M + rank * BMT + h * 128 + q * 32 + lane;
      const bool row_ok = m < p.M;
      uint4 pre[NV];
      if (prefetch) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
          const int64_t n = nbase + j * 8;
          pre[j] = (row_ok && n < p.N) ? *reinterpret_cast<const uint4*>(pre_src + m * pre_ld + n) : make_uint4(0, 0, 0, 0);
        }
      }
      if (h == 0) {
        ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), acc_phase, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
      }
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * ACC_COLS + h * BN + half * HC;
#pragma unroll
      for (int c = 0; c < HC / 32; ++c) {
        uint32_t r[32];
        tc_ld32(taddr + c * 32, r);
        tc_wait_ld();
        if (h == MH - 1 && c == HC / 32 - 1) {     // accumulator fully in registers: hand it back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));
            else mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
          }
        }
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int64_t n = nbase + c * 32 + j * 8;
            if (n < p.N) {
              float v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[j * 8 + i]);
              if (part) {
                float* dst = part + m * p.N + n;
                *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
              } else if (prefetch) {
                const uint4 qv = pre[c * 4 + j];
                const uint32_t wv[4] = {qv.x, qv.y, qv.z, qv.w};
                if (p.epi.op == EPI_SGD) {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    v[2 * i] = fmaf(p.epi.scale, v[2 * i], bf16_bits_to_f32(wv[i] & 0xFFFFu));
                    v[2 * i + 1] = fmaf(p.epi.scale, v[2 * i + 1], bf16_bits_to_f32(wv[i] >> 16));
                  }
                } else {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    if (!(bf16_bits_to_f32(wv[i] & 0xFFFFu) > 0.f)) v[2 * i] = 0.f;
                    if (!(bf16_bits_to_f32(wv[i] >> 16) > 0.f)) v[2 * i + 1] = 0.f;
                  }
                }
                uint4 o;
                o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
                o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
                *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.epi.out) + m * p.epi.ldo + n) = o;
              } else {
                epi_apply8(p.epi, m, n, v);
              }
            }
          }
        }
      }
      }   // h
    }
    }   // register epilogue
  }

  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();            // the peer may still signal barriers in this CTA's shared memory
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// A wait that cannot succeed: nothing ever arrives at `bar`.  Exercises the give-up path.
__global__ void selftest_timeout_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait_slow(smem_u32(&bar), 0, &abort_flag, status, DEV_TIMEOUT_EPILOGUE, limit_ns);
  __syncthreads();
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
// The opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of each kernel.
constexpr int MAX_DEVICES = 64;
bool g_attr_done[MAX_DEVICES] = {false};

// 2-D bf16 tensor map: `inner` contiguous elements per row, `rows` rows `ld` elements apart.
cudaError_t make_map(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t rows, uint64_t ld,
                     uint32_t box_inner, uint32_t box_rows) {
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// 3-D fp32 tensor map over partials[S][M][N]; box = [1][32 rows][32 columns] (128 bytes per row, 128B-swizzled).
cudaError_t make_planes_map(CUtensorMap* tm, const float* base, uint64_t N, uint64_t M, uint64_t S) {
  const cuuint64_t dims[3] = {N, M, S};
  const cuuint64_t strides[2] = {N * 4, N * M * 4};
  const cuuint32_t box[3] = {32, 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int A_MN, int B_MN>
cudaError_t set_attr() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 1, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 128, 1, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 2, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 2, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 2, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 256, 1, 0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 128, 1, 0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 128, 2, 0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, 128, 2, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_BYTES);
}

template <int A_MN, int B_MN>
cudaError_t launch_t(const TcGemm& g, const Params& p, cudaStream_t stream) {
  const size_t smem = SMEM_DYN_BYTES;
  const dim3 grid(g.grid), block(NUM_THREADS);
  if (g.pair && p.fix) {
    if (g.MH == 2) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 2, 1, 1>, grid, block, smem, stream, 2, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
    return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 1>, grid, block, smem, stream, 2, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  }
  if (p.join > 1) {        // (the planner admits only these four shapes)
    if (g.pair) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 2>, grid, block, smem, stream, 2, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
    if (g.BN == 256) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 1, 0, 2>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
    if (g.MH == 1) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 128, 1, 0, 2>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
    return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 128, 2, 0, 2>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  }
  if (g.pair && g.MH == 2) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 2, 1, 0>, grid, block, smem, stream, 2, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  if (g.pair) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 1, 1, 0>, grid, block, smem, stream, 2, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  if (g.BN == 256 && g.MH == 1) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 1, 0, 0>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  if (g.BN == 128 && g.MH == 1) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 128, 1, 0, 0>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  if (g.BN == 256) return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 256, 2, 0, 0>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
  return launch_pdl(gemm_tc_kernel<A_MN, B_MN, 128, 2, 0, 0>, grid, block, smem, stream, 1, g.tmA, g.tmB, g.tmOut, g.tmAux, p);
}

}  // namespace

cudaError_t tc_gemm_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (g_attr_done[dev]) return cudaSuccess;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  if ((e = set_attr<0, 0>()) != cudaSuccess) return e;
  if ((e = set_attr<0, 1>()) != cudaSuccess) return e;
  if ((e = set_attr<1, 1>()) != cudaSuccess) return e;
  g_attr_done[dev] = true;
  return cudaSuccess;
}

cudaError_t selftest_timeout_launch(int* status, int limit_ms, cudaStream_t stream) {
  selftest_timeout_kernel<<<1, 32, 0, stream>>>(status, static_cast<unsigned long long>(limit_ms) * 1000000ull);
  return cudaGetLastError();
}

// Everything about a contraction's launch that is decided on the host and needs no device: tile shape, CTA pairs,
// the pieces of K (the caller's, the planner's own cuts, pieces joined in tensor memory, the running sum), planes
// stored by TMA, the TMA epilogue (`want_te`: the result is bf16 and goes through an epilogue operation), the grid.
void tc_gemm_plan(TcGemm& g, int num_sms, bool want_te) {
  const int kb_total = (g.K + BK - 1) / BK;
  if (g.k_splits > kb_total) g.k_splits = kb_total;
  // Tile shape and (for the network's own contractions) an extra cut of K, chosen by a small cost
  // model in SM clocks.  Per 64-wide k-block a CTA either waits for the tensor pipe (128 x BN x 16
  // MMAs at 75 % / 85 % of peak for BN = 128 / 256) or for its operand fill (about 70 B/clk into
  // shared memory, measured); 256 x 256 tiles cannot overlap their epilogue; every extra piece of K
  // costs fp32 partial traffic and the reduction launch.  Checked against measurements: 8192^3 picks
  // 256 x 256 (1236 -> 1445 TFLOP/s), the batch-512 forward product 512 x 4096 x 25088 picks
  // 256 x 256 with K cut in 4; short-K and split products pick CTA pairs (cta_group::2).
  // Short pieces whose planes nobody asked to see may stay in tensor memory (`join`): the tile's K range is
  // walked piece by piece into accumulators of their own, and the epilogue adds them in ascending order -- the
  // sum of the reduction kernel over the same pieces, bit for bit, with no fp32 plane crossing HBM.  Needs
  // k_splits x (tile's TMEM columns) <= 512; measured: cfg3 1x16 (two pieces of 4 k-blocks) 0.67 -> 0.34 ms per step.
  const bool join_ok = g.allow_fix && (g.k_splits == 2 || g.k_splits == 4) && !getenv("MBD_NO_JOIN") &&
                       (kb_total / g.k_splits < 32 || getenv("MBD_JOIN_ANY"));        // tuning knobs
  g.join = 1;
  {
    double best = 1e30;
    int best_bn = 128, best_mh = 1, best_x = 1, best_pair = 0, best_join = 0;
    const int x_max = g.allow_extra_split ? 32 : 1;
    const bool x_any = getenv("MBD_TC_X_POW2") == nullptr;      // tuning knob: extra cuts in powers of two only
    for (int cand = 0; cand < 4; ++cand) {           // 0: 128-row tiles, 1: 256-row tiles, 2: CTA pairs, 3: pairs of 256-row CTAs
      const int mh = (cand == 1 || cand == 3) ? 2 : 1;
      const bool pair = cand >= 2;
      for (int bn = pair ? 256 : 128; bn <= 256; bn += 128) {
        for (int jn = 0; jn <= (join_ok && g.k_splits * mh * bn <= 512 ? 1 : 0); ++jn) {
        for (int x = 1; x <= (jn ? 1 : x_max); x = x_any ? x + 1 : x * 2) {
          const long long S = jn ? 1 : 1ll * g.k_splits * x;
          if (S > kb_total || (x > 1 && kb_total / S < 8)) continue;
          const double kb = static_cast<double>(kb_total) / S;
          const int tile_m = 128 * mh * (pair ? 2 : 1);
          const long long units = 1ll * ((g.M + tile_m - 1) / tile_m) * ((g.N + bn - 1) / bn) * S;
          const int slots = pair ? num_sms / 2 : num_sms;
          const double waves = static_cast<double>((units + slots - 1) / slots);
          // per SM and k-block: tensor-pipe clocks and operand-fill clocks; the efficiencies follow
          // the measured order 256 x 256 single < 256 x 256 pair < 512 x 256 pair on 8192^3
          const double eff = pair ? (mh == 2 ? 0.87 : 0.84) : (mh == 2 ? 0.80 : (bn == 256 ? 0.85 : 0.75));
          const double mma = 4.0 * mh * ((pair ? 256 : bn) / 2) / eff;
          const double fill = (pair ? 128.0 * mh + 128.0 : 128.0 * mh + bn) * 128.0 / 70.0;
          const double mainloop = kb * (mma > fill ? mma : fill);
          const double epi = 2500.0 * mh * bn / 256.0 * (S > 1 ? 2.0 : 1.0) * (jn ? 1.0 + 0.25 * (g.k_splits - 1) : 1.0);
          // (joined pieces take the shape the unsplit product would: a CTA pair whose two pieces fill tensor memory
          // measured 14 % faster than 128 x 128 tiles with room for two sets on the batch-512 product, 4 % slower on
          // the batch-256 one -- the model's epilogue estimate cannot tell them apart)
          const bool overlapped = mh * bn <= 256;        // two accumulators fit in TMEM
          double unit = overlapped ? (mainloop > epi ? mainloop : epi) : mainloop + epi;
          double t = waves * unit + 4000.0;
          if (S > 1 && (x > 1 || join_ok)) {   // the reduction exists anyway when the grid itself splits K and must keep planes
            const double bytes = (static_cast<double>(S) + 1.0) * g.M * g.N * 4.0;
            t += (5e-6 + bytes / 5.5e12) * 1.9e9;
          }
          if (t < best) { best = t; best_bn = bn; best_mh = mh; best_x = x; best_pair = pair ? 1 : 0; best_join = jn; }
        }
        }
      }
    }
    g.BN = best_bn; g.MH = best_mh; g.pair = best_pair;
    g.k_splits *= best_x;
    if (best_join) { g.join = g.k_splits; g.k_splits = 1; }
  }
  if (const char* ev = getenv("MBD_TC_MH")) {          // tuning knobs
    const int mh = atoi(ev);
    if (mh == 1 || mh == 2) { g.MH = mh; g.pair = 0; }
  }
  if (const char* ev = getenv("MBD_TC_BN")) {
    const int bn = atoi(ev);
    if (bn == 128 || bn == 256) g.BN = bn;
  }
  if (const char* ev = getenv("MBD_TC_PAIR")) {        // tuning knob: CTA pairs (256 x 256 per pair)
    if (atoi(ev) == 1) { g.pair = 1; g.MH = 1; g.BN = 256; }
    else if (atoi(ev) == 2) { g.pair = 1; g.MH = 2; g.BN = 256; }      // 512 x 256 per pair
    else if (atoi(ev) == 0) g.pair = 0;
  }
  if (g.pair) g.BN = 256;
  if (g.join > 1 && g.join * g.MH * g.BN > 512) { g.k_splits = g.join; g.join = 1; }     // a forced tile shape without room
  if (getenv("MBD_TC_DEBUG"))
    fprintf(stderr, "tc_gemm_prepare: variant %d  M %d N %d K %d  pieces of K %d%s  ->  %d x %d tile%s\n", g.variant, g.M, g.N,
            g.K, g.join > 1 ? g.join : g.k_splits, g.join > 1 ? " (joined in tensor memory)" : "", 128 * g.MH * (g.pair ? 2 : 1),
            g.BN, g.pair ? " (CTA pair)" : "");
  const int bmt = BM * g.MH * (g.pair ? 2 : 1);        // rows of one work unit's tile
  const int tiles_m = (g.M + bmt - 1) / bmt;
  const int tiles_n = (g.N + g.BN - 1) / g.BN;
  const long long total = 1ll * tiles_m * tiles_n * g.k_splits;
  g.grid = static_cast<int>(total < num_sms ? total : num_sms);
  if (g.pair) {
    const long long pairs = total < num_sms / 2 ? total : num_sms / 2;
    g.grid = static_cast<int>(2 * pairs);
  }
  // Running sum instead of S planes and a reduction launch: when the pieces of a tile are far apart in the
  // work order (at least as many tiles as CTA slots: the pieces of one tile never run at the same time) ...
  {
    const long long tiles = 1ll * tiles_m * tiles_n;
    const int slots = g.pair ? num_sms / 2 : num_sms;
    const int kb_piece = kb_total / (g.k_splits > 0 ? g.k_splits : 1);
    // ... and a piece's main loop must be long enough to hide the epilogue of the piece before it (which reads
    // the sum back row by row): short pieces are better served by S planes and the coalesced reduction kernel
    // ... and there must be just two of them: with more, most epilogues read a plane back and the step loses
    // (cfg5 with four pieces: 27 ms against 21 ms with two); the kernel itself handles any S.
    const bool two = g.k_splits == 2 || (g.k_splits > 2 && getenv("MBD_FIX_ANY_S") != nullptr);     // tuning knob
    g.fix = g.allow_fix && g.pair && two && tiles >= slots && kb_piece >= 32 ? 1 : 0;
    g.flag_words = g.fix ? tiles * 32 : 0;
  }
  // S planes of short pieces on 128-row tiles leave by TMA store: a piece of fewer than 32 k-blocks is over before
  // its predecessor's row-per-lane stores are (measured: batch-512 backward-weight products in 16 pieces of 8
  // k-blocks 0.49 -> 0.31 ms); long pieces hide those stores and keep the two extra ring stages instead
  // (8192-deep pieces of 64 k-blocks on CTA pairs: 2.5 % slower with the bulk stores).  The map is made at launch.
  // A launch with one work unit per CTA has no next tile to hide stores under, and its ring is idle once the unit's
  // accumulator is complete: the staging boxes then lie in the ring itself (te_ring), all stages are kept, and pieces
  // of any length leave by TMA store (measured: the forward products of the batch-256 network, cut in 4 by the planner).
  {
    const int kb_piece = kb_total / (g.k_splits > 0 ? g.k_splits : 1);
    const int slots = g.pair ? num_sms / 2 : num_sms;
    g.te_ring = total <= slots && !getenv("MBD_TC_NO_TE_RING");                     // tuning knob
    g.te_planes = g.k_splits > 1 && !g.fix && g.MH == 1 && (g.N & 3) == 0 && (kb_piece < 32 || g.te_ring) && !getenv("MBD_TC_NO_TE");
  }
  // TMA epilogue: bf16 output of an unsplit contraction on 128-row tiles (the maps are made by tc_gemm_prepare)
  g.te = want_te && g.MH == 1 && g.k_splits == 1 && !getenv("MBD_TC_NO_TE") ? 1 : 0;
}

cudaError_t tc_gemm_prepare(TcGemm& g, const void* A, int64_t lda, const void* B, int64_t ldb, int num_sms,
                            const Epi* te_epi) {
  cudaError_t e = tc_gemm_init();
  if (e != cudaSuccess) return e;
  if (g.cv.mode != 0 && g.cv.mode != g.variant + 1) return cudaErrorInvalidValue;
  tc_gemm_plan(g, num_sms, te_epi && te_epi->out_bf16 && te_epi->out);
  const bool a_mn = g.variant == 2, b_mn = g.variant >= 1;
  if (!a_mn) e = make_map(&g.tmA, A, g.cv.mode ? g.cv_a_inner : g.K, g.cv.mode && g.cv_a_rows ? g.cv_a_rows : g.M, lda, BK, BM * g.MH);   // A[M,K]: inner = K; box = the rows one CTA loads
  else e = make_map(&g.tmA, A, g.M, g.K, lda, 64, BK);             // A[K,M]: inner = M, one 64-wide chunk per box
  if (e != cudaSuccess) return e;
  if (!b_mn) e = make_map(&g.tmB, B, g.K, g.N, ldb, BK, g.pair ? g.BN / 2 : g.BN);    // B[N,K]
  else if (g.cv.mode) e = make_map(&g.tmB, B, g.cv_b_inner, g.cv_b_rows, ldb, 64, BK);     // the tensor as stored; the kernel shifts
  else e = make_map(&g.tmB, B, g.N, g.K, ldb, 64, BK);             // B[K,N]
  if (e != cudaSuccess) return e;
  g.tmOut = g.tmA;
  g.tmAux = g.tmA;
  if (g.te) {
    e = make_map(&g.tmOut, te_epi->out, g.N, g.M, te_epi->ldo, 64, 32);
    if (e != cudaSuccess) return e;
    if (te_epi->op == EPI_MASK && te_epi->mask) {
      e = make_map(&g.tmAux, te_epi->mask, g.N, g.M, te_epi->ldmask, 64, 32);
      if (e != cudaSuccess) return e;
    }
    g.te_epi = *te_epi;
  }
  return e;
}

cudaError_t tc_gemm_launch(const TcGemm& g, cudaStream_t stream) {
  Params p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.tiles_m = (g.M + BM * g.MH * (g.pair ? 2 : 1) - 1) / (BM * g.MH * (g.pair ? 2 : 1));
  p.tiles_n = (g.N + g.BN - 1) / g.BN;
  p.kb_total = (g.K + BK - 1) / BK;
  p.S = g.k_splits;
  p.group_m = 8;                        // m-tiles per raster group (L2 reuse of the B operand)
  if (const char* ev = getenv("MBD_TC_GROUP_M")) { const int gm = atoi(ev); if (gm >= 1) p.group_m = gm; }
  p.partials = g.partials;
  p.fix = g.fix && g.pair && g.flags != nullptr;
  if (p.fix && getenv("MBD_FIX_PLAIN_ORDER")) p.fix = 2;                 // tuning knob
  p.te_prefetch = getenv("MBD_TE_NO_PREFETCH") ? 0 : 1;                  // tuning knob
  p.te_ring = 0;
  p.flags = g.flags;
  p.join = g.join > 1 ? g.join : 1;
  p.cv = g.cv;
  p.epi = g.epi;
  p.status = g.status;
  p.te = g.te && g.epi.op == g.te_epi.op && g.epi.out == g.te_epi.out && g.epi.out_bf16 && g.epi.mask == g.te_epi.mask &&
         g.epi.ldo == g.te_epi.ldo && g.k_splits == 1 && !g.epi.master;   // the TMA epilogue has no master path
  // S planes on 128-row tiles: stored by TMA when the planes can be described by a tensor map
  if (g.te_planes && g.k_splits > 1 && !p.fix && g.partials && (reinterpret_cast<uintptr_t>(g.partials) & 15u) == 0) {
    if (g.planes_base != g.partials) {
      const cudaError_t e = make_planes_map(&g.tmPlanes, g.partials, g.N, g.M, g.k_splits);
      if (e != cudaSuccess) return e;
      g.planes_base = g.partials;
    }
    p.te = 2;
    p.te_ring = g.te_ring;
    TcGemm h = g;
    h.tmOut = g.tmPlanes;
    if (g.variant == 0) return launch_t<0, 0>(h, p, stream);
    if (g.variant == 1) return launch_t<0, 1>(h, p, stream);
    return launch_t<1, 1>(h, p, stream);
  }
  // (a tail operation that reads -- old weights, a mask source -- requests its boxes while the ring is still in use)
  p.te_ring = p.te == 1 && g.te_ring && (g.epi.op == EPI_ACT || (g.epi.op == EPI_MASK && g.epi.mask == nullptr));
  if (g.variant == 0) return launch_t<0, 0>(g, p, stream);
  if (g.variant == 1) return launch_t<0, 1>(g, p, stream);
  return launch_t<1, 1>(g, p, stream);
}

}  // namespace mbd
