// Domain-parallel 3x3 convolution stack (Section 2.2 and 2.4 of the paper): every image is
// cut into P_r row strips; a strip owner holds its rows plus one halo row per neighbour
// (forward: X halos, backward-data: dY halos).  The exchange is fused into whatever produces a
// tensor: the convolution epilogue stores a strip's first / last row a second time, into the
// neighbouring strip's halo row (one more TMA store of the same staging tile), and the staging pass
// from NCHW does the same.  The weight gradient is formed as per-owner partial sums that are then
// added (the all-reduce over the strips, third term of Eq. 7).
//
// Layout in HBM: every activation / gradient tensor lives as "strips": [Z = B*P_r][R = Hs+2]
// [W][C = 64] bf16 (channels innermost), row 0 and row Hs+1 of a strip being the halo rows
// (zero at the image border).  One pixel = 128 contiguous bytes = one 128B-swizzle row, so a
// TMA box {64 c, n pixels} is directly a K-major (forward, backward-data) or MN-major
// (backward-weight: pixels are the reduction index) tensor-core operand.
//
// conv_fwd_kernel  (forward and, with flipped / transposed weights, backward-data)
//     input-row stationary: every input row segment is loaded once, as ONE box of 130 pixels; the
//     three horizontally shifted operands are views of that box whose descriptors start 0, 1, 2
//     pixel rows (128 bytes) into it (the 128-byte swizzle depends on the shared-memory address
//     only, so a shifted view reads back what TMA wrote).  Each view is multiplied by the
//     stacked taps [K(0,v); K(1,v); K(2,v)] (N = 192); the three 64-column results belong to the
//     output rows r, r-1, r-2, whose accumulators sit next to each other in a ring of eight
//     TMEM blocks.  An output row is complete after three input rows; the epilogue drains it,
//     zeroes the block, and writes it through a swizzled staging tile that TMA stores (the mask
//     source of backward-data arrives by TMA too).  The weights (72 KB) stay resident in shared
//     memory.  A CTA owns one contiguous span of the flattened (strip, segment, row) space.
// conv_wgrad_kernel
//     dK[o,c,u,v] = sum_pixels dY[p,o] X[p + (u-1,v-1), c]: the three horizontal shifts of an X
//     row are again views of one 130-pixel box; two views one pixel apart form one M = 128
//     operand (leading offset 128 bytes); all nine taps accumulate in TMEM for the whole kernel
//     and each CTA writes one fp32 partial, summed in CTA order (= strip order) by wgrad_finish.
#include <stdlib.h>

#include <new>
#include <vector>

#include "conv.h"
#include "conv_general.h"
#include "epi.cuh"
#include "tc_common.cuh"

namespace mbd {

using namespace tc;
typedef __nv_bfloat16 bf16;

namespace {

constexpr int C = 64;                 // channels in and out
constexpr int FWD_PIX = 128;          // output pixels per forward tile (one per TMEM lane)
constexpr int FWD_W_BYTES = 3 * 192 * 128;   // stacked taps, 72 KB
// Ring of input rows: a stage holds ONE box of 130 pixels (x0 - 1 .. x0 + 128) of one row; the three
// horizontally shifted operands are views of it that start 0, 1 and 2 pixel rows (128 bytes each) into the box.
constexpr int FWD1_BOX_PIX = FWD_PIX + 2;
constexpr int FWD1_ROW_BYTES = 17 * 1024;     // 130 x 128 B = 16640 B, padded to the swizzle span
constexpr int FWD1_STAGES = 5;
// Behind the ring: two staging tiles of one output row segment each ([128 pixels][64 channels] bf16, 16 KB,
// 128B-swizzled like the strips' tensor maps) for TMA stores, and two for the rows of the mask source that
// the backward-data mode reads: the epilogue's global traffic goes through TMA.
constexpr int FWD_TILE_BYTES = FWD_PIX * 128;
constexpr int FWD_SMEM = FWD_W_BYTES + FWD1_STAGES * FWD1_ROW_BYTES + 4 * FWD_TILE_BYTES + 1024;
static_assert(FWD_SMEM <= 227 * 1024, "forward kernel's shared memory");
constexpr int FWD_THREADS = 320;      // producer warp, MMA warp, 8 epilogue warps
constexpr int WG_PIX = 128;           // pixels (reduction length) per backward-weight block
constexpr int WG_XSTAGES = 4;          // X rows: one box of 130 pixels each (17 KB), each row used once; 3 x 3 layers take them in pairs
constexpr int WG_YSTAGES = 6;          // dY rows: 16 KB each, plus mirror slots
constexpr int WG_YMIRROR = 3;          // a window of up to four dY rows is contiguous: the first three slots are mirrored behind the last
constexpr int WG_CHUNK = WG_PIX * 128;
constexpr int WG_XROW_BYTES = 17 * 1024;   // 130 x 128 B, padded to the swizzle span; the views may read one row past the box
constexpr int WG_SMEM = WG_XSTAGES * WG_XROW_BYTES + (WG_YSTAGES + WG_YMIRROR) * WG_CHUNK + 1024;
static_assert(WG_SMEM <= 227 * 1024, "backward-weight kernel's shared memory");
constexpr int NUM_THREADS = 192;

enum { MODE_RELU_STORE = 0, MODE_STORE_SSQ = 1, MODE_MASK = 2 };

// Strips of an image of H rows are the balanced ranges [floor(s H / P), floor((s + 1) H / P)): their heights differ by
// at most one.  Every strip is stored with the layout of the tallest one, Hs = ceil(H / P) own rows between two halo
// rows; a shorter strip keeps its lower halo row right behind its last own row (row index height + 1 = Hs), and its
// row Hs + 1 is never written and stays zero.  The kernels walk Hs rows per strip: what they compute for the one
// dead row of a short strip is not stored, and where a dead row would be read as data (the dY rows of the
// backward-weight product) the all-zero row Hs + 1 is read in its place.
__host__ __device__ __forceinline__ int strip_first(int s, int H, int P) { return static_cast<int>((static_cast<long long>(s) * H) / P); }
__host__ __device__ __forceinline__ int strip_height(int s, int H, int P) { return strip_first(s + 1, H, P) - strip_first(s, H, P); }
// The same inside the kernels, where they sit on the epilogue's critical path: strips of equal height (H = Hs P, the
// common case) need no division by P at all, the others one in 32 bits (H P < 2^31 is checked when the network is made).
__device__ __forceinline__ bool strips_uneven(int H, int P, int Hs) { return Hs * P != H; }
__device__ __forceinline__ int strip_first(int s, int H, int P, int Hs) {
  return !strips_uneven(H, P, Hs) ? s * Hs : static_cast<int>(static_cast<unsigned>(s * H) / static_cast<unsigned>(P));
}
__device__ __forceinline__ int strip_height(int s, int H, int P, int Hs) {
  return !strips_uneven(H, P, Hs) ? Hs : strip_first(s + 1, H, P, Hs) - strip_first(s, H, P, Hs);
}
__device__ __forceinline__ int strip_of_row(int h, int H, int P, int Hs) {
  return !strips_uneven(H, P, Hs) ? h / Hs : static_cast<int>(static_cast<unsigned>((h + 1) * P - 1) / static_cast<unsigned>(H));
}

// ------------------------------------------------------------------------------ layout kernels
// NCHW -> strips.  Block = 32 consecutive pixels of one image's flattened (h, w) plane (so narrow
// images fill their blocks too), all 64 channels; 128 threads.  A row that borders another strip is
// also written into that neighbour's halo row: this is the forward halo exchange for the network
// input (and the backward one for a gradient that arrives from above), fused into the staging pass.
__global__ void __launch_bounds__(128)
nchw_to_strips_kernel(const bf16* __restrict__ src, bf16* __restrict__ dst, int H, int W, int P_r, int Hs) {
  // shared memory holds channel PAIRS as 32-bit words, [pixel][pair] with an odd pitch, so both
  // phases are free of bank conflicts.
  __shared__ uint32_t tile[32][33];
  const int HW = H * W;
  const int p0 = blockIdx.x * 32, b = blockIdx.y;
  const int t = threadIdx.x;
  {
    const int cp = t >> 2, wq = (t & 3) * 8;          // channels 2cp, 2cp+1; pixels p0+wq .. p0+wq+7
    const bf16* q0 = src + (static_cast<int64_t>(b) * C + 2 * cp) * HW + p0 + wq;
    const bf16* q1 = q0 + HW;
    uint16_t lo[8], hi[8];
    if ((HW & 7) == 0 && p0 + wq + 8 <= HW) {
      const uint4 a = __ldcs(reinterpret_cast<const uint4*>(q0)), c = __ldcs(reinterpret_cast<const uint4*>(q1));
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        lo[2 * i] = aw[i] & 0xFFFFu; lo[2 * i + 1] = aw[i] >> 16;
        hi[2 * i] = cw[i] & 0xFFFFu; hi[2 * i + 1] = cw[i] >> 16;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const bool in = p0 + wq + i < HW;
        lo[i] = in ? __bfloat16_as_ushort(q0[i]) : 0;
        hi[i] = in ? __bfloat16_as_ushort(q1[i]) : 0;
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) tile[wq + i][cp] = static_cast<uint32_t>(lo[i]) | (static_cast<uint32_t>(hi[i]) << 16);
  }
  __syncthreads();
  const int px = t >> 2, cq = (t & 3) * 8;            // 8 words = channels 2cq .. 2cq+15 of pixel p0+px
  const int p = p0 + px;
  if (p >= HW) return;
  uint4 v0, v1;
  v0.x = tile[px][cq + 0]; v0.y = tile[px][cq + 1]; v0.z = tile[px][cq + 2]; v0.w = tile[px][cq + 3];
  v1.x = tile[px][cq + 4]; v1.y = tile[px][cq + 5]; v1.z = tile[px][cq + 6]; v1.w = tile[px][cq + 7];
  const int R = Hs + 2;
  const int h = p / W, w = p - h * W;
  const int s = strip_of_row(h, H, P_r, Hs), r = h - strip_first(s, H, P_r, Hs) + 1;
  auto put = [&](int ss, int rr) {
    bf16* q = dst + (((static_cast<int64_t>(b) * P_r + ss) * R + rr) * W + w) * C + 2 * cq;
    *reinterpret_cast<uint4*>(q) = v0;
    *reinterpret_cast<uint4*>(q + 8) = v1;
  };
  put(s, r);
  if (r == 1 && s > 0) put(s - 1, strip_height(s - 1, H, P_r, Hs) + 1);          // first row of a strip: lower halo of the strip above
  if (r == strip_height(s, H, P_r, Hs) && s < P_r - 1) put(s + 1, 0);            // last row of a strip: upper halo of the strip below
}

// strips -> NCHW: the mirror image (own rows only).  Used to hand the last convolution's output to the
// fully connected layers above it, and for read-back.
__global__ void __launch_bounds__(128)
strips_to_nchw_kernel(const bf16* __restrict__ src, bf16* __restrict__ dst, int H, int W, int P_r, int Hs) {
  __shared__ uint32_t tile[32][33];
  const int HW = H * W;
  const int p0 = blockIdx.x * 32, b = blockIdx.y;
  const int t = threadIdx.x;
  const int R = Hs + 2;
  {
    const int px = t >> 2, cq = (t & 3) * 8;
    const int p = p0 + px;
    if (p < HW) {
      const int h = p / W, w = p - h * W;
      const int s = strip_of_row(h, H, P_r, Hs), r = h - strip_first(s, H, P_r, Hs) + 1;
      const bf16* q = src + (((static_cast<int64_t>(b) * P_r + s) * R + r) * W + w) * C + 2 * cq;
      const uint4 v0 = *reinterpret_cast<const uint4*>(q), v1 = *reinterpret_cast<const uint4*>(q + 8);
      tile[px][cq + 0] = v0.x; tile[px][cq + 1] = v0.y; tile[px][cq + 2] = v0.z; tile[px][cq + 3] = v0.w;
      tile[px][cq + 4] = v1.x; tile[px][cq + 5] = v1.y; tile[px][cq + 6] = v1.z; tile[px][cq + 7] = v1.w;
    }
  }
  __syncthreads();
  const int cp = t >> 2, wq = (t & 3) * 8;            // channels 2cp, 2cp+1; pixels p0+wq .. p0+wq+7
  if (p0 + wq >= HW) return;
  uint32_t word[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) word[i] = tile[wq + i][cp];
  bf16* q0 = dst + (static_cast<int64_t>(b) * C + 2 * cp) * HW + p0 + wq;
  bf16* q1 = q0 + HW;
  if ((HW & 7) == 0 && p0 + wq + 8 <= HW) {
    uint4 a, c;
    a.x = (word[0] & 0xFFFFu) | (word[1] << 16); a.y = (word[2] & 0xFFFFu) | (word[3] << 16);
    a.z = (word[4] & 0xFFFFu) | (word[5] << 16); a.w = (word[6] & 0xFFFFu) | (word[7] << 16);
    c.x = (word[0] >> 16) | (word[1] & 0xFFFF0000u); c.y = (word[2] >> 16) | (word[3] & 0xFFFF0000u);
    c.z = (word[4] >> 16) | (word[5] & 0xFFFF0000u); c.w = (word[6] >> 16) | (word[7] & 0xFFFF0000u);
    *reinterpret_cast<uint4*>(q0) = a;
    *reinterpret_cast<uint4*>(q1) = c;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (p0 + wq + i < HW) {
        q0[i] = __ushort_as_bfloat16(static_cast<uint16_t>(word[i] & 0xFFFFu));
        q1[i] = __ushort_as_bfloat16(static_cast<uint16_t>(word[i] >> 16));
      }
  }
}

// Canonical K[o][c][u][v] -> forward operand Wf[v][(u,o)][c] and backward-data operand
// Wb[v'][(u',c)][o] = K[o][c][2-u'][2-v'] (taps flipped, channels swapped).
__global__ void pack_weights_kernel(const bf16* __restrict__ K, bf16* __restrict__ Wf, bf16* __restrict__ Wb) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C * C * 9) return;
  const int o = i / (C * 9), c = (i / 9) % C, u = (i % 9) / 3, v = i % 3;
  const bf16 k = K[i];
  Wf[((v * 3 + u) * C + o) * C + c] = k;
  Wb[(((2 - v) * 3 + (2 - u)) * C + c) * C + o] = k;
}

// A 1 x 1 convolution (the case that needs no halo, remark after Eq. 7) runs through the same kernels as
// a 3 x 3 kernel whose eight outer taps are zero and stay zero: its [o][c] weights live in the centre tap.
__global__ void embed_1x1_kernel(const bf16* __restrict__ K1, bf16* __restrict__ K) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C * C * 9) return;
  K[i] = (i % 9) == 4 ? K1[i / 9] : __float2bfloat16_rn(0.f);
}
template <typename T>
__global__ void extract_1x1_kernel(const T* __restrict__ K, T* __restrict__ K1) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < C * C) K1[i] = K[i * 9 + 4];
}

__global__ void embed_1x1_f32_kernel(const float* __restrict__ g1, float* __restrict__ g) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < C * C * 9) g[i] = (i % 9) == 4 ? g1[i / 9] : 0.f;
}

// One row of every image between the strips tensor and a dense [B][W][C] buffer (see conv_outer_rows).
__global__ void __launch_bounds__(256)
outer_rows_kernel(bf16* __restrict__ buf, bf16* __restrict__ rows, int W, int P_r, int R, int strip, int row, int set) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;      // 16-byte piece inside the row
  const int per_image = W * C / 8;
  if (i >= per_image) return;
  const int b = blockIdx.y;
  uint4* in_strips = reinterpret_cast<uint4*>(buf + ((static_cast<int64_t>(b) * P_r + strip) * R + row) * W * C) + i;
  uint4* in_rows = reinterpret_cast<uint4*>(rows + static_cast<int64_t>(b) * W * C) + i;
  if (set) *in_strips = *in_rows;
  else *in_rows = *in_strips;
}

// Sum of the per-CTA partials [G][9][c][o] in CTA order, into canonical [o][c][u][v]:
// either stored (dK) or applied as K += scale * dK (Eq. 1); the updated weight also goes into the
// two operand layouts the next step's kernels read (see pack_weights_kernel).
__global__ void __launch_bounds__(256)
wgrad_finish_kernel(const float* __restrict__ part, int G, float* __restrict__ dK, bf16* __restrict__ K,
                    bf16* __restrict__ Wf, bf16* __restrict__ Wb, float* __restrict__ K32, float scale, int centre_only) {
  // 64 outputs per block; four thread groups each add a contiguous quarter of the CTA partials in
  // ascending order, and the four sub-sums are added in ascending order too (a fixed order).
  __shared__ float sub[4][64];
  const int j = threadIdx.x & 63, q = threadIdx.x >> 6;
  const int i = blockIdx.x * 64 + j;
  const int g0 = (q * G) / 4, g1 = ((q + 1) * G) / 4;
  float s = 0.f;
  // twelve loads in flight per thread, the ragged tail as guarded loads of the same batch (a tail of dependent single
  // loads had cost as many round trips as the batches before it); the additions keep their ascending order
  for (int g = g0; g < g1; g += 12) {
    float v[12];
#pragma unroll
    for (int e = 0; e < 12; ++e) v[e] = g + e < g1 ? __ldcs(part + static_cast<int64_t>(g + e) * 9 * C * C + i) : 0.f;
#pragma unroll
    for (int e = 0; e < 12; ++e)
      if (g + e < g1) s += v[e];
  }
  sub[q][j] = s;
  __syncthreads();
  if (q != 0) return;
  s = ((sub[0][j] + sub[1][j]) + sub[2][j]) + sub[3][j];
  const int t = i / (C * C), c = (i / C) % C, o = i % C;
  const int e = (o * C + c) * 9 + t;
  if (centre_only && t != 4) {       // the outer taps of a 1 x 1 layer are not parameters: no gradient, no update
    if (dK) dK[e] = 0.f;
    return;
  }
  if (dK) dK[e] = s;
  if (K) {
    bf16 k;
    if (K32) {                       // fp32 master weights: the bf16 kernel is the rounded master
      const float m = fmaf(scale, s, K32[e]);
      K32[e] = m;
      k = __float2bfloat16_rn(m);
    } else {
      k = __float2bfloat16_rn(fmaf(scale, s, __bfloat162float(K[e])));
    }
    const int u = t / 3, v = t - 3 * u;
    K[e] = k;
    Wf[((v * 3 + u) * C + o) * C + c] = k;
    Wb[(((2 - v) * 3 + (2 - u)) * C + c) * C + o] = k;
  }
}

// ------------------------------------------------------------------------------ forward kernel
struct FwdParams {
  int W, Hs, R, nseg;
  int H;                  // image rows: strip s of an image owns strip_height(s, H, P_r) <= Hs of the Hs row slots
  int pack, Z;            // narrow images: `pack` strips share one 128-pixel tile, 128 / pack pixels each (see below)
  int P_r;                // strips per image: a boundary row is also stored into the neighbouring strip's halo row
  int k1;                 // 1 x 1 layer: an output row reads its own input row only, through the centre tap only
  int row_lo, nrows;      // the own rows this launch computes: row_lo .. row_lo + nrows - 1 (1-based; all of them: 1, Hs)
  int loss_add;           // MODE_STORE_SSQ: add to the per-CTA loss partials instead of overwriting them
  long long rows_total;   // output row segments: (strip group z, segment, row) flattened with the row fastest
  int mode;
  bf16* out;              // strips
  const bf16* mask_src;   // strips (MODE_MASK)
  float* loss_part;       // [gridDim.x * 8] (MODE_STORE_SSQ)
  int* status;
};

// A CTA owns a contiguous span of the flattened output rows and walks it as runs of rows of one
// (strip, segment) column; a run of n output rows reads n + 2 input rows.
//
// Narrow images (W <= 62): a 128-pixel tile would be mostly padding, so `pack` = 2, 4 or 8 strips with
// consecutive indices z share it.  Strip j of the group owns tile positions j*sub .. (j+1)*sub - 1,
// sub = 128 / pack >= W + 2, and is loaded / stored by its own TMA box of `sub` pixels; its box starts at
// pixel -1 like the wide one, so the shifted views still line up: position j*sub + i + v of the stage holds
// pixel i + v - 1 of strip j, and what a view reads across a strip boundary only reaches outputs i >= W,
// which are never stored.  `z` of a run is then the first strip of the group.
struct FwdRun {
  int z, seg, h0, n;
};
__device__ __forceinline__ FwdRun fwd_run(const FwdParams& p, long long pos, long long end) {
  const long long col = pos / p.nrows;
  FwdRun r;
  const int k = static_cast<int>(pos - col * p.nrows);       // position inside the launch's row range
  r.h0 = p.row_lo - 1 + k;
  const long long left = end - pos;
  r.n = static_cast<int>(left < p.nrows - k ? left : p.nrows - k);
  r.seg = static_cast<int>(col % p.nseg);
  r.z = static_cast<int>(col / p.nseg) * p.pack;
  return r;
}

// TMEM holds a ring of eight 64-column accumulators, one per output row in flight; output
// row g uses block 7 - (g mod 8), so that the rows r, r-1, r-2 fed by input row r sit in
// ascending, adjacent blocks and one N = 192 instruction updates all three (two instructions
// when the window wraps around the ring).  The epilogue zeroes a block after draining it, so
// every MMA accumulates.
__device__ __forceinline__ int acc_block(int g) { return 7 - (g & 7); }

// PACKED: several strips per tile (narrow images); the wide instantiation keeps its single box per row.
// UNEVEN: strips of unequal height (H mod P_r != 0): only this instantiation carries the dead-row handling -- as a
// run-time case in the common one it cost 1 - 7 % of the epilogue-bound launches.
template <bool PACKED, bool UNEVEN>
__global__ void __launch_bounds__(FWD_THREADS, 1)
conv_fwd_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmMask, const FwdParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[FWD1_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[FWD1_STAGES];
  __shared__ __align__(8) uint64_t acc_full_bar[8];
  __shared__ __align__(8) uint64_t acc_empty_bar[8];
  __shared__ __align__(8) uint64_t w_bar;
  __shared__ __align__(8) uint64_t mask_full_bar[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t w_smem = base;                         // 3 (v) x [192 rows (u, o) x 128 B]
  const uint32_t ring = base + FWD_W_BYTES;             // slot = one input row (one box of 130 pixels)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pack = PACKED ? p.pack : 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < FWD1_STAGES; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), 1); }
    for (int i = 0; i < 8; ++i) { mbar_init(smem_u32(&acc_full_bar[i]), 1); mbar_init(smem_u32(&acc_empty_bar[i]), 8); }
    mbar_init(smem_u32(&w_bar), 1);
    mbar_init(smem_u32(&mask_full_bar[0]), 1);
    mbar_init(smem_u32(&mask_full_bar[1]), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc<512>(smem_u32(&tmem_base_slot));
  if (pack > 1 && threadIdx.x >= 64 && threadIdx.x < 64 + FWD1_STAGES * 16) {
    // packed stages: positions 128, 129 (read by the shifted views, written by no box) hold zeros
    const int i = threadIdx.x - 64;
    uint8_t* ring_gen = smem_raw + (ring - smem_u32(smem_raw));
    *reinterpret_cast<uint4*>(ring_gen + (i >> 4) * FWD1_ROW_BYTES + FWD_PIX * 128 + (i & 15) * 16) = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;
  pdl_trigger();                           // set-up done: the next kernel may be scheduled
  pdl_wait();                              // from here on global memory: earlier kernels must have finished

  const long long r0 = (static_cast<long long>(blockIdx.x) * p.rows_total) / gridDim.x;
  const long long r1 = (static_cast<long long>(blockIdx.x + 1) * p.rows_total) / gridDim.x;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&w_bar), FWD_W_BYTES);
      for (int v = 0; v < 3; ++v) tma_load_2d(w_smem + v * (192 * 128), &tmW, 0, v * 192, smem_u32(&w_bar));
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long pos = r0; pos < r1 && ok;) {
        const FwdRun run = fwd_run(p, pos, r1);
        // 3 x 3: a run of n output rows reads n + 2 input rows, from the row above its first one on;
        // 1 x 1: its own n rows (row index + 1: row 0 of a strip is the upper halo row)
        const int n_in = p.k1 ? run.n : run.n + 2, row_in0 = p.k1 ? run.h0 + 1 : run.h0;
        for (int r = 0; r < n_in; ++r) {
          ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abortp, p.status, DEV_TIMEOUT_PRODUCER);
          if (!ok) break;
          const uint32_t fb = smem_u32(&full_bar[stage]);
          if (pack == 1) {
            mbar_expect_tx(fb, FWD1_BOX_PIX * 128);
            tma_load_4d(ring + stage * FWD1_ROW_BYTES, &tmX, 0, run.seg * FWD_PIX - 1, row_in0 + r, run.z, fb);
          } else {
            const int sub_bytes = (FWD_PIX / pack) * 128;
            mbar_expect_tx(fb, FWD_PIX * 128);
            for (int j = 0; j < pack; ++j)      // a strip index beyond Z reads as zeros
              tma_load_4d(ring + stage * FWD1_ROW_BYTES + j * sub_bytes, &tmX, 0, -1, row_in0 + r, run.z + j, fb);
          }
          if (++stage == FWD1_STAGES) { stage = 0; phase ^= 1u; }
        }
        pos += run.n;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = mbar_wait(smem_u32(&w_bar), 0, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
      int stage = 0;
      uint32_t phase = 0;
      int g0 = 0;              // output rows of earlier runs of this CTA
      for (long long pos = r0; pos < r1 && ok;) {
        const FwdRun run = fwd_run(p, pos, r1);
        if (p.k1) {
          // 1 x 1 layer (the layer that needs no halo, remark after Eq. 7): output row r is the product of input
          // row r with the centre tap alone -- one view (shifted by one pixel: the box starts at pixel -1), N = 64
          for (int r = 0; r < run.n && ok; ++r) {
            const int g = g0 + r, blk = acc_block(g);
            ok = mbar_wait(smem_u32(&acc_empty_bar[blk]), (g >> 3) & 1u, abortp, p.status, DEV_TIMEOUT_MMA_TMEM);
            if (!ok) break;
            ok = mbar_wait(smem_u32(&full_bar[stage]), phase, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
            if (!ok) break;
            tc_fence_after();
            const uint64_t adesc = make_desc(ring + stage * FWD1_ROW_BYTES + 128, 16, 1024);
            const uint64_t bdesc = make_desc(w_smem + 192 * 128 + 64 * 128, 16, 1024);       // tap (u, v) = (1, 1)
            const uint32_t idesc = make_idesc(128, 64, 0, 0);
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_bf16(tmem_base + blk * 64, adesc + k * 2, bdesc + k * 2, idesc, 1u);
            tc_commit(smem_u32(&empty_bar[stage]));
            if (++stage == FWD1_STAGES) { stage = 0; phase ^= 1u; }
            tc_commit(smem_u32(&acc_full_bar[blk]));
          }
          g0 += run.n;
          pos += run.n;
          continue;
        }
        for (int r = 0; r < run.n + 2 && ok; ++r) {
          if (r < run.n) {     // this input row opens output row r: its block must be drained and zeroed
            const int g = g0 + r;
            ok = mbar_wait(smem_u32(&acc_empty_bar[acc_block(g)]), (g >> 3) & 1u, abortp, p.status, DEV_TIMEOUT_MMA_TMEM);
            if (!ok) break;
          }
          ok = mbar_wait(smem_u32(&full_bar[stage]), phase, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          const int u_lo = max(0, r - (run.n - 1)), u_hi = min(2, r);     // taps whose output row r - u exists
          const uint32_t xa = ring + stage * FWD1_ROW_BYTES;
          int u_s = u_lo;
          while (u_s <= u_hi) {
            const int bs = acc_block(g0 + r - u_s);
            int u_e = u_s;
            while (u_e < u_hi && bs + (u_e + 1 - u_s) <= 7) ++u_e;          // stay inside the ring
            const uint32_t idesc = make_idesc(128, 64 * (u_e - u_s + 1), 0, 0);
            const uint32_t d_tmem = tmem_base + bs * 64;
#pragma unroll
            for (int v = 0; v < 3; ++v) {
              // The view shifted by v pixels starts v rows (128 bytes each) into the box.  The 128-byte
              // swizzle is a function of the shared-memory address itself, so the rows of a view are read
              // back exactly as TMA wrote them (checked: bit-identical to three separately loaded copies).
              const uint64_t adesc = make_desc(xa + v * 128, 16, 1024);
              const uint64_t bdesc = make_desc(w_smem + v * (192 * 128) + u_s * (64 * 128), 16, 1024);
#pragma unroll
              for (int k = 0; k < 4; ++k) tc_mma_bf16(d_tmem, adesc + k * 2, bdesc + k * 2, idesc, 1u);
            }
            u_s = u_e + 1;
          }
          tc_commit(smem_u32(&empty_bar[stage]));                           // the row is used only here
          if (++stage == FWD1_STAGES) { stage = 0; phase ^= 1u; }
          if (r >= 2) tc_commit(smem_u32(&acc_full_bar[acc_block(g0 + r - 2)]));   // output row r-2 is complete
        }
        g0 += run.n;
        pos += run.n;
      }
    }
  } else {
    // Eight epilogue warps: warp & 3 selects the TMEM lane quarter (32 pixels), (warp - 2) >> 2 the
    // channel half.  Drain a finished block, zero it for its next use, apply the tail operation.
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int pl = q * 32 + lane;                       // pixel inside the 128-pixel segment
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 32;
    for (int b = 0; b < 8; ++b) {                        // all blocks start out zero and free
      asm volatile(
          "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
          "{%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
          "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
          ::"r"(lane_base + b * 64), "r"(0u) : "memory");
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    tc_fence_before();
    __syncwarp();
    if (lane == 0)
      for (int b = 0; b < 8; ++b) mbar_arrive(smem_u32(&acc_empty_bar[b]));
    int g = 0;
    float ssq = 0.f;
    bool ok = true;
    {
      // ---- TMA epilogue.  The eight warps fill one staging tile per output row segment (a thread owns
      // 32 channels of one pixel: four 16-byte cells of that pixel's 128-byte row, at the cell positions of
      // the 128-byte swizzle), one thread stores the tile with TMA; the mask source of the backward-data
      // mode arrives the same way, two rows ahead.  The LSU never touches global memory (32 sectors per
      // instruction made it the bottleneck of this kernel).
      const uint32_t stg_out = ring + FWD1_STAGES * FWD1_ROW_BYTES;
      const uint32_t stg_mask = stg_out + 2 * FWD_TILE_BYTES;
      uint8_t* out_gen = smem_raw + (stg_out - smem_u32(smem_raw));
      const uint8_t* mask_gen = smem_raw + (stg_mask - smem_u32(smem_raw));
      const bool use_mask = p.mode == MODE_MASK && p.mask_src != nullptr;
      const bool issuer = warp == 2 && lane == 0;
      const int n_rows = static_cast<int>(r1 - r0);
      // Position of an output row in the flattened (strip group, segment, row) space, advanced row by row
      // (no divisions inside the loop): `cur` is the row being drained, `ahead` the one whose mask is loaded.
      struct Pos { int x0, row, z; };
      auto pos_at = [&](long long pos) {
        const long long col = pos / p.nrows;
        Pos q;
        q.z = static_cast<int>(col / p.nseg) * pack;
        q.x0 = static_cast<int>(col % p.nseg) * FWD_PIX;
        q.row = static_cast<int>(pos - col * p.nrows) + p.row_lo;
        return q;
      };
      auto advance = [&](Pos& q) {
        if (++q.row >= p.row_lo + p.nrows) {
          q.row = p.row_lo;
          q.x0 += FWD_PIX;
          if (q.x0 >= p.nseg * FWD_PIX) { q.x0 = 0; q.z += pack; }
        }
      };
      constexpr bool uneven = UNEVEN;
      const int sub = FWD_PIX / pack;                   // tile positions per strip
      const int sub_bytes = sub * 128;
      auto load_mask = [&](int k, const Pos& q) {
        const uint32_t mb = smem_u32(&mask_full_bar[k & 1]);
        mbar_expect_tx(mb, FWD_TILE_BYTES);
        for (int j = 0; j < pack; ++j)
          tma_load_4d(stg_mask + (k & 1) * FWD_TILE_BYTES + j * sub_bytes, &tmMask, 0, q.x0, q.row, q.z + j, mb);
      };
      Pos cur = pos_at(r0), ahead = cur;
      if (use_mask && issuer) {
        if (n_rows > 0) load_mask(0, ahead);
        advance(ahead);
        if (n_rows > 1) load_mask(1, ahead);
        advance(ahead);
      }
      const int cell0 = half * 4;                         // first 16-byte cell of this thread's channels
      const int pl_sub = PACKED ? pl % sub : pl, pl_strip = PACKED ? pl / sub : 0;
      for (; g < n_rows; ++g, advance(cur)) {
        const int buf = g & 1;
        const int x0 = cur.x0, row = cur.row, z = cur.z;
        // (a row beyond its strip's height is the dead row of a short strip: computed, never stored or counted)
        const bool valid = (PACKED ? (pl_sub < p.W && z + pl_strip < p.Z) : x0 + pl < p.W) &&
                           (row < p.Hs || !uneven || row <= strip_height((z + pl_strip) % p.P_r, p.H, p.P_r, p.Hs));
        const int blk = acc_block(g);
        if (issuer) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the store of row g - 2 has read this tile
        asm volatile("bar.sync 1, 256;" ::: "memory");
        ok = mbar_wait(smem_u32(&acc_full_bar[blk]), (g >> 3) & 1u, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        if (ok && use_mask) ok = mbar_wait(smem_u32(&mask_full_bar[buf]), (g >> 1) & 1u, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
          tc_fence_after();
          uint32_t d[32];
          tc_ld32(lane_base + blk * 64, d);
          tc_wait_ld();
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
              "{%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
              "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
              ::"r"(lane_base + blk * 64), "r"(0u) : "memory");
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&acc_empty_bar[blk]));
          float y[32];
#pragma unroll
          for (int c = 0; c < 32; ++c) y[c] = __uint_as_float(d[c]);
          if (p.mode == MODE_RELU_STORE) {
#pragma unroll
            for (int c = 0; c < 32; ++c) y[c] = fmaxf(y[c], 0.f);
          } else if (p.mode == MODE_STORE_SSQ) {
            if (valid) {
#pragma unroll
              for (int c = 0; c < 32; ++c) ssq = fmaf(y[c], y[c], ssq);
            }
          } else if (use_mask) {
            const uint8_t* mrow = mask_gen + buf * FWD_TILE_BYTES + pl * 128;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 mq = *reinterpret_cast<const uint4*>(mrow + (((cell0 + j) ^ (pl & 7)) << 4));
              const uint32_t mw[4] = {mq.x, mq.y, mq.z, mq.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                if (!(bf16_bits_to_f32(mw[e] & 0xFFFFu) > 0.f)) y[j * 8 + 2 * e] = 0.f;
                if (!(bf16_bits_to_f32(mw[e] >> 16) > 0.f)) y[j * 8 + 2 * e + 1] = 0.f;
              }
            }
          }
          uint8_t* orow = out_gen + buf * FWD_TILE_BYTES + pl * 128;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint4 o;
            o.x = pack_bf16x2(y[j * 8 + 0], y[j * 8 + 1]); o.y = pack_bf16x2(y[j * 8 + 2], y[j * 8 + 3]);
            o.z = pack_bf16x2(y[j * 8 + 4], y[j * 8 + 5]); o.w = pack_bf16x2(y[j * 8 + 6], y[j * 8 + 7]);
            *reinterpret_cast<uint4*>(orow + (((cell0 + j) ^ (pl & 7)) << 4)) = o;
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // tile written (and mask tile read) before TMA touches them
        {   // the eight warps meet here: either all of them go on or none does
          int all_ok;
          asm volatile(
              "{\n\t.reg .pred pp, qq;\n\t"
              "setp.ne.b32 pp, %1, 0;\n\t"
              "bar.red.and.pred qq, 1, 256, pp;\n\t"
              "selp.b32 %0, 1, 0, qq;\n\t}"
              : "=r"(all_ok) : "r"(static_cast<int>(ok)) : "memory");
          ok = all_ok != 0;
        }
        if (!ok) break;
        if (issuer) {
          for (int j = 0; j < pack; ++j) {           // one box per strip of the group; all of them in one bulk group
            const int zj = z + j;
            if (zj >= p.Z) break;
            const int hs_j = uneven ? strip_height(zj % p.P_r, p.H, p.P_r, p.Hs) : p.Hs;
            if (uneven && row > hs_j) continue;        // dead row of a short strip
            const uint32_t src = stg_out + buf * FWD_TILE_BYTES + j * sub_bytes;
            asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                         ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(0), "r"(x0), "r"(row), "r"(zj), "r"(src)
                         : "memory");
            // Halo exchange (Section 2.2), fused: the first / last own row of a strip is also the lower / upper
            // halo row of the strip above / below it in the same image.
            if (row == 1 && p.P_r > 1 && zj % p.P_r > 0)
              asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                           ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(0), "r"(x0), "r"(uneven ? strip_height(zj % p.P_r - 1, p.H, p.P_r, p.Hs) + 1 : p.Hs + 1), "r"(zj - 1), "r"(src)
                           : "memory");
            if (row == hs_j && p.P_r > 1 && zj % p.P_r < p.P_r - 1)
              asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                           ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(0), "r"(x0), "r"(0), "r"(zj + 1), "r"(src)
                           : "memory");
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          if (use_mask && g + 2 < n_rows) { load_mask(g + 2, ahead); advance(ahead); }
        }
      }
      if (issuer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores done before the CTA exits
    }
    if (p.mode == MODE_STORE_SSQ) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, o);
      if (lane == 0) {
        float* slot = p.loss_part + blockIdx.x * 8 + (warp - 2);
        *slot = p.loss_add ? *slot + ssq : ssq;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc<512>(tmem_base);
  }
}

// ------------------------------------------------------------------------------ backward-weight kernel
struct WgParams {
  int W, Hs, R, nseg;
  int H, P_r;             // image rows and strips per image (heights of the strips: see strip_height)
  int pack;               // narrow images: strips per 128-pixel block, as in the forward kernel
  int k1;                 // 1 x 1 layer: a dY row meets its own X row only, and only the centre tap is formed
  long long rows_total;   // dY row segments: (strip group z, segment, row) flattened with the row fastest
  float* part;            // [gridDim.x][9][C][C]
  int* status;
};

// As in the forward kernel a CTA owns a contiguous span of the flattened rows and walks it as runs
// of rows of one (strip, segment) column; a run of n dY rows meets n + 2 X rows.
struct WgRun {
  int z, seg, h0, n;
};
__device__ __forceinline__ WgRun wg_run(const WgParams& p, long long pos, long long end) {
  const long long col = pos / p.Hs;
  WgRun r;
  r.h0 = static_cast<int>(pos - col * p.Hs);
  const long long left = end - pos;
  r.n = static_cast<int>(left < p.Hs - r.h0 ? left : p.Hs - r.h0);
  r.seg = static_cast<int>(col % p.nseg);
  r.z = static_cast<int>(col / p.nseg) * p.pack;
  return r;
}

// One X row (one box of 130 pixels, read through three shifted views) meets the up to three dY rows it contributes to in ONE
// instruction: B = [dY_{r-2} | dY_{r-1} | dY_r] (N = 64 per row, rows adjacent in the dY ring), A = (shift 0 | shift 1),
// so tap (u, v <= 1) accumulates in TMEM lanes (v, c) and columns (2 - u, o).  The third shift has only 64 lanes of its
// own: the X rows are taken in PAIRS (r, r + 1; two adjacent ring stages) and one instruction A = (shift 2 of row r |
// shift 2 of row r + 1) meets the four dY rows r-2 .. r+1 (N = 256): lanes 0-63 accumulate tap (u, 2) in column block
// 2 - u, lanes 64-127 in block 3 - u (block 3 of the first half and block 0 of the second are products no tap
// needs), and the epilogue adds the two halves.  Five instructions of 128 x (192, 192, 256) per pair of rows instead
// of four of 128 x 192 with half the lanes of every second one wasted.  An odd last row pairs with a row of zeros.
// The dY ring mirrors its first three slots behind its last one so that a window is always contiguous in shared memory.
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_wgrad_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const WgParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t xfull[WG_XSTAGES], xempty[WG_XSTAGES], yfull[WG_YSTAGES], yempty[WG_YSTAGES];
  __shared__ __align__(8) uint64_t done_bar, init_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t xring = base;                                    // slot = one 130-pixel box of an X row
  const uint32_t yring = base + WG_XSTAGES * WG_XROW_BYTES;       // WG_YSTAGES slots + 2 mirror slots
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < WG_XSTAGES; ++i) { mbar_init(smem_u32(&xfull[i]), 1); mbar_init(smem_u32(&xempty[i]), 1); }
    for (int i = 0; i < WG_YSTAGES; ++i) { mbar_init(smem_u32(&yfull[i]), 1); mbar_init(smem_u32(&yempty[i]), 1); }
    mbar_init(smem_u32(&done_bar), 1);
    mbar_init(smem_u32(&init_bar), 4);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc<512>(smem_u32(&tmem_base_slot));
  if (p.pack > 1 && threadIdx.x >= 64) {
    // packed X stages: the pixel rows behind position 127 (read by the shifted views, written by no box)
    // must be finite, since they meet the zero-filled tail of the dY block in the reduction
    uint8_t* ring_gen = smem_raw + (xring - smem_u32(smem_raw));
    for (int i = threadIdx.x - 64; i < WG_XSTAGES * 64; i += NUM_THREADS - 64)
      *reinterpret_cast<uint4*>(ring_gen + (i >> 6) * WG_XROW_BYTES + WG_PIX * 128 + (i & 63) * 16) = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;
  pdl_trigger();                           // set-up done: the next kernel may be scheduled
  pdl_wait();                              // from here on global memory: earlier kernels must have finished

  const long long r0 = (static_cast<long long>(blockIdx.x) * p.rows_total) / gridDim.x;
  const long long r1 = (static_cast<long long>(blockIdx.x + 1) * p.rows_total) / gridDim.x;

  if (warp == 0) {
    if (lane == 0) {
      const int sub_bytes = (WG_PIX / p.pack) * 128;
      int xs = 0, ys = 0;
      uint32_t xph = 0, yph = 0;
      bool ok = true;
      for (long long pos = r0; pos < r1 && ok;) {
        const WgRun run = wg_run(p, pos, r1);
        pos += run.n;
        const int z = run.z;
        const int x0 = run.seg * WG_PIX;
        // 3 x 3: n dY rows meet n + 2 X rows (from the row above the first one on); 1 x 1: their own n X rows
        const int n_x = p.k1 ? run.n : run.n + 2, xrow0 = p.k1 ? run.h0 + 1 : run.h0;
        auto load_y = [&](int r) {            // dY row r of the run into the next ring slot (and its mirror)
          ok = mbar_wait(smem_u32(&yempty[ys]), yph ^ 1u, abortp, p.status, DEV_TIMEOUT_PRODUCER);
          if (!ok) return;
          const uint32_t fy = smem_u32(&yfull[ys]);
          const bool mirrored = ys < WG_YMIRROR && !p.k1;       // (a 1 x 1 layer reads one dY row at a time: no window)
          mbar_expect_tx(fy, mirrored ? 2 * WG_CHUNK : WG_CHUNK);
          for (int j = 0; j < p.pack; ++j) {     // one box per strip of the group (pixels beyond W and strips beyond Z read as zeros)
            // the dead row of a short strip holds the neighbour's row (it is that strip's halo row): read the all-zero row instead
            const int yrow = run.h0 + r + 1 == p.Hs && strips_uneven(p.H, p.P_r, p.Hs) && p.Hs > strip_height((z + j) % p.P_r, p.H, p.P_r, p.Hs)
                                 ? p.Hs + 1 : run.h0 + r + 1;
            tma_load_4d(yring + ys * WG_CHUNK + j * sub_bytes, &tmY, 0, x0, yrow, z + j, fy);
            if (mirrored) tma_load_4d(yring + (WG_YSTAGES + ys) * WG_CHUNK + j * sub_bytes, &tmY, 0, x0, yrow, z + j, fy);
          }
          if (++ys == WG_YSTAGES) { ys = 0; yph ^= 1u; }
        };
        // one X row into ring stage `stage`, counted on barrier `fb`; row < 0: a row of zeros (a coordinate outside
        // the tensor: TMA fills the box and counts its bytes all the same)
        auto load_x = [&](int stage, int row, uint32_t fb) {
          const int yc = row < 0 ? -8 : row;
          if (p.pack == 1) {
            tma_load_4d(xring + stage * WG_XROW_BYTES, &tmX, 0, x0 - 1, yc, z, fb);
          } else {
            for (int j = 0; j < p.pack; ++j)
              tma_load_4d(xring + stage * WG_XROW_BYTES + j * sub_bytes, &tmX, 0, -1, yc, z + j, fb);
          }
        };
        const int x_bytes = p.pack == 1 ? (WG_PIX + 2) * 128 : WG_PIX * 128;
        if (p.k1) {
          for (int r = 0; r < n_x && ok; ++r) {
            load_y(r);
            if (!ok) break;
            ok = mbar_wait(smem_u32(&xempty[xs]), xph ^ 1u, abortp, p.status, DEV_TIMEOUT_PRODUCER);
            if (!ok) break;
            const uint32_t fb = smem_u32(&xfull[xs]);
            mbar_expect_tx(fb, x_bytes);
            load_x(xs, xrow0 + r, fb);
            if (++xs == WG_XSTAGES) { xs = 0; xph ^= 1u; }
          }
        } else {
          // X rows in pairs: stages (xs, xs + 1) with xs even, both counted on the barrier of stage xs
          for (int r = 0; r < n_x && ok; r += 2) {
            if (r < run.n) load_y(r);
            if (ok && r + 1 < run.n) load_y(r + 1);
            if (!ok) break;
            ok = mbar_wait(smem_u32(&xempty[xs]), xph ^ 1u, abortp, p.status, DEV_TIMEOUT_PRODUCER);
            if (!ok) break;
            const uint32_t fb = smem_u32(&xfull[xs]);
            mbar_expect_tx(fb, 2 * x_bytes);
            load_x(xs, xrow0 + r, fb);
            load_x(xs + 1, r + 1 < n_x ? xrow0 + r + 1 : -1, fb);
            xs += 2;
            if (xs == WG_XSTAGES) { xs = 0; xph ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int xw = 0, yw = 0;            // next slots to wait for
      uint32_t xwph = 0, ywph = 0;
      int y_slot0 = 0;               // ring slot of the current item's dY row 0
      bool ok = mbar_wait(smem_u32(&init_bar), 0, abortp, p.status, DEV_TIMEOUT_MMA_TMEM);   // accumulators zeroed
      tc_fence_after();
      for (long long pos = r0; pos < r1 && ok;) {
        const WgRun run = wg_run(p, pos, r1);
        pos += run.n;
        const int npx = p.pack > 1 ? WG_PIX : min(WG_PIX, p.W - run.seg * WG_PIX);
        const int ksteps = (npx + UMMA_K - 1) / UMMA_K;
        int yhave = 0;
        if (p.k1) {
          // 1 x 1 layer: dY row r meets X row r; the operand (shift 0 | shift 1) carries the centre tap in its upper
          // 64 lanes (the lower ones form a tap that is thrown away), the result sits in column block 1 (u = 1)
          for (int r = 0; r < run.n && ok; ++r) {
            ok = mbar_wait(smem_u32(&yfull[yw]), ywph, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
            if (!ok) break;
            ok = mbar_wait(smem_u32(&xfull[xw]), xwph, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
            if (!ok) break;
            tc_fence_after();
            const uint32_t idesc = make_idesc(128, 64, 1, 1);
            const uint64_t bdesc = make_desc(yring + yw * WG_CHUNK, WG_CHUNK, 1024);
            const uint64_t a01 = make_desc(xring + xw * WG_XROW_BYTES, 128, 1024);
            for (int k = 0; k < ksteps; ++k) tc_mma_bf16(tmem_base + 64, a01 + k * 128, bdesc + k * 128, idesc, 1u);
            tc_commit(smem_u32(&xempty[xw]));
            tc_commit(smem_u32(&yempty[yw]));
            if (++xw == WG_XSTAGES) { xw = 0; xwph ^= 1u; }
            if (++yw == WG_YSTAGES) { yw = 0; ywph ^= 1u; }
          }
          y_slot0 = (y_slot0 + run.n) % WG_YSTAGES;
          continue;
        }
        for (int r = 0; r < run.n + 2 && ok; r += 2) {
          const bool two = r + 1 < run.n + 2;                  // (an odd last row is paired with a row of zeros)
          const int i_top = min(two ? r + 1 : r, run.n - 1);   // last dY row any instruction of this pair reads
          while (yhave <= i_top && ok) {
            ok = mbar_wait(smem_u32(&yfull[yw]), ywph, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
            if (++yw == WG_YSTAGES) { yw = 0; ywph ^= 1u; }
            ++yhave;
          }
          if (!ok) break;
          ok = mbar_wait(smem_u32(&xfull[xw]), xwph, abortp, p.status, DEV_TIMEOUT_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          // The operand shifted by v pixels is the view of the box that starts v pixel rows (128 bytes) in; the
          // two 64-channel chunks of an M = 128 operand are two such views: one pixel row apart (shifts 0 | 1 of one
          // X row, leading offset 128) or one ring stage apart (shift 2 of two X rows, leading offset = the stage size).
          const uint32_t xa = xring + xw * WG_XROW_BYTES;
          for (int h = 0; h < (two ? 2 : 1); ++h) {            // shifts 0 | 1 of X row r + h against its window of dY rows
            const int rr = r + h;
            const int i_hi = min(rr, run.n - 1), i_lo = max(0, rr - 2);
            const int n = i_hi - i_lo + 1;                     // dY rows in the window
            const int b0 = 2 - (rr - i_lo);                    // column block of the first of them
            const uint32_t idesc = make_idesc(128, 64 * n, 1, 1);
            const int ys0 = (y_slot0 + i_lo) % WG_YSTAGES;     // window may run into the mirror slots
            const uint64_t bdesc = make_desc(yring + ys0 * WG_CHUNK, WG_CHUNK, 1024);
            const uint64_t a01 = make_desc(xa + h * WG_XROW_BYTES, 128, 1024);          // lanes: (shift 0 | shift 1) x c
            for (int k = 0; k < ksteps; ++k) tc_mma_bf16(tmem_base + b0 * 64, a01 + k * 128, bdesc + k * 128, idesc, 1u);
          }
          {   // shift 2 of both rows against dY rows r-2 .. r+1: lanes 0-63 block 2 - u, lanes 64-127 block 3 - u
            const int i_lo = max(0, r - 2);
            const int n = i_top - i_lo + 1;
            const int b0 = 2 - (r - i_lo);
            const uint32_t idesc = make_idesc(128, 64 * n, 1, 1);
            const int ys0 = (y_slot0 + i_lo) % WG_YSTAGES;
            const uint64_t bdesc = make_desc(yring + ys0 * WG_CHUNK, WG_CHUNK, 1024);
            const uint64_t a22 = make_desc(xa + 2 * 128, WG_XROW_BYTES, 1024);        // lanes: (row r | row r + 1) shift 2 x c
            for (int k = 0; k < ksteps; ++k) tc_mma_bf16(tmem_base + 256 + b0 * 64, a22 + k * 128, bdesc + k * 128, idesc, 1u);
          }
          tc_commit(smem_u32(&xempty[xw]));
          xw += 2;
          if (xw == WG_XSTAGES) { xw = 0; xwph ^= 1u; }
          // dY rows r - 2 and r - 1 have no later reader
          if (r >= 2) tc_commit(smem_u32(&yempty[(y_slot0 + r - 2) % WG_YSTAGES]));
          if (r >= 1 && r - 1 < run.n) tc_commit(smem_u32(&yempty[(y_slot0 + r - 1) % WG_YSTAGES]));
        }
        y_slot0 = (y_slot0 + run.n) % WG_YSTAGES;
      }
      if (ok) tc_commit(smem_u32(&done_bar));
    }
  } else {
    const int q = warp & 3;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    {   // zero both accumulators (columns 0..191 and 256..511) before the first MMA
      for (int cb = 0; cb < 14; ++cb) {
        const uint32_t col = cb < 6 ? cb * 32 : 256 + (cb - 6) * 32;
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
            "{%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
            "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
            ::"r"(lane_base + col), "r"(0u) : "memory");
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&init_bar));
    }
    bool ok = mbar_wait(smem_u32(&done_bar), 0, abortp, p.status, DEV_TIMEOUT_EPILOGUE);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const int row = q * 32 + lane;                 // TMEM lane: (shift-in-pair, c)
      const int c = row & 63;
      float* dst_base = p.part + static_cast<int64_t>(blockIdx.x) * 9 * C * C;
      // shifts 0 and 1: lanes (v, c), column blocks 2 - u
      for (int blk = 0; blk < 3; ++blk) {
        const int u = 2 - blk, v = row >> 6;
        float* dst = dst_base + ((u * 3 + v) * C + c) * C;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tc_ld32(lane_base + blk * 64 + half * 32, r);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<float4*>(dst + half * 32 + j * 4) =
                make_float4(__uint_as_float(r[j * 4]), __uint_as_float(r[j * 4 + 1]), __uint_as_float(r[j * 4 + 2]),
                            __uint_as_float(r[j * 4 + 3]));
        }
      }
      // shift 2: lanes 64-127 (the second X row of every pair) hand their blocks 3 - u over through shared memory (the
      // rings are idle now: every MMA has completed), lanes 0-63 add them to their blocks 2 - u and store tap (u, 2)
      float* comb = reinterpret_cast<float*>(smem_raw + (xring - smem_u32(smem_raw)));      // [64 c][3 u][64 o] floats, 48 KB
      if (row >= 64 && !p.k1) {                  // (a 1 x 1 layer forms no shift-2 tap: that accumulator is zero)
        for (int u = 0; u < 3; ++u) {
#pragma unroll 1
          for (int half = 0; half < 2; ++half) {
            uint32_t r[32];
            tc_ld32(lane_base + 256 + (3 - u) * 64 + half * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<float4*>(comb + (c * 3 + u) * C + half * 32 + j * 4) =
                  make_float4(__uint_as_float(r[j * 4]), __uint_as_float(r[j * 4 + 1]), __uint_as_float(r[j * 4 + 2]),
                              __uint_as_float(r[j * 4 + 3]));
          }
        }
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");           // the four epilogue warps
      if (row < 64) {
        for (int u = 0; u < 3; ++u) {
          float* dst = dst_base + ((u * 3 + 2) * C + c) * C;
#pragma unroll 1
          for (int half = 0; half < 2; ++half) {
            uint32_t r[32];
            tc_ld32(lane_base + 256 + (2 - u) * 64 + half * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float4 o = p.k1 ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(comb + (c * 3 + u) * C + half * 32 + j * 4);
              *reinterpret_cast<float4*>(dst + half * 32 + j * 4) =
                  make_float4(__uint_as_float(r[j * 4]) + o.x, __uint_as_float(r[j * 4 + 1]) + o.y, __uint_as_float(r[j * 4 + 2]) + o.z,
                              __uint_as_float(r[j * 4 + 3]) + o.w);
            }
          }
        }
      }
    } else {
      asm volatile("bar.sync 2, 128;" ::: "memory");           // (keeps the barrier's count when the wait gave up)
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc<512>(tmem_base);
  }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

cudaError_t conv_init() {
  if (g_encode) return cudaSuccess;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
  if ((e = cudaFuncSetAttribute(conv_fwd_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(conv_fwd_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(conv_fwd_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(conv_fwd_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM)) != cudaSuccess) return e;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return cudaSuccess;
}

// strips tensor [Z][R][W][64] as a 4-D map (c, w, r, z) with a box of `box_w` pixels of one row.
bool make_strip_map(CUtensorMap* tm, const void* base, int W, int R, int64_t Z, int box_w) {
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(R),
                              static_cast<cuuint64_t>(Z)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(C) * 2, static_cast<cuuint64_t>(W) * C * 2,
                                 static_cast<cuuint64_t>(R) * W * C * 2};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(C), static_cast<cuuint32_t>(box_w), 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_weight_map(CUtensorMap* tm, const void* base) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(C), 9 * C};
  const cuuint64_t strides[1] = {C * 2};
  const cuuint32_t box[2] = {C, 192};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct ConvNet {
  int L = 0, H = 0, W = 0, P_r = 1, Hs = 0, R = 0, num_sms = 148, grid = 148;
  int pack = 1;                      // strips per 128-pixel tile (narrow images: 2, 4 or 8)
  int64_t B = 0, Z = 0;
  size_t strip_elems = 0;
  int* status = nullptr;
  cudaStream_t stream = nullptr;
  Profiler* prof = nullptr;
  std::vector<bf16*> act;            // act[0] = staged input, act[i+1] = stored output of layer i
  std::vector<bf16*> dY;             // dY[i]: gradient w.r.t. the output of layer i; dY[L-1] == act[L]
  std::vector<bf16*> K, Wf, Wb;
  std::vector<float*> dK;
  GenConv* gen = nullptr;            // layers these kernels do not cover: every call is forwarded (conv_general.cu)
  // Convolutions split in different ways within one stack (each layer in L_M or L_D on its own, Section 2.4): one general
  // stack per run of layers with the same split, chained through NCHW buffers -- the re-distribution between two
  // distributions of an activation (Eq. 6) -- forward (activations) and backward (gradients)
  struct Seg { GenConv* g; int first, n; bf16* out_nchw; };
  std::vector<Seg> segs;
  std::vector<float*> K32;           // fp32 master weights (empty unless enabled)
  std::vector<float*> Vk;            // momentum: velocities of the kernels (empty unless enabled), canonical [o][c][3][3]
  float mu = 0.f;
  std::vector<int> relu;
  std::vector<int> k1;               // 1 x 1 layer: weights in the centre tap, outer taps zero
  std::vector<CUtensorMap> act_fwd, dY_fwd, dY_wg, wf_map, wb_map;   // act_fwd / dY_fwd: 130-pixel boxes (also the X operand of backward-weight)
  std::vector<CUtensorMap> act_tile, dY_tile;     // [128 pixels][64 channels] boxes: TMA stores of outputs, mask rows
  float* wpart = nullptr;
  float* loss_part = nullptr;
  bf16* scratch_nchw = nullptr;
  int state = 0;                     // 0 idle, 1 forward done, 2 backward (gradients kept), 3 backward (fused)
  bool fc_above = false;             // fully connected layers follow: no loss here, dY of the last layer comes from above
};

namespace {

// row_lo / nrows: the own rows to compute (default: all Hs of them); loss_add: see FwdParams
void launch_fwd(ConvNet* c, int cls, int layer, const CUtensorMap& in, const CUtensorMap& w, bf16* out, const CUtensorMap& out_tile, int mode,
                const bf16* mask, const CUtensorMap* mask_tile, int row_lo = 1, int nrows = -1, int loss_add = 0) {
  FwdParams p;
  if (nrows < 0) nrows = c->Hs;
  if (nrows == 0) return;
  p.row_lo = row_lo; p.nrows = nrows; p.loss_add = loss_add;
  p.W = c->W; p.Hs = c->Hs; p.R = c->R; p.H = c->H;
  p.nseg = (c->W + FWD_PIX - 1) / FWD_PIX;
  p.pack = c->pack; p.Z = static_cast<int>(c->Z); p.P_r = c->P_r;
  p.k1 = c->k1[layer] && !getenv("MBD_CONV_1X1_AS_3X3");       // tuning knob: a 1 x 1 layer through all nine taps
  p.rows_total = ((c->Z + c->pack - 1) / c->pack) * p.nseg * nrows;
  p.mode = mode; p.out = out; p.mask_src = mask; p.loss_part = c->loss_part; p.status = c->status;
  const int grid = p.rows_total < c->grid ? static_cast<int>(p.rows_total) : c->grid;
  if (mode == MODE_STORE_SSQ && !loss_add) cudaMemsetAsync(c->loss_part, 0, sizeof(float) * c->grid * 8, c->stream);
  const double flops = 2.0 * c->B * c->H * c->W * (c->k1[layer] ? 1.0 : 9.0) * C * C * nrows / c->Hs;   // the method's flops, not the kernel's
  c->prof->begin(cls, flops);
  const bool uneven = c->H % c->P_r != 0;
  if (c->pack > 1)
    launch_pdl(uneven ? conv_fwd_kernel<true, true> : conv_fwd_kernel<true, false>, dim3(grid), dim3(FWD_THREADS), FWD_SMEM, c->stream, 1, in, w, out_tile,
               mask_tile ? *mask_tile : out_tile, p);
  else
    launch_pdl(uneven ? conv_fwd_kernel<false, true> : conv_fwd_kernel<false, false>, dim3(grid), dim3(FWD_THREADS), FWD_SMEM, c->stream, 1, in, w, out_tile,
               mask_tile ? *mask_tile : out_tile, p);
  c->prof->end();
}

void launch_stage_in(ConvNet* c, const bf16* nchw, bf16* strips) {
  dim3 g((c->H * c->W + 31) / 32, static_cast<unsigned>(c->B));
  c->prof->begin(MBD_K_HALO, 2.0 * c->B * C * c->H * c->W * 2.0);
  nchw_to_strips_kernel<<<g, 128, 0, c->stream>>>(nchw, strips, c->H, c->W, c->P_r, c->Hs);
  c->prof->end();
}

}  // namespace

namespace {
// how a split kind uses the P_r x P_c grid: strips, batch blocks, groups over the output channels
void kind_grid(int split, int P_r, int P_c, int* strips, int* blocks, int* model_groups) {
  if (split == MBD_SPLIT_BATCH) { *strips = 1; *blocks = P_r * P_c; *model_groups = 1; }        // Section 3's improved case: 1 x P
  else if (split == MBD_SPLIT_MODEL) { *strips = 1; *blocks = P_c; *model_groups = P_r; }       // L_M: Eq. 8
  else { *strips = P_r; *blocks = P_c; *model_groups = 1; }                                     // L_D: Eq. 7
}
// the general stack that holds `layer` (rewritten to its index there); null for the 64-channel kernels
GenConv* gen_of(const ConvNet* c, int* layer, int* seg = nullptr) {
  if (c->gen) return c->gen;
  for (size_t k = 0; k < c->segs.size(); ++k)
    if (*layer >= c->segs[k].first && *layer < c->segs[k].first + c->segs[k].n) {
      *layer -= c->segs[k].first;
      if (seg) *seg = static_cast<int>(k);
      return c->segs[k].g;
    }
  return c->segs.empty() ? nullptr : c->segs.back().g;         // (out of range: the callee reports it)
}
}  // namespace

mbd_status conv_create(const mbd_layer* layers, int L, int64_t B, int P_r_grid, int P_c_grid, int max_partials, int num_sms, int* status,
                       cudaStream_t stream, Profiler* prof, bool fc_above, ConvNet** out) {
  bool uniform = true;
  for (int i = 1; i < L; ++i) uniform = uniform && layers[i].split == layers[0].split;
  if (!uniform) {
    ConvNet* c = new (std::nothrow) ConvNet();
    if (!c) return MBD_E_ALLOC;
    c->L = L; c->B = B; c->stream = stream;
    for (int a = 0; a < L;) {
      int b = a + 1;
      while (b < L && layers[b].split == layers[a].split) ++b;
      int strips, blocks, groups;
      kind_grid(layers[a].split, P_r_grid, P_c_grid, &strips, &blocks, &groups);
      ConvNet::Seg sg{nullptr, a, b - a, nullptr};
      const mbd_status s = gconv_create(layers + a, b - a, B, strips, blocks, max_partials, num_sms, status, stream, prof, b < L ? true : fc_above,
                                        groups, a > 0, a > 0 ? layers[a - 1].relu : 0, &sg.g);
      if (s != MBD_OK) { conv_destroy(c); return s; }
      c->segs.push_back(sg);
      a = b;
    }
    for (size_t k = 0; k + 1 < c->segs.size(); ++k)
      if (cudaMalloc(reinterpret_cast<void**>(&c->segs[k].out_nchw), gconv_input_bytes(c->segs[k + 1].g)) != cudaSuccess) {
        (void)cudaGetLastError();
        conv_destroy(c);
        return MBD_E_ALLOC;
      }
    *out = c;
    return MBD_OK;
  }
  int P_r, P_c, model_P_r;
  kind_grid(layers[0].split, P_r_grid, P_c_grid, &P_r, &P_c, &model_P_r);
  if (gconv_needed(layers, L)) {
    ConvNet* c = new (std::nothrow) ConvNet();
    if (!c) return MBD_E_ALLOC;
    const mbd_status s = gconv_create(layers, L, B, P_r, P_c, max_partials, num_sms, status, stream, prof, fc_above, model_P_r, false, 0, &c->gen);
    if (s != MBD_OK) { delete c; return s; }
    c->L = L; c->B = B;
    *out = c;
    return MBD_OK;
  }
  if (conv_init() != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  const int H = layers[0].H, W = layers[0].W;
  if (B > 65535 || static_cast<int64_t>(H) * W > INT32_MAX) return MBD_E_UNSUPPORTED;   // grid.y of the staging kernels
  if ((static_cast<int64_t>(H) + 1) * P_r > INT32_MAX) return MBD_E_UNSUPPORTED;               // 32-bit strip arithmetic in the kernels
  ConvNet* c = new (std::nothrow) ConvNet();
  if (!c) return MBD_E_ALLOC;
  c->L = L; c->B = B; c->H = H; c->W = W; c->P_r = P_r; c->Hs = (H + P_r - 1) / P_r; c->R = c->Hs + 2; c->Z = B * P_r;
  c->num_sms = num_sms; c->grid = num_sms; c->status = status; c->stream = stream; c->prof = prof;
  c->fc_above = fc_above;
  c->strip_elems = static_cast<size_t>(c->Z) * c->R * W * C;
  auto alloc = [&](void** p, size_t bytes) -> bool {
    if (cudaMalloc(p, bytes) != cudaSuccess) { (void)cudaGetLastError(); *p = nullptr; return false; }
    return cudaMemsetAsync(*p, 0, bytes, stream) == cudaSuccess;
  };
  bool ok = true;
  c->act.assign(L + 1, nullptr); c->dY.assign(L, nullptr);
  c->K.assign(L, nullptr); c->Wf.assign(L, nullptr); c->Wb.assign(L, nullptr); c->dK.assign(L, nullptr);
  c->relu.resize(L);
  c->k1.resize(L);
  for (int i = 0; i <= L && ok; ++i) ok = alloc(reinterpret_cast<void**>(&c->act[i]), c->strip_elems * 2);
  for (int i = 0; i < L && ok; ++i) {
    c->relu[i] = layers[i].relu;
    c->k1[i] = layers[i].kh == 1;
    if (i < L - 1 || fc_above) ok = alloc(reinterpret_cast<void**>(&c->dY[i]), c->strip_elems * 2);
    else c->dY[i] = c->act[L];                       // half-SSQ loss: dY_L = Y_L
    ok = ok && alloc(reinterpret_cast<void**>(&c->K[i]), 9 * C * C * 2) && alloc(reinterpret_cast<void**>(&c->Wf[i]), 9 * C * C * 2) &&
         alloc(reinterpret_cast<void**>(&c->Wb[i]), 9 * C * C * 2) && alloc(reinterpret_cast<void**>(&c->dK[i]), 9 * C * C * 4);
  }
  ok = ok && alloc(reinterpret_cast<void**>(&c->wpart), static_cast<size_t>(c->grid) * 9 * C * C * 4);
  ok = ok && alloc(reinterpret_cast<void**>(&c->loss_part), sizeof(float) * c->grid * 8);
  ok = ok && alloc(reinterpret_cast<void**>(&c->scratch_nchw), static_cast<size_t>(B) * C * H * W * 2);
  if (!ok) { conv_destroy(c); return MBD_E_ALLOC; }
  // narrow images: as many strips per 128-pixel tile as fit with their two border pixels
  c->pack = W + 2 <= 16 ? 8 : W + 2 <= 32 ? 4 : W + 2 <= 64 ? 2 : 1;
  if (getenv("MBD_CONV_NO_PACK")) c->pack = 1;       // tuning knob
  if (c->Z > INT32_MAX - 8) { conv_destroy(c); return MBD_E_UNSUPPORTED; }
  const int sub = FWD_PIX / c->pack;
  const int fwd_box = c->pack > 1 ? sub : FWD1_BOX_PIX;
  const int tile_box = c->pack > 1 ? sub : FWD_PIX;
  c->act_fwd.resize(L + 1); c->dY_fwd.resize(L); c->dY_wg.resize(L);
  c->act_tile.resize(L + 1); c->dY_tile.resize(L);
  c->wf_map.resize(L); c->wb_map.resize(L);
  for (int i = 0; i <= L && ok; ++i)
    ok = make_strip_map(&c->act_fwd[i], c->act[i], W, c->R, c->Z, fwd_box) && make_strip_map(&c->act_tile[i], c->act[i], W, c->R, c->Z, tile_box);
  for (int i = 0; i < L && ok; ++i)
    ok = make_strip_map(&c->dY_fwd[i], c->dY[i], W, c->R, c->Z, fwd_box) && make_strip_map(&c->dY_wg[i], c->dY[i], W, c->R, c->Z, tile_box) &&
         make_strip_map(&c->dY_tile[i], c->dY[i], W, c->R, c->Z, tile_box) &&
         make_weight_map(&c->wf_map[i], c->Wf[i]) && make_weight_map(&c->wb_map[i], c->Wb[i]);
  if (!ok) { conv_destroy(c); return MBD_E_CUDA; }
  if (cudaStreamSynchronize(stream) != cudaSuccess) { conv_destroy(c); return MBD_E_CUDA; }
  *out = c;
  return MBD_OK;
}

void conv_destroy(ConvNet* c) {
  if (c && c->gen) { gconv_destroy(c->gen); delete c; return; }
  if (c && !c->segs.empty()) {
    for (ConvNet::Seg& sg : c->segs) { gconv_destroy(sg.g); cudaFree(sg.out_nchw); }
    (void)cudaGetLastError();
    delete c;
    return;
  }
  if (!c) return;
  for (size_t i = 0; i < c->act.size(); ++i) cudaFree(c->act[i]);
  for (int i = 0; i < c->L; ++i)
    if (c->dY[i] != c->act[c->L]) cudaFree(c->dY[i]);
  for (int i = 0; i < c->L; ++i) { cudaFree(c->K[i]); cudaFree(c->Wf[i]); cudaFree(c->Wb[i]); cudaFree(c->dK[i]); }
  for (float* m : c->K32) cudaFree(m);
  for (float* m : c->Vk) cudaFree(m);
  cudaFree(c->wpart); cudaFree(c->loss_part); cudaFree(c->scratch_nchw);
  (void)cudaGetLastError();
  delete c;
}

namespace {
mbd_status launch_pack(ConvNet* c, int layer) {
  c->prof->begin(MBD_K_OTHER, 9.0 * C * C * 6.0);
  pack_weights_kernel<<<(9 * C * C + 255) / 256, 256, 0, c->stream>>>(c->K[layer], c->Wf[layer], c->Wb[layer]);
  c->prof->end();
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}
}  // namespace

mbd_status conv_set_weights(ConvNet* c, int layer, const void* K_dev) {
  if (GenConv* g = gen_of(c, &layer)) return gconv_set_weights(g, layer, K_dev);
  if (c->k1[layer]) {
    embed_1x1_kernel<<<(9 * C * C + 255) / 256, 256, 0, c->stream>>>(static_cast<const bf16*>(K_dev), c->K[layer]);
    if (cudaGetLastError() != cudaSuccess) return MBD_E_CUDA;
  } else if (cudaMemcpyAsync(c->K[layer], K_dev, 9 * C * C * 2, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) {
    return MBD_E_CUDA;
  }
  if (!c->K32.empty() && widen_bf16_launch(c->K[layer], c->K32[layer], 9 * C * C, c->num_sms, c->stream) != cudaSuccess) return MBD_E_CUDA;
  return launch_pack(c, layer);
}

mbd_status conv_enable_master(ConvNet* c) {
  if (c->gen) return gconv_enable_master(c->gen);
  if (!c->segs.empty()) {
    for (ConvNet::Seg& sg : c->segs) { const mbd_status st = gconv_enable_master(sg.g); if (st != MBD_OK) return st; }
    return MBD_OK;
  }
  if (!c->K32.empty()) return MBD_OK;
  std::vector<float*> m(c->L, nullptr);
  for (int i = 0; i < c->L; ++i) {
    if (cudaMalloc(reinterpret_cast<void**>(&m[i]), 9 * C * C * 4) != cudaSuccess ||
        widen_bf16_launch(c->K[i], m[i], 9 * C * C, c->num_sms, c->stream) != cudaSuccess) {
      (void)cudaGetLastError();
      for (float* q : m) cudaFree(q);
      return MBD_E_ALLOC;
    }
  }
  c->K32 = m;
  return MBD_OK;
}

mbd_status conv_enable_momentum(ConvNet* c, float mu) {
  if (c->gen) return gconv_enable_momentum(c->gen, mu);
  if (!c->segs.empty()) {
    for (ConvNet::Seg& sg : c->segs) { const mbd_status st = gconv_enable_momentum(sg.g, mu); if (st != MBD_OK) return st; }
    return MBD_OK;
  }
  if (c->Vk.empty()) {
    std::vector<float*> v(c->L, nullptr);
    for (int i = 0; i < c->L; ++i) {
      if (cudaMalloc(reinterpret_cast<void**>(&v[i]), 9 * C * C * 4) != cudaSuccess) {
        (void)cudaGetLastError();
        for (float* q : v) cudaFree(q);
        return MBD_E_ALLOC;
      }
    }
    c->Vk = v;
  }
  for (int i = 0; i < c->L; ++i)
    if (cudaMemsetAsync(c->Vk[i], 0, 9 * C * C * 4, c->stream) != cudaSuccess) return MBD_E_CUDA;
  c->mu = mu;
  return MBD_OK;
}

namespace {
// momentum update of layer i from its materialised gradient, then the two operand layouts of the new weights
mbd_status momentum_update(ConvNet* c, int i, float eta) {
  c->prof->begin(MBD_K_SGD, 9.0 * C * C * 14.0);
  const cudaError_t e = sgd_momentum_update_launch(c->K[i], 1, c->K32.empty() ? nullptr : c->K32[i], c->Vk[i], c->dK[i], 9 * C * C, c->mu,
                                                   1.f / static_cast<float>(c->B), eta, c->num_sms, c->stream);
  c->prof->end();
  if (e != cudaSuccess) return MBD_E_CUDA;
  return launch_pack(c, i);
}
}  // namespace

mbd_status conv_get_weights(ConvNet* c, int layer, void* K_dev) {
  if (GenConv* g = gen_of(c, &layer)) return gconv_get_weights(g, layer, K_dev);
  if (c->k1[layer]) {
    extract_1x1_kernel<bf16><<<(C * C + 255) / 256, 256, 0, c->stream>>>(c->K[layer], static_cast<bf16*>(K_dev));
    return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
  }
  if (cudaMemcpyAsync(K_dev, c->K[layer], 9 * C * C * 2, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) return MBD_E_CUDA;
  return MBD_OK;
}

size_t conv_input_bytes(const ConvNet* c) {
  if (!c->segs.empty()) return gconv_input_bytes(c->segs[0].g);
  return c->gen ? gconv_input_bytes(c->gen) : static_cast<size_t>(c->B) * C * c->H * c->W * 2;
}

// The step, piece by piece (a multi-process driver exchanges the image's outer halo rows between the pieces;
// conv_forward / conv_backward below are these pieces in a row).
mbd_status conv_stage_input(ConvNet* c, const void* X_nchw) {
  if (c->gen) return gconv_stage_input(c->gen, X_nchw);
  if (!c->segs.empty()) return gconv_stage_input(c->segs[0].g, X_nchw);
  // the input goes into strips (with the halo rows between its own strips); the operand layouts of the weights
  // are kept current by whatever changes the weights (conv_set_weights, the fused update, conv_sgd_step)
  launch_stage_in(c, static_cast<const bf16*>(X_nchw), c->act[0]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

namespace {
// Section 2.2: "the halo exchange can be overlapped with the interior computation".  With one strip per network
// (a process of a multi-process driver) the rows 2 .. Hs - 1 of a 3 x 3 layer's output read no halo row: they
// are the interior, computable while the halo rows travel; rows 1 and Hs are the boundary.  A 1 x 1 layer reads
// no halo at all: all of its rows are interior.  Calls `launch(row_lo, nrows, first)` for the ranges of `rows`.
template <typename F>
void for_rows(const ConvNet* c, int layer, int rows, F launch) {
  const int Hs = c->Hs;
  if (rows == MBD_ROWS_ALL) { launch(1, Hs, true); return; }
  if (c->k1[layer]) {
    if (rows == MBD_ROWS_INTERIOR) launch(1, Hs, true);
    return;
  }
  if (rows == MBD_ROWS_INTERIOR) {
    if (Hs > 2) launch(2, Hs - 2, true);
  } else {
    launch(1, 1, Hs <= 2);                     // with no interior rows the boundary launch is the first one
    if (Hs > 1) launch(Hs, 1, false);
  }
}
}  // namespace

mbd_status conv_forward_layer(ConvNet* c, int i, float* loss_sum_dev, int rows) {
  if (c->gen) return rows == MBD_ROWS_ALL ? gconv_forward_layer(c->gen, i, loss_sum_dev) : MBD_E_UNSUPPORTED;
  if (!c->segs.empty()) {
    if (rows != MBD_ROWS_ALL) return MBD_E_UNSUPPORTED;
    if (i < 0 || i >= c->L) return MBD_E_INVALID;
    int k = 0, j = i;
    GenConv* g = gen_of(c, &j, &k);
    if (j == 0 && k > 0) {       // the output of the run below, re-distributed: out of its layout into NCHW, from there into this run's
      mbd_status st = gconv_output_to_nchw(c->segs[k - 1].g, c->segs[k - 1].out_nchw);
      if (st == MBD_OK) st = gconv_stage_input(g, c->segs[k - 1].out_nchw);
      if (st != MBD_OK) return st;
    }
    return gconv_forward_layer(g, j, loss_sum_dev);
  }
  if (i < 0 || i >= c->L) return MBD_E_INVALID;
  if (rows != MBD_ROWS_ALL && (c->P_r != 1 || (rows != MBD_ROWS_INTERIOR && rows != MBD_ROWS_BOUNDARY))) return MBD_E_UNSUPPORTED;
  const bool last = i == c->L - 1;
  // forward halo exchange (first halo term of Eq. 7): the kernel that produced act[i] (or the staging pass,
  // for the network input) has already stored its boundary rows into the neighbouring strips' halo rows
  const int mode = (last && !c->fc_above) ? MODE_STORE_SSQ : (c->relu[i] ? MODE_RELU_STORE : MODE_MASK);
  for_rows(c, i, rows, [&](int row_lo, int nrows, bool first) {
    launch_fwd(c, MBD_K_CONV_FWD, i, c->act_fwd[i], c->wf_map[i], c->act[i + 1], c->act_tile[i + 1], mode, nullptr, nullptr,
               row_lo, nrows, first ? 0 : 1);          // a later launch of the same layer adds to the loss partials
  });
  if (rows == MBD_ROWS_INTERIOR) return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;   // the boundary rows complete the layer
  if (last && loss_sum_dev && !c->fc_above) {
    c->prof->begin(MBD_K_OTHER, c->grid * 32.0);
    if (sum_f32_launch(c->loss_part, c->grid * 8, 0.5f, loss_sum_dev, c->stream) != cudaSuccess) return MBD_E_CUDA;
    c->prof->end();
  }
  if (cudaGetLastError() != cudaSuccess) return MBD_E_CUDA;
  if (last) c->state = 1;
  return MBD_OK;
}

mbd_status conv_forward(ConvNet* c, const void* X_nchw, float* loss_sum_dev) {
  if (c->gen) return gconv_forward(c->gen, X_nchw, loss_sum_dev);      // (a stack of several runs goes layer by layer, below)
  mbd_status s = conv_stage_input(c, X_nchw);
  for (int i = 0; i < c->L && s == MBD_OK; ++i) s = conv_forward_layer(c, i, loss_sum_dev, MBD_ROWS_ALL);
  return s;
}

mbd_status conv_backward_layer(ConvNet* c, int i, float fused_eta, int rows) {
  if (c->gen) return rows == MBD_ROWS_ALL ? gconv_backward_layer(c->gen, i, fused_eta) : MBD_E_UNSUPPORTED;
  if (!c->segs.empty()) {
    if (rows != MBD_ROWS_ALL) return MBD_E_UNSUPPORTED;
    if (i < 0 || i >= c->L) return MBD_E_INVALID;
    int k = 0, j = i;
    GenConv* g = gen_of(c, &j, &k);
    mbd_status st = gconv_backward_layer(g, j, fused_eta);
    if (st == MBD_OK && j == 0 && k > 0) {       // the gradient w.r.t. this run's input goes back to the run below the same way
      st = gconv_input_grad_to_nchw(g, c->segs[k - 1].out_nchw);
      if (st == MBD_OK) st = gconv_top_grad_from_nchw(c->segs[k - 1].g, c->segs[k - 1].out_nchw);
    }
    return st;
  }
  if (i < 0 || i >= c->L) return MBD_E_INVALID;
  if (rows != MBD_ROWS_ALL && (c->P_r != 1 || (rows != MBD_ROWS_INTERIOR && rows != MBD_ROWS_BOUNDARY))) return MBD_E_UNSUPPORTED;
  const bool momentum = !c->Vk.empty();
  const bool fused = fused_eta > 0.f && !momentum;       // momentum: the gradient first, then the update kernel
  const float scale = -fused_eta / static_cast<float>(c->B);
  if (i > 0) {
    // backward halo exchange (second halo term of Eq. 7), then dY_{i-1} = convT(K_i, dY_i) * [X_i > 0]
    // (the producer of dY_i has stored its boundary rows into the neighbours' halo rows)
    for_rows(c, i, rows, [&](int row_lo, int nrows, bool) {
      launch_fwd(c, MBD_K_CONV_BWD_DATA, i, c->dY_fwd[i], c->wb_map[i], c->dY[i - 1], c->dY_tile[i - 1], MODE_MASK,
                 c->relu[i - 1] ? c->act[i] : nullptr, c->relu[i - 1] ? &c->act_tile[i] : nullptr, row_lo, nrows);
    });
  }
  if (rows == MBD_ROWS_INTERIOR) return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;   // the weight gradient follows the boundary rows
  WgParams p;
  p.W = c->W; p.Hs = c->Hs; p.R = c->R; p.H = c->H; p.P_r = c->P_r;
  p.nseg = (c->W + WG_PIX - 1) / WG_PIX;
  p.pack = c->pack;
  p.k1 = c->k1[i] && !getenv("MBD_CONV_1X1_AS_3X3");
  p.rows_total = ((c->Z + c->pack - 1) / c->pack) * p.nseg * c->Hs;
  p.part = c->wpart; p.status = c->status;
  const int grid = p.rows_total < c->grid ? static_cast<int>(p.rows_total) : c->grid;
  c->prof->begin(MBD_K_CONV_BWD_WEIGHT, 2.0 * c->B * c->H * c->W * (c->k1[i] ? 1.0 : 9.0) * C * C);
  launch_pdl(conv_wgrad_kernel, dim3(grid), dim3(NUM_THREADS), WG_SMEM, c->stream, 1, c->act_fwd[i], c->dY_wg[i], p);
  c->prof->end();
  c->prof->begin(MBD_K_REDUCE, (grid + 1.0) * 9 * C * C * 4.0);
  wgrad_finish_kernel<<<9 * C * C / 64, 256, 0, c->stream>>>(c->wpart, grid, fused ? nullptr : c->dK[i],
                                                                    fused ? c->K[i] : nullptr, c->Wf[i], c->Wb[i],
                                                                    c->K32.empty() ? nullptr : c->K32[i], scale, c->k1[i]);
  c->prof->end();
  if (cudaGetLastError() != cudaSuccess) return MBD_E_CUDA;
  if (momentum && fused_eta > 0.f && momentum_update(c, i, fused_eta) != MBD_OK) return MBD_E_CUDA;
  if (i == 0) c->state = fused_eta > 0.f ? 3 : 2;
  return MBD_OK;
}

mbd_status conv_backward(ConvNet* c, float fused_eta) {
  if (c->gen) return gconv_backward(c->gen, fused_eta);      // (a stack of several runs goes layer by layer, below)
  mbd_status s = MBD_OK;
  for (int i = c->L - 1; i >= 0 && s == MBD_OK; --i) s = conv_backward_layer(c, i, fused_eta, MBD_ROWS_ALL);
  return s;
}

// The outer rows of every image: its first / last own row (what a neighbouring process needs as a halo row) is
// read out, or its upper / lower halo row (zero unless a neighbour supplies it) is written.  `side` 0 = top,
// 1 = bottom; the row buffer is [B][W][C] bf16.  which / layer as in conv_get_tensor; layer -1 = the staged input.
mbd_status conv_outer_rows(ConvNet* c, int which, int layer, int side, void* rows, size_t bytes, int set) {
  if (c->gen || !c->segs.empty()) return MBD_E_UNSUPPORTED;
  if (layer < -1 || layer >= c->L || (side != 0 && side != 1)) return MBD_E_INVALID;
  if (bytes != static_cast<size_t>(c->B) * c->W * C * 2) return MBD_E_INVALID;
  bf16* buf = which == MBD_T_ACT ? c->act[layer + 1] : (which == MBD_T_DY && layer >= 0) ? c->dY[layer] : nullptr;
  if (!buf) return MBD_E_INVALID;
  const int strip = side == 0 ? 0 : c->P_r - 1;
  const int hs_last = strip_height(c->P_r - 1, c->H, c->P_r);      // the bottom strip may be shorter than the row slots
  const int row = set ? (side == 0 ? 0 : hs_last + 1) : (side == 0 ? 1 : hs_last);
  const int per_image = c->W * C / 8;                       // 16-byte pieces per row
  dim3 g((per_image + 255) / 256, static_cast<unsigned>(c->B));
  outer_rows_kernel<<<g, 256, 0, c->stream>>>(buf, static_cast<bf16*>(rows), c->W, c->P_r, c->R, strip, row, set);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status conv_get_product(const ConvNet* c, int layer, int product, const TcGemm** out) {
  if (const GenConv* g = gen_of(c, &layer)) return gconv_get_product(g, layer, product, out);
  return MBD_E_UNSUPPORTED;
}

mbd_status conv_set_dw(ConvNet* c, int layer, const void* src, size_t bytes) {
  if (GenConv* g = gen_of(c, &layer)) return gconv_set_dw(g, layer, src, bytes);
  if (layer < 0 || layer >= c->L) return MBD_E_INVALID;
  if (c->k1[layer]) {
    if (bytes != C * C * 4) return MBD_E_INVALID;
    embed_1x1_f32_kernel<<<(9 * C * C + 255) / 256, 256, 0, c->stream>>>(static_cast<const float*>(src), c->dK[layer]);
    return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
  }
  if (bytes != 9 * C * C * 4) return MBD_E_INVALID;
  return cudaMemcpyAsync(c->dK[layer], src, bytes, cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status conv_sgd_step(ConvNet* c, float eta) {
  if (c->gen) return gconv_sgd_step(c->gen, eta);
  if (!c->segs.empty()) {
    for (ConvNet::Seg& sg : c->segs) { const mbd_status st = gconv_sgd_step(sg.g, eta); if (st != MBD_OK) return st; }
    return MBD_OK;
  }
  const float scale = -eta / static_cast<float>(c->B);
  for (int i = 0; i < c->L; ++i) {
    if (!c->Vk.empty()) {
      if (momentum_update(c, i, eta) != MBD_OK) return MBD_E_CUDA;
      continue;
    }
    c->prof->begin(MBD_K_SGD, 9.0 * C * C * 8.0);
    const cudaError_t e = c->K32.empty() ? sgd_update_launch(c->K[i], 1, c->dK[i], 9 * C * C, scale, c->num_sms, c->stream)
                                         : sgd_master_update_launch(c->K32[i], c->K[i], c->dK[i], 9 * C * C, scale, c->num_sms, c->stream);
    if (e != cudaSuccess) return MBD_E_CUDA;
    c->prof->end();
    if (launch_pack(c, i) != MBD_OK) return MBD_E_CUDA;
  }
  return MBD_OK;
}

// Between the domain-parallel and the model-parallel layers (Section 2.4): the strips of the last
// convolution's output become the [B, C*H*W] matrix (NCHW order) the first fully connected layer reads,
// and that layer's input gradient goes back into strips, its boundary rows also into the neighbours' halos.
mbd_status conv_output_to_nchw(ConvNet* c, void* dst) {
  if (c->gen) return gconv_output_to_nchw(c->gen, dst);
  if (!c->segs.empty()) return gconv_output_to_nchw(c->segs.back().g, dst);
  dim3 g((c->H * c->W + 31) / 32, static_cast<unsigned>(c->B));
  c->prof->begin(MBD_K_HALO, 2.0 * c->B * C * c->H * c->W * 2.0);
  strips_to_nchw_kernel<<<g, 128, 0, c->stream>>>(c->act[c->L], static_cast<bf16*>(dst), c->H, c->W, c->P_r, c->Hs);
  c->prof->end();
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status conv_top_grad_from_nchw(ConvNet* c, const void* src) {
  if (c->gen) return gconv_top_grad_from_nchw(c->gen, src);
  if (!c->segs.empty()) return gconv_top_grad_from_nchw(c->segs.back().g, src);
  if (!c->fc_above) return MBD_E_STATE;
  launch_stage_in(c, static_cast<const bf16*>(src), c->dY[c->L - 1]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

int conv_last_relu(const ConvNet* c) {
  if (!c->segs.empty()) return gconv_last_relu(c->segs.back().g);
  return c->gen ? gconv_last_relu(c->gen) : c->relu[c->L - 1];
}

mbd_status conv_get_tensor(ConvNet* c, int which, int layer, void* dst, size_t bytes) {
  if (GenConv* g = gen_of(c, &layer)) return gconv_get_tensor(g, which, layer, dst, bytes);
  const size_t nchw_bytes = conv_input_bytes(c);
  if (which == MBD_T_DW || which == MBD_T_MASTER || which == MBD_T_VELOCITY) {
    if (layer < 0 || layer >= c->L) return MBD_E_INVALID;
    if (which == MBD_T_MASTER && c->K32.empty()) return MBD_E_STATE;
    if (which == MBD_T_VELOCITY && c->Vk.empty()) return MBD_E_STATE;
    const float* src32 = which == MBD_T_DW ? c->dK[layer] : which == MBD_T_MASTER ? c->K32[layer] : c->Vk[layer];
    if (c->k1[layer]) {
      if (bytes != C * C * 4) return MBD_E_INVALID;
      extract_1x1_kernel<float><<<(C * C + 255) / 256, 256, 0, c->stream>>>(src32, static_cast<float*>(dst));
      return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
    }
    if (bytes != 9 * C * C * 4) return MBD_E_INVALID;
    if (cudaMemcpyAsync(dst, src32, bytes, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) return MBD_E_CUDA;
    return MBD_OK;
  }
  if (which == MBD_T_PARTIALS) {
    if (bytes > static_cast<size_t>(c->grid) * 9 * C * C * 4) return MBD_E_INVALID;
    if (cudaMemcpyAsync(dst, c->wpart, bytes, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) return MBD_E_CUDA;
    return MBD_OK;
  }
  if (layer < 0 || layer >= c->L || bytes != nchw_bytes) return MBD_E_INVALID;
  const bf16* src = which == MBD_T_ACT ? c->act[layer + 1] : which == MBD_T_DY ? c->dY[layer] : nullptr;
  if (!src) return MBD_E_INVALID;
  dim3 g((c->H * c->W + 31) / 32, static_cast<unsigned>(c->B));
  strips_to_nchw_kernel<<<g, 128, 0, c->stream>>>(src, static_cast<bf16*>(dst), c->H, c->W, c->P_r, c->Hs);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status conv_set_tensor(ConvNet* c, int which, int layer, const void* src, size_t bytes) {
  {
    int k = -1, local = layer;
    if (GenConv* g = gen_of(c, &local, &k)) {
      const mbd_status st = gconv_set_tensor(g, which, local, src, bytes);
      // the last activation of a run of layers is also the staged input of the next run: it follows what was set
      if (st == MBD_OK && which == MBD_T_ACT && k >= 0 && k + 1 < static_cast<int>(c->segs.size()) && local == c->segs[k].n - 1)
        return gconv_stage_input(c->segs[k + 1].g, src);
      return st;
    }
  }
  if (layer < 0 || layer >= c->L || bytes != conv_input_bytes(c)) return MBD_E_INVALID;
  bf16* dst = which == MBD_T_ACT ? c->act[layer + 1] : which == MBD_T_DY ? c->dY[layer] : nullptr;
  if (!dst) return MBD_E_INVALID;
  dim3 g((c->H * c->W + 31) / 32, static_cast<unsigned>(c->B));
  nchw_to_strips_kernel<<<g, 128, 0, c->stream>>>(static_cast<const bf16*>(src), dst, c->H, c->W, c->P_r, c->Hs);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

}  // namespace mbd
