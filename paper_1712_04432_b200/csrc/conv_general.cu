// General domain-parallel convolution layers (Section 2.2 / 2.4): any odd k_h x k_w up to 11 x 11, stride 1 to 4, zero
// padding floor(k/2), C_in and C_out multiples of 8, row strips with floor(k_h/2) halo rows.  The layers with 64
// channels and 3 x 3 / 1 x 1 kernels have kernels of their own (conv.cu); everything else runs here, on the
// tensor-core contraction kernel of the fully connected layers (gemm_tc.cu) fed with shifted views.
//
// Layout.  Every activation / gradient tensor is pixel-major with its zero padding stored:
//     T[z][r][x][c],  z = b P_r + s (image b, strip s),  r in [0, Hs + 2 ph),  x in [0, W + 2 pw),  c in [0, C)
// ph, pw = the largest floor(k_h/2), floor(k_w/2) of the network.  Rows ph .. ph+Hs-1 and columns pw .. pw+W-1 are
// the strip's own pixels; the other columns are zero; the other rows are the halo rows -- copies of the
// neighbouring strips' boundary rows (the halo exchange of Section 2.2, here a copy kernel), zero where the image
// ends.  With p the flattened pixel index (z, r, x), tap (u, v) of a layer reads pixel p + (u - kh/2) Wp + (v - kw/2):
// a convolution is a contraction over (tap, channel) whose operand tiles are row-shifted views of ONE 2-D tensor
// [pixels][channels] -- no patch matrix is ever formed.  The products compute every pixel position, padding
// included (a few per cent of extra rows); a small kernel then restores the zeros and the halo rows.
//     forward         Y[p][o]      = sum_{t,c} X[p + off_t][c] Wm[o][t][c]
//     backward-data   dX[p][c]     = sum_{t,o} dY[p - off_t][o] Wm[o][t][c]        (then the ReLU mask)
//     backward-weight dWm[o][t][c] = sum_p dY[p][o] X[p + off_t][c]   (dY zero outside the strips' own pixels)
// Wm[o][t][c] is the kernel K[o][c][u][v] with t = u k_w + v and the channel index padded to a multiple of 64 (zero
// weights, which stay zero: their gradient is a sum of zero-filled operand columns).  The weight gradient is a
// contraction over ALL pixels: its K range is cut by the planner into enough pieces to fill the SMs, the grid's
// S = min(P, max_partials) partial sums being the first cut.
#include "conv_general.h"

#include <algorithm>
#include <cstdlib>
#include <new>
#include <vector>

namespace mbd {

typedef __nv_bfloat16 bf16;

namespace {

struct Geo {
  int B, H, W, P_r, Hs, R, Wp, ph, pw;
  long long Z, Ptot;
};

// ------------------------------------------------------------------------------ layout kernels
// NCHW <-> pixel-major (own pixels only; padding and halos are the business of pad_fix_kernel).  A block moves a
// tile of 32 rows x 32 pixels of 32-bit words through shared memory, a row being one PAIR of channels of a run of 32
// consecutive pixels of one image (pixels counted through the image, h * W + w: a channel plane is contiguous in
// NCHW), so that both sides are accessed 16 bytes at a time -- 8 pixels of a channel on the NCHW side, 8 channels of a
// pixel on the pixel-major side -- and shared memory holds whole words at an odd pitch (no bank conflicts in either
// phase).  With 64 channels or more the rows are the 32 pairs of 64 channels of one run; with fewer (cpb = C < 64
// channels per block) they are the pairs of G = 64 / cpb runs, so that a block still moves about 4 KB (an 8-channel
// input tensor: 256 pixels per block instead of 32).  grid = (ceil(H W / (32 G)), B, ceil(C / cpb)), 128 threads.
struct StageTile {
  int cpb, G;                        // channels per block (a multiple of 8, at most 64), pixel runs per block
};
__host__ __device__ inline StageTile stage_tile(int C) {
  StageTile t;
  t.cpb = C < 64 ? C : 64;
  t.G = 64 / t.cpb;
  return t;
}
// Strips of an image: the balanced ranges [floor(s H / P_r), floor((s + 1) H / P_r)) -- heights differ by at most one row;
// every strip has Hs = ceil(H / P_r) row slots, and a shorter strip's last slot is a dead row (zero, like the padding).
__host__ __device__ __forceinline__ bool geo_ragged(const Geo& g) { return g.Hs * g.P_r != g.H; }
__host__ __device__ __forceinline__ int geo_first(const Geo& g, int s) {
  return !geo_ragged(g) ? s * g.Hs : static_cast<int>((static_cast<long long>(s) * g.H) / g.P_r);
}
__host__ __device__ __forceinline__ int geo_height(const Geo& g, int s) { return !geo_ragged(g) ? g.Hs : geo_first(g, s + 1) - geo_first(g, s); }
__host__ __device__ __forceinline__ int geo_strip_of(const Geo& g, int h) {
  return !geo_ragged(g) ? h / g.Hs : static_cast<int>(((static_cast<long long>(h) + 1) * g.P_r - 1) / g.H);
}
__device__ __forceinline__ long long pix_index(const Geo& g, int b, int q) {     // pixel q = h * W + w of image b in the padded layout
  const int h = q / g.W, w = q - h * g.W;
  const int s = geo_strip_of(g, h), r = h - geo_first(g, s) + g.ph;
  return ((static_cast<long long>(b) * g.P_r + s) * g.R + r) * g.Wp + w + g.pw;
}

// The same pixel in the s^2 phase planes a strided layer reads its input through (see decimate_kernel): plane
// (h mod s, w mod s) of the strip, at (h / s, w / s) in the geometry `go` of the layer's output.
__device__ __forceinline__ long long plane_index(const Geo& g, const Geo& go, int s, int b, int q) {
  const int h = q / g.W, w = q - h * g.W;
  const int st = h / g.Hs, hl = h - st * g.Hs;
  const int hq = hl / s, wq = w / s;
  const long long z = static_cast<long long>(b) * g.P_r + st;
  return ((hl - hq * s) * s + (w - wq * s)) * go.Ptot + (z * go.R + hq + go.ph) * go.Wp + wq + go.pw;
}

// WIDE: 64 channels per block, one run (no division by the channel count)
// PLANES: the destination is the phase planes of a stride-s layer (geometry go), not the tensor in geometry g: the input
// of a strided first layer goes from NCHW straight into the form its products read
template <bool WIDE, bool PLANES>
__global__ void __launch_bounds__(128)
nchw_to_pix_kernel(const bf16* __restrict__ src, bf16* __restrict__ dst, Geo g, int C, StageTile st, Geo go, int s) {
  __shared__ uint32_t tile[32][33];                   // [pixel of its run][pair row]
  const int HW = g.H * g.W;
  const int b = blockIdx.y, q0 = blockIdx.x * 32 * st.G, c0 = blockIdx.z * st.cpb;
  const int hp = st.cpb >> 1;                         // pair rows per run
  const int t = threadIdx.x;
  {
    const int pr = t >> 2, wq = (t & 3) * 8;          // pair row = (run, channel pair); pixels q .. q + 7 of that run
    const int pg = WIDE ? 0 : pr / hp, cp = pr - pg * hp;
    const int q = q0 + pg * 32 + wq, ch = c0 + 2 * cp;
    if (pg < st.G && ch < C && q < HW) {
      const bf16* p0 = src + (static_cast<long long>(b) * C + ch) * HW + q;
      const bf16* p1 = p0 + HW;
      uint16_t lo[8], hi[8];
      if ((HW & 7) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {      // 16 aligned bytes, all inside the plane
        const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p0)), c = __ldcs(reinterpret_cast<const uint4*>(p1));
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          lo[2 * i] = aw[i] & 0xFFFFu; lo[2 * i + 1] = aw[i] >> 16;
          hi[2 * i] = cw[i] & 0xFFFFu; hi[2 * i + 1] = cw[i] >> 16;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const bool in = q + i < HW;
          lo[i] = in ? __bfloat16_as_ushort(p0[i]) : 0;
          hi[i] = in ? __bfloat16_as_ushort(p1[i]) : 0;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) tile[wq + i][pr] = static_cast<uint32_t>(lo[i]) | (static_cast<uint32_t>(hi[i]) << 16);
    }
  }
  __syncthreads();
  const int px = t >> 2;                              // pixel px of its run; two groups of four pair rows = 8 channels each
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int pr0 = ((t & 3) + 4 * k) * 4;          // (the four threads of a pixel cover 64 contiguous bytes per access)
    const int pg = WIDE ? 0 : pr0 / hp, cp0 = pr0 - pg * hp;       // (hp is a multiple of 4: the four rows lie in one run)
    const int q = q0 + pg * 32 + px, ch = c0 + 2 * cp0;
    if (pg >= st.G || q >= HW || ch >= C) continue;
    uint4 o;
    o.x = tile[px][pr0]; o.y = tile[px][pr0 + 1]; o.z = tile[px][pr0 + 2]; o.w = tile[px][pr0 + 3];
    *reinterpret_cast<uint4*>(dst + (PLANES ? plane_index(g, go, s, b, q) : pix_index(g, b, q)) * C + ch) = o;
  }
}

template <bool WIDE>
__global__ void __launch_bounds__(128)
pix_to_nchw_kernel(const bf16* __restrict__ src, bf16* __restrict__ dst, Geo g, int C, StageTile st) {
  __shared__ uint32_t tile[32][33];
  const int HW = g.H * g.W;
  const int b = blockIdx.y, q0 = blockIdx.x * 32 * st.G, c0 = blockIdx.z * st.cpb;
  const int hp = st.cpb >> 1;
  const int t = threadIdx.x;
  {
    const int px = t >> 2;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int pr0 = ((t & 3) + 4 * k) * 4;          // (the four threads of a pixel cover 64 contiguous bytes per access)
      const int pg = WIDE ? 0 : pr0 / hp, cp0 = pr0 - pg * hp;
      const int q = q0 + pg * 32 + px, ch = c0 + 2 * cp0;
      if (pg >= st.G || q >= HW || ch >= C) continue;
      const uint4 v = *reinterpret_cast<const uint4*>(src + pix_index(g, b, q) * C + ch);
      tile[px][pr0] = v.x; tile[px][pr0 + 1] = v.y; tile[px][pr0 + 2] = v.z; tile[px][pr0 + 3] = v.w;
    }
  }
  __syncthreads();
  const int pr = t >> 2, wq = (t & 3) * 8;
  const int pg = WIDE ? 0 : pr / hp, cp = pr - pg * hp;
  const int q = q0 + pg * 32 + wq, ch = c0 + 2 * cp;
  if (pg >= st.G || ch >= C || q >= HW) return;
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) w[i] = tile[wq + i][pr];
  bf16* p0 = dst + (static_cast<long long>(b) * C + ch) * HW + q;
  bf16* p1 = p0 + HW;
  if ((HW & 7) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
    uint4 a, c;
    a.x = (w[0] & 0xFFFFu) | (w[1] << 16); a.y = (w[2] & 0xFFFFu) | (w[3] << 16);
    a.z = (w[4] & 0xFFFFu) | (w[5] << 16); a.w = (w[6] & 0xFFFFu) | (w[7] << 16);
    c.x = (w[0] >> 16) | (w[1] & 0xFFFF0000u); c.y = (w[2] >> 16) | (w[3] & 0xFFFF0000u);
    c.z = (w[4] >> 16) | (w[5] & 0xFFFF0000u); c.w = (w[6] >> 16) | (w[7] & 0xFFFF0000u);
    *reinterpret_cast<uint4*>(p0) = a;
    *reinterpret_cast<uint4*>(p1) = c;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (q + i < HW) {
        p0[i] = __ushort_as_bfloat16(static_cast<uint16_t>(w[i] & 0xFFFFu));
        p1[i] = __ushort_as_bfloat16(static_cast<uint16_t>(w[i] >> 16));
      }
  }
}

// Everything that is not a strip's own pixel: the padding columns and the image's outer rows become zero; a halo
// row becomes the copy of the neighbouring strip's boundary row (fill_halos) -- the halo exchange of Section 2.2:
// floor(k_h/2) rows per neighbour and direction -- or zero (a gradient about to enter the weight-gradient sum, whose
// pixels must each be counted once); the dead row of a strip that is one row shorter than the slots becomes zero.
// One thread per 16 bytes of padding: per strip the 2 ph halo rows (and one more row slot when heights differ), then
// the 2 pw side columns of its own rows.
__global__ void __launch_bounds__(256)
pad_fix_kernel(bf16* __restrict__ T, Geo g, int C, int fill_halos) {
  const int c8 = C / 8;
  const int extra = geo_ragged(g) ? 1 : 0;
  const int n_rows = (2 * g.ph + extra) * g.Wp * c8;   // chunks in the rows of a strip that are not its own
  const int n_side = g.Hs * 2 * g.pw * c8;             // chunks in the side columns of its own rows
  const int per_strip = n_rows + n_side;
  const long long total = g.Z * per_strip;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
    const long long z = i / per_strip;
    int k = static_cast<int>(i - z * per_strip);
    const int s = static_cast<int>(z % g.P_r);
    const int hs = geo_height(g, s);                   // this strip's own rows: ph .. ph + hs - 1
    int r, x, cg;
    if (k < n_rows) {
      cg = k % c8; k /= c8;
      x = k % g.Wp; k /= g.Wp;                         // k: 0 .. 2 ph - 1 (+ 1)
      r = k < g.ph ? k : k + hs;
      if (r >= g.R) continue;                          // (a strip of full height has no dead row)
    } else {
      k -= n_rows;
      cg = k % c8; k /= c8;
      const int side = k % (2 * g.pw); k /= 2 * g.pw;  // k: row slot 0 .. Hs - 1
      if (k >= hs) continue;                           // (the dead row was zeroed as a whole)
      x = side < g.pw ? side : side + g.W;
      r = k + g.ph;
    }
    uint4 v = make_uint4(0, 0, 0, 0);
    if (fill_halos && x >= g.pw && x < g.pw + g.W) {
      if (r < g.ph && s > 0)                                        // rows above the strip: the last rows of the strip above
        v = *reinterpret_cast<const uint4*>(T + ((((z - 1) * g.R) + r + geo_height(g, s - 1)) * g.Wp + x) * C + cg * 8);
      else if (r >= g.ph + hs && r < 2 * g.ph + hs && s < g.P_r - 1)   // rows below it: the first rows of the strip below
        v = *reinterpret_cast<const uint4*>(T + ((((z + 1) * g.R) + r - hs) * g.Wp + x) * C + cg * 8);
    }
    *reinterpret_cast<uint4*>(T + ((z * g.R + r) * g.Wp + x) * C + cg * 8) = v;
  }
}

// Per-CTA sums of squares of a bf16 tensor (padding is zero, so the whole buffer may be summed); fixed order.
__global__ void __launch_bounds__(256)
ssq_partial_kernel(const bf16* __restrict__ T, long long n8, float* __restrict__ part) {
  float s = 0.f;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n8; i += gridDim.x * 256ll) {
    const uint4 q = *reinterpret_cast<const uint4*>(T + i * 8);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = __uint_as_float(w[j] << 16), b = __uint_as_float(w[j] & 0xFFFF0000u);
      s = fmaf(a, a, s);
      s = fmaf(b, b, s);
    }
  }
  __shared__ float sh[256];
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = sh[0];
}

// Public kernel K[o][c][u][v]  <->  internal Wm[o][j], j < ldw.  `colmap[j]` = t * Cin + c (t = u kw + v) for the kernel
// element that column j holds, or -1 for a padding column (a zero weight that stays zero).  Unfolded layers:
// j = t * Cp + c with the channels padded to Cp; a folded first layer: j = run * 64 + g * Cin + c (see fold_runs).
template <typename T>
__global__ void pack_w_kernel(const T* __restrict__ K, T* __restrict__ Wm, const int* __restrict__ colmap, int Cout, int Cin, int taps, int ldw) {
  const long long n = static_cast<long long>(Cout) * ldw;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
    const int j = static_cast<int>(i % ldw);
    const int o = static_cast<int>(i / ldw);
    const int m = colmap[j];
    T v = T(0.f);
    if (m >= 0) v = K[(static_cast<long long>(o) * Cin + m % Cin) * taps + m / Cin];
    Wm[i] = v;
  }
}
template <typename T>
__global__ void unpack_w_kernel(const T* __restrict__ Wm, T* __restrict__ K, const int* __restrict__ colmap, int Cout, int Cin, int taps, int ldw) {
  const long long n = static_cast<long long>(Cout) * ldw;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
    const int j = static_cast<int>(i % ldw);
    const int o = static_cast<int>(i / ldw);
    const int m = colmap[j];
    if (m >= 0) K[(static_cast<long long>(o) * Cin + m % Cin) * taps + m / Cin] = Wm[i];
  }
}

// A strided layer (stride s) reads its input through s^2 phase planes: plane (a, b) holds the pixels (s h' + a, s w' + b)
// of every strip in the geometry of the layer's OUTPUT (`go`), so that tap (u, v), with u - k_h/2 = s du + a and
// v - k_w/2 = s dv + b, reads plane (a, b) at the output pixel shifted by (du, dv): the strided layer becomes a
// stride-1 product over shifted views again, with no position computed that is not kept.
// decimate: own pixels of T (geometry gi) -> planes P[s^2][go.Ptot][C]; undecimate: the way back (a gradient).
__global__ void __launch_bounds__(256)
decimate_kernel(bf16* __restrict__ T, bf16* __restrict__ P, Geo gi, Geo go, int C, int s, int to_planes) {
  const int c8 = C / 8;
  const long long total = gi.Z * gi.Hs * gi.W * c8;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
    const int cg = static_cast<int>(i % c8);
    long long q = i / c8;
    const int w = static_cast<int>(q % gi.W); q /= gi.W;
    const int h = static_cast<int>(q % gi.Hs);
    const long long z = q / gi.Hs;
    const int a = h % s, b = w % s;
    const long long pin = (z * gi.R + h + gi.ph) * gi.Wp + w + gi.pw;
    const long long pout = (a * s + b) * go.Ptot + (z * go.R + h / s + go.ph) * go.Wp + w / s + go.pw;
    if (to_planes) *reinterpret_cast<uint4*>(P + pout * C + cg * 8) = *reinterpret_cast<const uint4*>(T + pin * C + cg * 8);
    else *reinterpret_cast<uint4*>(T + pin * C + cg * 8) = *reinterpret_cast<const uint4*>(P + pout * C + cg * 8);
  }
}

int grid_1d(long long n, int num_sms) {
  const long long b = (n + 255) / 256;
  const long long cap = static_cast<long long>(num_sms) * 16;
  return static_cast<int>(std::max(1ll, std::min(b, cap)));
}
int round64(int c) { return (c + 63) / 64 * 64; }
int floor_div(int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }

}  // namespace

struct GenConv {
  int L = 0;
  int64_t B = 0;
  int P_r = 1, P = 1, S = 1;              // strips; processes of the grid; fp32 partial sums per weight gradient asked for
  int model_P_r = 1, S_dx = 1;            // model-parallel layers: groups that split the output channels; partial sums per dX asked for
  bool need_dx0 = false;                  // this stack continues another one: the gradient w.r.t. its input is formed too (dX0)
  int in_relu = 0;                        // ... and its input is the ReLU output of the layer below (mask of that gradient)
  bf16* dX0 = nullptr;
  std::vector<Geo> geo;                   // geometry of tensor i (act[i]; dY[i] has that of act[i + 1])
  std::vector<int> Cin, Cout, kh, kw, relu, taps, Cp, stride;
  std::vector<int> ldw;                   // columns of the internal weight matrix of layer i
  std::vector<int*> colmap;               // device: column -> kernel element (see pack_w_kernel)
  std::vector<int> folded;                // layer 0 with few input channels: several taps per 64-wide k-block (fold_runs)
  std::vector<bf16*> act, dY, Wm;
  std::vector<bf16*> xph, dxph;           // strided layers: phase planes of the input / of the gradient below
  std::vector<float*> dWm;
  std::vector<float*> Wm32, Vm;           // fp32 master weights / momentum velocities in the layout of Wm (empty unless enabled)
  float mu = 0.f;
  std::vector<TcGemm> fwd, bwd_weight;
  std::vector<std::vector<TcGemm>> bwd_data;   // one product (stride 1) or one per phase plane
  std::vector<std::vector<int>> bwd_taps;      // taps of each of those products (an empty plane gets zeros)
  float* partials = nullptr;
  float* loss_part = nullptr;
  int loss_grid = 0;
  int* status = nullptr;
  cudaStream_t stream = nullptr;
  Profiler* prof = nullptr;
  int num_sms = 148;
  bool fc_above = false;
};

namespace {

Epi make_epi_act(void* out, int64_t ldo, int out_bf16, int relu) {
  Epi e{};
  e.op = EPI_ACT; e.out_bf16 = out_bf16; e.out = out; e.ldo = ldo; e.relu = relu;
  return e;
}
Epi make_epi_mask(void* out, int64_t ldo, const void* mask, int64_t ldmask) {
  Epi e{};
  e.op = EPI_MASK; e.out_bf16 = 1; e.out = out; e.ldo = ldo; e.mask = mask; e.ldmask = ldmask;
  return e;
}
Epi make_epi_sgd(void* w, int64_t ldo, float scale) {
  Epi e{};
  e.op = EPI_SGD; e.out_bf16 = 1; e.out = w; e.ldo = ldo; e.scale = scale;
  return e;
}

// One product and, when its K range was cut into planes, their reduction with the tail operation.
mbd_status run(GenConv* c, TcGemm& t, int cls, double flops, const Epi& epi) {
  t.epi = epi;
  t.partials = c->partials;
  t.flags = nullptr;
  c->prof->begin(cls, flops, c->stream);
  if (tc_gemm_launch(t, c->stream) != cudaSuccess) return MBD_E_CUDA;
  c->prof->end();
  if (t.k_splits > 1) {
    const double esz = epi.out_bf16 ? 2.0 : 4.0;
    c->prof->begin(MBD_K_REDUCE, static_cast<double>(t.M) * t.N * (4.0 * t.k_splits + 2.0 * esz), c->stream);
    if (reduce_partials_launch(c->partials, t.k_splits, t.M, t.N, epi, c->num_sms, c->stream) != cudaSuccess) return MBD_E_CUDA;
    c->prof->end();
  }
  return MBD_OK;
}

// `planes` > 1: the tensor is that many phase planes of geometry g, one after another (the strips of plane q are
// strips q Z .. of the stack; Z is a multiple of P_r, so a strip's neighbours are in its own plane)
void pad_fix(GenConv* c, bf16* T, Geo g, int C, bool fill_halos, int planes = 1) {
  g.Z *= planes;
  g.Ptot *= planes;
  const long long chunks = g.Z * ((2ll * g.ph + (geo_ragged(g) ? 1 : 0)) * g.Wp + 2ll * g.Hs * g.pw) * (C / 8);
  c->prof->begin(MBD_K_HALO, static_cast<double>(chunks) * 16.0, c->stream);
  if (chunks > 0) pad_fix_kernel<<<grid_1d(chunks, c->num_sms), 256, 0, c->stream>>>(T, g, C, fill_halos ? 1 : 0);
  c->prof->end();
}

void decimate(GenConv* c, bf16* T, bf16* planes, const Geo& gi, const Geo& go, int C, int s, bool to_planes) {
  const long long n = gi.Z * gi.Hs * gi.W * (C / 8);
  c->prof->begin(MBD_K_HALO, static_cast<double>(n) * 32.0, c->stream);
  decimate_kernel<<<grid_1d(n, c->num_sms), 256, 0, c->stream>>>(T, planes, gi, go, C, s, to_planes ? 1 : 0);
  c->prof->end();
}

// Offsets of a layer's taps in pixel rows of the tensor its products read: stride 1: the input itself in geometry g;
// stride s: the phase planes in the OUTPUT geometry g (plane start + shift inside the plane).
void tap_offsets(int kh, int kw, int s, const Geo& g, int* off, int* plane) {
  for (int u = 0; u < kh; ++u)
    for (int v = 0; v < kw; ++v) {
      const int du = floor_div(u - kh / 2, s), dv = floor_div(v - kw / 2, s);
      const int a = (u - kh / 2) - du * s, b = (v - kw / 2) - dv * s;
      plane[u * kw + v] = a * s + b;
      off[u * kw + v] = du * g.Wp + dv;
    }
}

// A first layer with few input channels (8, 16 or 32) would fill an eighth to a half of a 64-wide k-block per tap.  Its
// input is pixel-major, so the channels of G = 64 / C_in CONSECUTIVE pixels are 64 contiguous elements: through a
// tensor map whose rows overlap (row pitch = one pixel = C_in elements, row length 64) one TMA box holds the operands
// of G horizontally adjacent taps at once.  A run = up to G taps of one kernel row that read the same phase plane at
// consecutive pixels; the k-blocks of the folded layer are its runs (columns of absent taps carry zero weights).
struct Run { int plane, off, n, tap[8]; };
std::vector<Run> fold_runs(int kh, int kw, int s, int Cin, const Geo& g) {
  int off[MAX_TAPS], plane[MAX_TAPS];
  tap_offsets(kh, kw, s, g, off, plane);
  const int G = 64 / Cin;
  std::vector<Run> runs;
  std::vector<char> used(kh * kw, 0);
  for (int t = 0; t < kh * kw; ++t) {
    if (used[t]) continue;
    Run r{};
    r.plane = plane[t]; r.off = off[t]; r.n = 0;
    for (int g2 = 0; g2 < G; ++g2) r.tap[g2] = -1;
    // taps of the same kernel row (same u) in the same plane, at this tap's pixel + 0 .. G-1
    for (int t2 = t; t2 < kh * kw && t2 / kw == t / kw; ++t2)
      if (!used[t2] && plane[t2] == r.plane && off[t2] - r.off >= 0 && off[t2] - r.off < G) {
        r.tap[off[t2] - r.off] = t2;
        used[t2] = 1;
        ++r.n;
      }
    runs.push_back(r);
  }
  return runs;
}

}  // namespace

bool gconv_needed(const mbd_layer* layers, int L) {
  if (getenv("MBD_CONV_GENERAL")) return true;        // tuning knob: the listed 64-channel layers through this path too
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    const bool k3 = l.kh == 3 && l.kw == 3, k1 = l.kh == 1 && l.kw == 1;
    if (!(k3 || k1) || l.C_in != 64 || l.C_out != 64 || l.stride > 1) return true;
    if (l.split == MBD_SPLIT_MODEL) return true;      // output channels over the P_r groups: products with a cut of K over channel blocks
  }
  return false;
}

void gconv_destroy(GenConv* c) {
  if (!c) return;
  for (size_t i = 0; i < c->act.size(); ++i) cudaFree(c->act[i]);
  for (size_t i = 0; i < c->dY.size(); ++i)
    if (c->dY[i] && (c->act.size() <= static_cast<size_t>(c->L) || c->dY[i] != c->act[c->L])) cudaFree(c->dY[i]);
  for (bf16* p : c->Wm) cudaFree(p);
  for (int* p : c->colmap) cudaFree(p);
  for (bf16* p : c->xph) cudaFree(p);
  for (bf16* p : c->dxph) cudaFree(p);
  for (float* p : c->dWm) cudaFree(p);
  for (float* p : c->Wm32) cudaFree(p);
  for (float* p : c->Vm) cudaFree(p);
  cudaFree(c->partials); cudaFree(c->loss_part); cudaFree(c->dX0);
  delete c;
}

mbd_status gconv_create(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, int max_partials, int num_sms, int* status,
                        cudaStream_t stream, Profiler* prof, bool fc_above, int model_P_r, bool need_dx0, int in_relu, GenConv** out) {
  if (tc_gemm_init() != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  // one padding for every tensor: what the widest reach of any layer needs at the resolution it works in
  int ph = 0, pw = 0, H = layers[0].H, W = layers[0].W;
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    const int s = l.stride > 1 ? l.stride : 1;
    if (l.kh < 1 || l.kw < 1 || l.kh > 11 || l.kw > 11 || l.kh % 2 == 0 || l.kw % 2 == 0 || s > 4) return MBD_E_UNSUPPORTED;
    if (l.C_in < 8 || l.C_out < 8 || l.C_in % 8 || l.C_out % 8) return MBD_E_UNSUPPORTED;       // 16-byte rows for TMA
    if (i > 0 && l.C_in != layers[i - 1].C_out) return MBD_E_INVALID;
    if (l.H != H || l.W != W || H % s || W % s) return MBD_E_INVALID;                            // sizes chain through the strides
    if ((H % P_r != 0 || (H / s) % P_r != 0) && s > 1) return MBD_E_UNSUPPORTED;                 // a strided layer's phase planes need strips of equal height
    ph = std::max(ph, (l.kh / 2 + s - 1) / s); pw = std::max(pw, (l.kw / 2 + s - 1) / s);
    H /= s; W /= s;
  }
  GenConv* c = new (std::nothrow) GenConv();
  if (!c) return MBD_E_ALLOC;
  c->L = L; c->B = B; c->P_r = P_r; c->status = status; c->stream = stream; c->prof = prof; c->num_sms = num_sms; c->fc_above = fc_above;
  c->geo.resize(L + 1);
  H = layers[0].H; W = layers[0].W;
  for (int t = 0; t <= L; ++t) {
    Geo& g = c->geo[t];
    g.B = static_cast<int>(B); g.H = H; g.W = W; g.P_r = P_r; g.Hs = (H + P_r - 1) / P_r; g.ph = ph; g.pw = pw;      // row slots: the tallest strip
    g.R = g.Hs + 2 * ph; g.Wp = W + 2 * pw; g.Z = B * P_r; g.Ptot = g.Z * g.R * g.Wp;
    if (P_r > 1 && H / P_r < ph) { delete c; return MBD_E_GRID; }          // a halo row must come from the adjacent strip (the shortest one too)
    const int s = t < L && layers[t].stride > 1 ? layers[t].stride : 1;
    if (B > INT32_MAX / std::max(1, P_r) || g.Ptot * s * s > INT32_MAX - 512) { delete c; return MBD_E_UNSUPPORTED; }   // TMA coordinates are 32-bit
    if (t < L) { H /= s; W /= s; }
  }
  c->P = P_r * P_c;
  c->S = max_partials < 1 ? 1 : std::min(c->P, max_partials);
  // Model-parallel layers (Eq. 8): no strips (P_r = 1 here), the weight gradient's rows are independent, so its partial
  // sums are over the P_c batch blocks (c->S above), and dX = sum over the model_P_r groups of W_r^T dY_r is a cut of
  // backward-data's K range over blocks of output channels
  c->need_dx0 = need_dx0; c->in_relu = in_relu;
  c->model_P_r = model_P_r < 1 ? 1 : model_P_r;
  c->S_dx = max_partials < 1 ? 1 : std::min(c->model_P_r, max_partials);
  auto alloc = [&](void** p, size_t bytes) -> bool {
    if (cudaMalloc(p, bytes) != cudaSuccess) { (void)cudaGetLastError(); *p = nullptr; return false; }
    return cudaMemsetAsync(*p, 0, bytes, stream) == cudaSuccess;
  };
  bool ok = true;
  c->act.assign(L + 1, nullptr); c->dY.assign(L, nullptr); c->Wm.assign(L, nullptr); c->dWm.assign(L, nullptr);
  c->xph.assign(L, nullptr); c->dxph.assign(L, nullptr);
  c->fwd.resize(L); c->bwd_data.resize(L); c->bwd_taps.resize(L); c->bwd_weight.resize(L);
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    c->Cin.push_back(l.C_in); c->Cout.push_back(l.C_out); c->kh.push_back(l.kh); c->kw.push_back(l.kw);
    c->stride.push_back(l.stride > 1 ? l.stride : 1);
    // the output of the last layer of a convolution-only network goes into the half-SSQ loss as it is
    c->relu.push_back((i == L - 1 && !fc_above) ? 0 : l.relu);
    c->taps.push_back(l.kh * l.kw); c->Cp.push_back(round64(l.C_in));
  }
  // (256 bytes of slack behind the tensors a folded layer reads: its last rows reach up to 64 - C_in elements further)
  for (int i = 0; i <= L && ok; ++i) {
    const int C = i == 0 ? c->Cin[0] : c->Cout[i - 1];
    if (i == 0 && c->stride[0] > 1 && !need_dx0) continue;          // the input of a strided first layer lives in its phase planes only
    ok = alloc(reinterpret_cast<void**>(&c->act[i]), static_cast<size_t>(c->geo[i].Ptot) * C * 2 + 256);
  }
  if (need_dx0) ok = ok && alloc(reinterpret_cast<void**>(&c->dX0), static_cast<size_t>(c->geo[0].Ptot) * c->Cin[0] * 2);
  // internal weight layouts
  c->ldw.assign(L, 0); c->colmap.assign(L, nullptr); c->folded.assign(L, 0);
  std::vector<std::vector<Run>> runs(L);
  for (int i = 0; i < L && ok; ++i) {
    const int Cin = c->Cin[i], taps = c->taps[i], Cp = c->Cp[i];
    std::vector<int> map;
    const bool fold = i == 0 && !need_dx0 && (Cin == 8 || Cin == 16 || Cin == 32) && taps > 1 && !getenv("MBD_CONV_NO_FOLD");      // tuning knob (a folded layer has no backward-data product)
    if (fold) {
      runs[i] = fold_runs(c->kh[i], c->kw[i], c->stride[i], Cin, c->geo[i + 1]);
      if (static_cast<int>(runs[i].size()) <= MAX_TAPS && static_cast<int>(runs[i].size()) * 64 < taps * Cp) {
        c->folded[i] = 1;
        map.assign(runs[i].size() * 64, -1);
        for (size_t r = 0; r < runs[i].size(); ++r)
          for (int g2 = 0; g2 < 64 / Cin; ++g2)
            if (runs[i][r].tap[g2] >= 0)
              for (int ch = 0; ch < Cin; ++ch) map[r * 64 + g2 * Cin + ch] = runs[i][r].tap[g2] * Cin + ch;
      }
    }
    if (!c->folded[i]) {
      map.assign(static_cast<size_t>(taps) * Cp, -1);
      for (int t = 0; t < taps; ++t)
        for (int ch = 0; ch < Cin; ++ch) map[static_cast<size_t>(t) * Cp + ch] = t * Cin + ch;
    }
    c->ldw[i] = static_cast<int>(map.size());
    ok = alloc(reinterpret_cast<void**>(&c->colmap[i]), map.size() * sizeof(int)) &&
         cudaMemcpyAsync(c->colmap[i], map.data(), map.size() * sizeof(int), cudaMemcpyHostToDevice, stream) == cudaSuccess &&
         cudaStreamSynchronize(stream) == cudaSuccess;          // `map` is a local
  }
  for (int i = 0; i < L && ok; ++i) {
    const Geo& go = c->geo[i + 1];
    if (i < L - 1 || fc_above) ok = alloc(reinterpret_cast<void**>(&c->dY[i]), static_cast<size_t>(go.Ptot) * c->Cout[i] * 2);
    else c->dY[i] = c->act[L];                       // half-SSQ loss: dY_L = Y_L
    const size_t nw = static_cast<size_t>(c->Cout[i]) * c->ldw[i];
    ok = ok && alloc(reinterpret_cast<void**>(&c->Wm[i]), nw * 2) && alloc(reinterpret_cast<void**>(&c->dWm[i]), nw * 4);
    if (c->stride[i] > 1) {
      const size_t pl = static_cast<size_t>(c->stride[i]) * c->stride[i] * go.Ptot * c->Cin[i] * 2;
      ok = ok && alloc(reinterpret_cast<void**>(&c->xph[i]), pl + 256);
      if (i > 0 || need_dx0) ok = ok && alloc(reinterpret_cast<void**>(&c->dxph[i]), pl);
    }
  }
  c->loss_grid = num_sms * 4;
  ok = ok && alloc(reinterpret_cast<void**>(&c->loss_part), sizeof(float) * c->loss_grid);
  if (!ok) { gconv_destroy(c); return MBD_E_ALLOC; }
  size_t part_elems = 0;
  for (int i = 0; i < L; ++i) {
    const int Cin = c->Cin[i], Cout = c->Cout[i], taps = c->taps[i], Cp = c->Cp[i], Cop = round64(Cout), s = c->stride[i];
    const int ldw = c->ldw[i];
    const Geo& go = c->geo[i + 1];                   // the products run over the pixels of the layer's output geometry
    const int M = static_cast<int>(go.Ptot);
    bf16* xin = s > 1 ? c->xph[i] : c->act[i];       // what the forward and weight-gradient products read
    int off[MAX_TAPS], plane[MAX_TAPS];
    tap_offsets(c->kh[i], c->kw[i], s, go, off, plane);
    // forward
    TcGemm& f = c->fwd[i];
    f = TcGemm{};
    f.variant = 0; f.M = M; f.N = Cout; f.K = ldw; f.k_splits = 1; f.status = status;
    f.cv.mode = 1;
    if (c->folded[i]) {            // k-block = run; the A rows are the overlapping 64-element windows of the pixel-major input
      f.cv.taps = static_cast<int>(runs[i].size()); f.cv.blocks = 1; f.cv.Cp = 64;
      for (int r = 0; r < f.cv.taps; ++r) { f.cv.off[r] = runs[i][r].plane * M + runs[i][r].off; f.cv.tap[r] = r; }
      f.cv_a_inner = 64;
    } else {
      f.cv.taps = taps; f.cv.blocks = Cp / 64; f.cv.Cp = Cp;
      for (int t = 0; t < taps; ++t) { f.cv.off[t] = plane[t] * M + off[t]; f.cv.tap[t] = t; }
      f.cv_a_inner = Cin;
    }
    f.cv_a_rows = static_cast<int64_t>(s) * s * M;
    const Epi ef = make_epi_act(c->act[i + 1], Cout, 1, c->relu[i]);
    if (tc_gemm_prepare(f, xin, Cin, c->Wm[i], ldw, num_sms, &ef) != cudaSuccess) { gconv_destroy(c); return MBD_E_CUDA; }
    // backward-data: one product (stride 1), or one per phase plane with the taps that read that plane
    if (i > 0 || need_dx0) {
      c->bwd_data[i].resize(s * s);
      c->bwd_taps[i].assign(s * s, 0);
      for (int q = 0; q < s * s; ++q) {
        TcGemm& d = c->bwd_data[i][q];
        d = TcGemm{};
        d.variant = 1; d.M = M; d.N = Cin; d.k_splits = c->S_dx; d.status = status;
        d.allow_fix = c->S_dx < c->model_P_r;          // fewer partial sums than groups: intermediate ones, they may stay in tensor memory
        d.cv.mode = 2; d.cv.blocks = Cop / 64; d.cv.Cp = Cp;
        d.cv.chan_major = c->model_P_r > 1;            // pieces of K = blocks of output channels, every tap of each
        int n = 0;
        for (int t = 0; t < taps; ++t)
          if (plane[t] == q) { d.cv.off[n] = off[t]; d.cv.tap[n] = t; ++n; }
        d.cv.taps = n;
        c->bwd_taps[i][q] = n;
        if (n == 0) continue;                          // no tap reads this plane: its gradient is zero
        d.K = n * Cop;
        d.cv_a_inner = Cout; d.cv_b_inner = ldw; d.cv_b_rows = Cout;
        bf16* outp = s > 1 ? c->dxph[i] + static_cast<size_t>(q) * M * Cin : (i > 0 ? c->dY[i - 1] : c->dX0);
        const bf16* maskp = !(i > 0 ? c->relu[i - 1] : c->in_relu) ? nullptr : (s > 1 ? c->xph[i] + static_cast<size_t>(q) * M * Cin : c->act[i]);
        const Epi ed = make_epi_mask(outp, Cin, maskp, Cin);
        if (tc_gemm_prepare(d, c->dY[i], Cout, c->Wm[i], ldw, num_sms, &ed) != cudaSuccess) { gconv_destroy(c); return MBD_E_CUDA; }
        if (d.k_splits > 1) part_elems = std::max(part_elems, static_cast<size_t>(d.k_splits) * M * Cin);
      }
    }
    // backward-weight: few output tiles, a very long K (all pixels): the planner cuts K to fill the SMs
    TcGemm& w = c->bwd_weight[i];
    w = TcGemm{};
    w.variant = 2; w.M = Cout; w.N = ldw; w.K = M; w.k_splits = c->S; w.status = status;
    w.allow_extra_split = 1;
    w.cv.mode = 3; w.cv.blocks = 0;
    if (c->folded[i]) {
      w.cv.taps = static_cast<int>(runs[i].size()); w.cv.Cp = 64;
      for (int r = 0; r < w.cv.taps; ++r) { w.cv.off[r] = runs[i][r].plane * M + runs[i][r].off; w.cv.tap[r] = r; }
      w.cv_b_inner = 64;
    } else {
      w.cv.taps = taps; w.cv.Cp = Cp;
      for (int t = 0; t < taps; ++t) { w.cv.off[t] = plane[t] * M + off[t]; w.cv.tap[t] = t; }
      w.cv_b_inner = Cin;
    }
    w.cv_b_rows = static_cast<int64_t>(s) * s * M;
    const Epi ew = make_epi_sgd(c->Wm[i], ldw, 0.f);
    if (tc_gemm_prepare(w, c->dY[i], Cout, xin, Cin, num_sms, &ew) != cudaSuccess) { gconv_destroy(c); return MBD_E_CUDA; }
    if (w.k_splits > 1) part_elems = std::max(part_elems, static_cast<size_t>(w.k_splits) * Cout * ldw);
  }
  if (part_elems && !alloc(reinterpret_cast<void**>(&c->partials), part_elems * 4)) { gconv_destroy(c); return MBD_E_ALLOC; }
  if (cudaStreamSynchronize(stream) != cudaSuccess) { gconv_destroy(c); return MBD_E_CUDA; }
  *out = c;
  return MBD_OK;
}

size_t gconv_input_bytes(const GenConv* c) { return static_cast<size_t>(c->B) * c->Cin[0] * c->geo[0].H * c->geo[0].W * 2; }
int gconv_last_relu(const GenConv* c) { return c->relu[c->L - 1]; }

mbd_status gconv_set_weights(GenConv* c, int i, const void* K_dev) {
  const long long n = static_cast<long long>(c->Cout[i]) * c->ldw[i];
  pack_w_kernel<bf16><<<grid_1d(n, c->num_sms), 256, 0, c->stream>>>(static_cast<const bf16*>(K_dev), c->Wm[i], c->colmap[i], c->Cout[i], c->Cin[i], c->taps[i], c->ldw[i]);
  if (!c->Wm32.empty() && widen_bf16_launch(c->Wm[i], c->Wm32[i], n, c->num_sms, c->stream) != cudaSuccess) return MBD_E_CUDA;
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

// fp32 master weights / momentum: the update leaves the weight-gradient product (which then only materialises dWm)
// and becomes one streaming kernel per layer over the internal weight layout -- as for the fully connected layers.
mbd_status gconv_enable_master(GenConv* c) {
  if (!c->Wm32.empty()) return MBD_OK;
  std::vector<float*> m(c->L, nullptr);
  for (int i = 0; i < c->L; ++i) {
    const long long n = static_cast<long long>(c->Cout[i]) * c->ldw[i];
    if (cudaMalloc(reinterpret_cast<void**>(&m[i]), n * 4) != cudaSuccess || widen_bf16_launch(c->Wm[i], m[i], n, c->num_sms, c->stream) != cudaSuccess) {
      (void)cudaGetLastError();
      for (float* q : m) cudaFree(q);
      return MBD_E_ALLOC;
    }
  }
  c->Wm32 = m;
  return MBD_OK;
}

mbd_status gconv_enable_momentum(GenConv* c, float mu) {
  if (c->Vm.empty()) {
    std::vector<float*> v(c->L, nullptr);
    for (int i = 0; i < c->L; ++i)
      if (cudaMalloc(reinterpret_cast<void**>(&v[i]), static_cast<size_t>(c->Cout[i]) * c->ldw[i] * 4) != cudaSuccess) {
        (void)cudaGetLastError();
        for (float* q : v) cudaFree(q);
        return MBD_E_ALLOC;
      }
    c->Vm = v;
  }
  for (int i = 0; i < c->L; ++i)
    if (cudaMemsetAsync(c->Vm[i], 0, static_cast<size_t>(c->Cout[i]) * c->ldw[i] * 4, c->stream) != cudaSuccess) return MBD_E_CUDA;
  c->mu = mu;
  return MBD_OK;
}

namespace {
// Eq. 1 (or its momentum form) from the materialised gradient of layer i
mbd_status update_from_gradient(GenConv* c, int i, float eta) {
  const long long n = static_cast<long long>(c->Cout[i]) * c->ldw[i];
  const float scale = -eta / static_cast<float>(c->B);
  float* w32 = c->Wm32.empty() ? nullptr : c->Wm32[i];
  c->prof->begin(MBD_K_SGD, static_cast<double>(n) * (8.0 + (w32 ? 8.0 : 0.0) + (c->Vm.empty() ? 0.0 : 8.0)), c->stream);
  cudaError_t e;
  if (!c->Vm.empty()) e = sgd_momentum_update_launch(c->Wm[i], 1, w32, c->Vm[i], c->dWm[i], n, c->mu, 1.f / static_cast<float>(c->B), eta, c->num_sms, c->stream);
  else if (w32) e = sgd_master_update_launch(w32, c->Wm[i], c->dWm[i], n, scale, c->num_sms, c->stream);
  else e = sgd_update_launch(c->Wm[i], 1, c->dWm[i], n, scale, c->num_sms, c->stream);
  c->prof->end();
  return e == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}
}  // namespace
mbd_status gconv_get_weights(GenConv* c, int i, void* K_dev) {
  const long long n = static_cast<long long>(c->Cout[i]) * c->ldw[i];
  unpack_w_kernel<bf16><<<grid_1d(n, c->num_sms), 256, 0, c->stream>>>(c->Wm[i], static_cast<bf16*>(K_dev), c->colmap[i], c->Cout[i], c->Cin[i], c->taps[i], c->ldw[i]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

namespace {
// go / s: the tensor is the input of a stride-s layer whose output has geometry *go: it is stored as that layer's
// phase planes (dst = the planes), and the planes' padding and halo rows are fixed instead of the tensor's
void stage(GenConv* c, const bf16* nchw, bf16* dst, const Geo& g, int C, bool fill_halos, const Geo* go = nullptr, int s = 1) {
  const StageTile t = stage_tile(C);
  const dim3 grid((g.H * g.W + 32 * t.G - 1) / (32 * t.G), static_cast<unsigned>(g.B), (C + t.cpb - 1) / t.cpb);
  c->prof->begin(MBD_K_HALO, 2.0 * g.B * C * g.H * g.W * 2.0, c->stream);
  if (go) {
    if (t.cpb == 64) nchw_to_pix_kernel<true, true><<<grid, 128, 0, c->stream>>>(nchw, dst, g, C, t, *go, s);
    else nchw_to_pix_kernel<false, true><<<grid, 128, 0, c->stream>>>(nchw, dst, g, C, t, *go, s);
  } else {
    if (t.cpb == 64) nchw_to_pix_kernel<true, false><<<grid, 128, 0, c->stream>>>(nchw, dst, g, C, t, g, 1);
    else nchw_to_pix_kernel<false, false><<<grid, 128, 0, c->stream>>>(nchw, dst, g, C, t, g, 1);
  }
  c->prof->end();
  if (go) pad_fix(c, dst, *go, C, fill_halos, s * s);
  else pad_fix(c, dst, g, C, fill_halos);
}
void unstage(GenConv* c, const bf16* src, bf16* nchw, const Geo& g, int C) {
  const StageTile t = stage_tile(C);
  const dim3 grid((g.H * g.W + 32 * t.G - 1) / (32 * t.G), static_cast<unsigned>(g.B), (C + t.cpb - 1) / t.cpb);
  c->prof->begin(MBD_K_HALO, 2.0 * g.B * C * g.H * g.W * 2.0, c->stream);
  if (t.cpb == 64) pix_to_nchw_kernel<true><<<grid, 128, 0, c->stream>>>(src, nchw, g, C, t);
  else pix_to_nchw_kernel<false><<<grid, 128, 0, c->stream>>>(src, nchw, g, C, t);
  c->prof->end();
}
}  // namespace

mbd_status gconv_stage_input(GenConv* c, const void* X_nchw) {
  if (c->stride[0] > 1 && !c->need_dx0)      // a strided first layer: straight into its phase planes (the input has no other reader)
    stage(c, static_cast<const bf16*>(X_nchw), c->xph[0], c->geo[0], c->Cin[0], true, &c->geo[1], c->stride[0]);
  else
    stage(c, static_cast<const bf16*>(X_nchw), c->act[0], c->geo[0], c->Cin[0], true);     // the forward halo exchange of the input rides along
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_forward_layer(GenConv* c, int i, float* loss_sum_dev) {
  if (i < 0 || i >= c->L) return MBD_E_INVALID;
  const bool last = i == c->L - 1;
  const Geo& go = c->geo[i + 1];
  const int s = c->stride[i];
  const double flops = 2.0 * c->B * go.H * go.W * c->taps[i] * c->Cin[i] * c->Cout[i];     // the method's flops
  if (s > 1 && (i > 0 || c->need_dx0)) {       // (otherwise the network's input was staged as planes)
    // the input's own pixels sorted into the s^2 phase planes; their halo rows exchanged plane by plane
    decimate(c, c->act[i], c->xph[i], c->geo[i], go, c->Cin[i], s, true);
    pad_fix(c, c->xph[i], go, c->Cin[i], true, s * s);
  }
  const Epi e = make_epi_act(c->act[i + 1], c->Cout[i], 1, c->relu[i]);
  mbd_status st = run(c, c->fwd[i], MBD_K_CONV_FWD, flops, e);
  if (st != MBD_OK) return st;
  // the output's halo exchange for the next layer (first halo term of Eq. 7); the last output is the top gradient of
  // the half-SSQ loss and enters the weight-gradient sum: zeros outside the strips' own pixels
  pad_fix(c, c->act[i + 1], go, c->Cout[i], !last);
  if (last && loss_sum_dev && !c->fc_above) {
    const long long n8 = go.Ptot * c->Cout[i] / 8;
    c->prof->begin(MBD_K_OTHER, static_cast<double>(n8) * 16.0, c->stream);
    ssq_partial_kernel<<<c->loss_grid, 256, 0, c->stream>>>(c->act[i + 1], n8, c->loss_part);
    if (sum_f32_launch(c->loss_part, c->loss_grid, 0.5f, loss_sum_dev, c->stream) != cudaSuccess) return MBD_E_CUDA;
    c->prof->end();
  }
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_forward(GenConv* c, const void* X_nchw, float* loss_sum_dev) {
  mbd_status s = gconv_stage_input(c, X_nchw);
  for (int i = 0; i < c->L && s == MBD_OK; ++i) s = gconv_forward_layer(c, i, loss_sum_dev);
  return s;
}

mbd_status gconv_backward_layer(GenConv* c, int i, float fused_eta) {
  if (i < 0 || i >= c->L) return MBD_E_INVALID;
  const bool own_update = !c->Wm32.empty() || !c->Vm.empty();      // masters / momentum: gradient first, then the update kernel
  const bool fused = fused_eta > 0.f && !own_update;
  const float scale = -fused_eta / static_cast<float>(c->B);
  const Geo& go = c->geo[i + 1];
  const int s = c->stride[i], Cin = c->Cin[i];
  const double flops = 2.0 * c->B * go.H * go.W * c->taps[i] * Cin * c->Cout[i];
  const int ldw = c->ldw[i];
  if (i > 0 || c->need_dx0) {
    bf16* below = i > 0 ? c->dY[i - 1] : c->dX0;
    const int relu_below = i > 0 ? c->relu[i - 1] : c->in_relu;
    // backward halo exchange (second halo term of Eq. 7), then dY_{i-1} = convT(K_i, dY_i) * [X_i > 0] -- with the
    // weights as they are BEFORE this step's update, so this product comes first
    if (c->P_r > 1) pad_fix(c, c->dY[i], go, c->Cout[i], true);
    for (int q = 0; q < s * s; ++q) {
      bf16* outp = s > 1 ? c->dxph[i] + static_cast<size_t>(q) * go.Ptot * Cin : below;
      if (c->bwd_taps[i][q] == 0) {                // (a 1 x 1 kernel with stride 2: three of four planes)
        if (cudaMemsetAsync(outp, 0, static_cast<size_t>(go.Ptot) * Cin * 2, c->stream) != cudaSuccess) return MBD_E_CUDA;
        continue;
      }
      const bf16* maskp = !relu_below ? nullptr : (s > 1 ? c->xph[i] + static_cast<size_t>(q) * go.Ptot * Cin : c->act[i]);
      const Epi ed = make_epi_mask(outp, Cin, maskp, Cin);
      const mbd_status st = run(c, c->bwd_data[i][q], MBD_K_CONV_BWD_DATA, flops * c->bwd_taps[i][q] / c->taps[i], ed);
      if (st != MBD_OK) return st;
    }
    if (s > 1) decimate(c, below, c->dxph[i], c->geo[i], go, Cin, s, false);      // the planes' own pixels back in place
    pad_fix(c, below, c->geo[i], Cin, false);
    if (c->P_r > 1) pad_fix(c, c->dY[i], go, c->Cout[i], false);      // the halo copies must not enter the sum below
  }
  // dY_i is zero outside the strips' own pixels here: every pixel enters the weight gradient once (the sum over the
  // strips and batch blocks is the all-reduce over all P processes, last term of Eq. 9)
  const Epi ew = fused ? make_epi_sgd(c->Wm[i], ldw, scale) : make_epi_act(c->dWm[i], ldw, 0, 0);
  const mbd_status st = run(c, c->bwd_weight[i], MBD_K_CONV_BWD_WEIGHT, flops, ew);
  if (st != MBD_OK) return st;
  if (own_update && fused_eta > 0.f && update_from_gradient(c, i, fused_eta) != MBD_OK) return MBD_E_CUDA;
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_backward(GenConv* c, float fused_eta) {
  mbd_status s = MBD_OK;
  for (int i = c->L - 1; i >= 0 && s == MBD_OK; --i) s = gconv_backward_layer(c, i, fused_eta);
  return s;
}

mbd_status gconv_sgd_step(GenConv* c, float eta) {
  for (int i = 0; i < c->L; ++i)
    if (update_from_gradient(c, i, eta) != MBD_OK) return MBD_E_CUDA;
  return MBD_OK;
}

mbd_status gconv_output_to_nchw(GenConv* c, void* dst) {
  unstage(c, c->act[c->L], static_cast<bf16*>(dst), c->geo[c->L], c->Cout[c->L - 1]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_top_grad_from_nchw(GenConv* c, const void* src) {
  if (!c->fc_above) return MBD_E_STATE;
  stage(c, static_cast<const bf16*>(src), c->dY[c->L - 1], c->geo[c->L], c->Cout[c->L - 1], false);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

// The gradient w.r.t. this stack's input (a stack that continues another one: need_dx0), back in NCHW
mbd_status gconv_input_grad_to_nchw(GenConv* c, void* dst) {
  if (!c->need_dx0) return MBD_E_STATE;
  unstage(c, c->dX0, static_cast<bf16*>(dst), c->geo[0], c->Cin[0]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_get_tensor(GenConv* c, int which, int layer, void* dst, size_t bytes) {
  if (layer < 0 || layer >= c->L) return MBD_E_INVALID;
  if (which == MBD_T_DW || which == MBD_T_MASTER || which == MBD_T_VELOCITY) {
    const long long n = static_cast<long long>(c->Cout[layer]) * c->Cin[layer] * c->taps[layer];
    if (bytes != static_cast<size_t>(n) * 4) return MBD_E_INVALID;
    if ((which == MBD_T_MASTER && c->Wm32.empty()) || (which == MBD_T_VELOCITY && c->Vm.empty())) return MBD_E_STATE;
    const float* src32 = which == MBD_T_DW ? c->dWm[layer] : which == MBD_T_MASTER ? c->Wm32[layer] : c->Vm[layer];
    unpack_w_kernel<float><<<grid_1d(static_cast<long long>(c->Cout[layer]) * c->ldw[layer], c->num_sms), 256, 0, c->stream>>>(
        src32, static_cast<float*>(dst), c->colmap[layer], c->Cout[layer], c->Cin[layer], c->taps[layer], c->ldw[layer]);
    return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
  }
  if (which != MBD_T_ACT && which != MBD_T_DY) return MBD_E_INVALID;
  const int C = c->Cout[layer];
  const Geo& g = c->geo[layer + 1];
  if (bytes != static_cast<size_t>(c->B) * C * g.H * g.W * 2) return MBD_E_INVALID;
  unstage(c, which == MBD_T_ACT ? c->act[layer + 1] : c->dY[layer], static_cast<bf16*>(dst), g, C);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_set_tensor(GenConv* c, int which, int layer, const void* src, size_t bytes) {
  if (layer < 0 || layer >= c->L || which != MBD_T_ACT) return MBD_E_INVALID;
  const int C = c->Cout[layer];
  const Geo& g = c->geo[layer + 1];
  if (bytes != static_cast<size_t>(c->B) * C * g.H * g.W * 2) return MBD_E_INVALID;
  stage(c, static_cast<const bf16*>(src), c->act[layer + 1], g, C, layer + 1 < c->L);
  // a strided layer above reads its phase planes, made from this tensor in its forward pass: refresh them, so that
  // the ReLU decisions of the backward pass are taken on what was just stored
  if (layer + 1 < c->L && c->stride[layer + 1] > 1) {
    const int s = c->stride[layer + 1];
    decimate(c, c->act[layer + 1], c->xph[layer + 1], g, c->geo[layer + 2], C, s, true);
    pad_fix(c, c->xph[layer + 1], c->geo[layer + 2], C, true, s * s);
  }
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

mbd_status gconv_get_product(const GenConv* c, int layer, int product, const TcGemm** out) {
  if (layer < 0 || layer >= c->L) return MBD_E_INVALID;
  if (product == 1 && layer == 0) return MBD_E_INVALID;                 // nothing is propagated below the first layer
  if (product == 1) {                                                   // (a strided layer: the first plane that has taps)
    for (size_t q = 0; q < c->bwd_data[layer].size(); ++q)
      if (c->bwd_taps[layer][q] > 0) { *out = &c->bwd_data[layer][q]; return MBD_OK; }
    return MBD_E_INVALID;
  }
  *out = product == 0 ? &c->fwd[layer] : &c->bwd_weight[layer];
  return MBD_OK;
}

mbd_status gconv_set_dw(GenConv* c, int layer, const void* src, size_t bytes) {
  if (layer < 0 || layer >= c->L) return MBD_E_INVALID;
  const long long n = static_cast<long long>(c->Cout[layer]) * c->ldw[layer];
  if (bytes != static_cast<size_t>(c->Cout[layer]) * c->Cin[layer] * c->taps[layer] * 4) return MBD_E_INVALID;
  pack_w_kernel<float><<<grid_1d(n, c->num_sms), 256, 0, c->stream>>>(static_cast<const float*>(src), c->dWm[layer], c->colmap[layer], c->Cout[layer],
                                                                      c->Cin[layer], c->taps[layer], c->ldw[layer]);
  return cudaGetLastError() == cudaSuccess ? MBD_OK : MBD_E_CUDA;
}

}  // namespace mbd
