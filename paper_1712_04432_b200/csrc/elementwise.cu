// Memory-bound kernels of the training step:
//   reduce_partials  sum of the per-block fp32 partial sums in ascending block order,
//                    standing in for the all-reduce over the P_r group (dX) or the P_c
//                    group (dW) of Section 2.3 / Appendix A.2, with the tail operation
//                    (ReLU mask, SGD update, plain store) fused
//   softmax_xent     loss and top gradient dY_L = softmax(Y_L) - onehot
//   colsum           db = dY 1 (bias gradient), deterministic two-stage
//   sgd_update       Eq. 1 applied to materialised gradients
//   sum_f32          fixed-order sum (total loss)
// All of them are bound by HBM bandwidth: 16-byte accesses, grids sized in multiples of
// the SM count, no atomics on floats (results are bitwise reproducible).
#include "epi.cuh"

namespace mbd {
namespace {

// ------------------------------------------------------------------ reduce_partials
// Vector path: M*N and N multiples of 8; each thread owns 8 consecutive columns of a row.
__global__ void __launch_bounds__(256)
reduce_partials_vec8(const float* __restrict__ parts, int S, int64_t M, int64_t N, const Epi epi) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  const int64_t n8 = N >> 3;
  const int64_t total = M * n8;
  const int64_t plane = M * N;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t m = i / n8;
    const int64_t n0 = (i - m * n8) << 3;
    const float* src = parts + m * N + n0;
    float4 a = __ldcs(reinterpret_cast<const float4*>(src));
    float4 b = __ldcs(reinterpret_cast<const float4*>(src + 4));
    for (int s = 1; s < S; ++s) {
      const float4 c = __ldcs(reinterpret_cast<const float4*>(src + s * plane));
      const float4 d = __ldcs(reinterpret_cast<const float4*>(src + s * plane + 4));
      a.x += c.x; a.y += c.y; a.z += c.z; a.w += c.w;
      b.x += d.x; b.y += d.y; b.z += d.z; b.w += d.w;
    }
    float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    epi_apply8(epi, m, n0, v);
  }
}

// The common case of two planes: a thread handles two pieces per iteration and issues the loads of both planes
// of both pieces before the first add, so that enough bytes are in flight per SM (5.7 -> 6.0 TB/s on 268 MB planes).
__global__ void __launch_bounds__(256)
reduce_partials_vec8_two_planes(const float* __restrict__ parts, int64_t M, int64_t N, const Epi epi) {
  pdl_wait();
  const int64_t n8 = N >> 3;
  const int64_t total = M * n8;
  const int64_t plane = M * N;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i0 = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i0 < total; i0 += 2 * stride) {
    const int64_t i1 = i0 + stride;
    const bool two = i1 < total;
    const int64_t m0 = i0 / n8, m1 = two ? i1 / n8 : m0;
    const int64_t c0 = (i0 - m0 * n8) << 3, c1 = two ? (i1 - m1 * n8) << 3 : c0;
    const float* s0 = parts + m0 * N + c0;
    const float* s1 = parts + m1 * N + c1;
    float4 a0 = __ldcs(reinterpret_cast<const float4*>(s0)), b0 = __ldcs(reinterpret_cast<const float4*>(s0 + 4));
    float4 a1 = __ldcs(reinterpret_cast<const float4*>(s1)), b1 = __ldcs(reinterpret_cast<const float4*>(s1 + 4));
    const float4 p0 = __ldcs(reinterpret_cast<const float4*>(s0 + plane)), q0 = __ldcs(reinterpret_cast<const float4*>(s0 + plane + 4));
    const float4 p1 = __ldcs(reinterpret_cast<const float4*>(s1 + plane)), q1 = __ldcs(reinterpret_cast<const float4*>(s1 + plane + 4));
    a0.x += p0.x; a0.y += p0.y; a0.z += p0.z; a0.w += p0.w; b0.x += q0.x; b0.y += q0.y; b0.z += q0.z; b0.w += q0.w;
    a1.x += p1.x; a1.y += p1.y; a1.z += p1.z; a1.w += p1.w; b1.x += q1.x; b1.y += q1.y; b1.z += q1.z; b1.w += q1.w;
    float v0[8] = {a0.x, a0.y, a0.z, a0.w, b0.x, b0.y, b0.z, b0.w};
    epi_apply8(epi, m0, c0, v0);
    if (two) {
      float v1[8] = {a1.x, a1.y, a1.z, a1.w, b1.x, b1.y, b1.z, b1.w};
      epi_apply8(epi, m1, c1, v1);
    }
  }
}

__global__ void __launch_bounds__(256)
reduce_partials_scalar(const float* __restrict__ parts, int S, int64_t M, int64_t N, const Epi epi) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  const int64_t total = M * N;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float a = parts[i];
    for (int s = 1; s < S; ++s) a += parts[i + s * total];
    const int64_t m = i / N;
    epi_apply1(epi, m, i - m * N, a);
  }
}

// ------------------------------------------------------------------ softmax cross-entropy
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One CTA of NW warps per sample (row).  Three passes over the row (max, sum of exp,
// write); the row (<= 32 KB) stays in L1/L2 between them.
template <int NW>
__global__ void __launch_bounds__(NW * 32)
softmax_xent_kernel(const float* __restrict__ logits, int64_t d, const int32_t* __restrict__ labels,
                    void* __restrict__ dY, int dy_bf16, float* __restrict__ per_sample) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  __shared__ float red[NW];
  const int64_t b = blockIdx.x;
  const float* row = logits + b * d;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float mx = -INFINITY;
  for (int64_t k = tid; k < d; k += NW * 32) mx = fmaxf(mx, row[k]);
  mx = warp_max(mx);
  if (NW > 1) {
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) mx = fmaxf(mx, red[i]);
    __syncthreads();
  }
  float sum = 0.f;
  for (int64_t k = tid; k < d; k += NW * 32) sum += expf(row[k] - mx);
  sum = warp_sum(sum);
  if (NW > 1) {
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    sum = red[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) sum += red[i];
  }
  const float inv = 1.f / sum;
  const int label = labels[b];
  for (int64_t k = tid; k < d; k += NW * 32) {
    float g = expf(row[k] - mx) * inv;
    if (k == label) g -= 1.f;
    if (dy_bf16) reinterpret_cast<__nv_bfloat16*>(dY)[b * d + k] = __float2bfloat16_rn(g);
    else reinterpret_cast<float*>(dY)[b * d + k] = g;
  }
  // a label outside [0, d) is never used as an index: the sample's loss is reported as NaN
  if (tid == 0) per_sample[b] = (label >= 0 && label < d) ? mx + logf(sum) - row[label] : __int_as_float(0x7fc00000);
}

// Same, with the whole row held in registers (VPT values per thread): one pass over HBM.
// VEC: d is a multiple of 4 and every thread owns groups of 4 consecutive classes (16-byte loads).
template <int NW, int VPT, bool VEC>
__global__ void __launch_bounds__(NW * 32)
softmax_xent_reg_kernel(const float* __restrict__ logits, int64_t d, const int32_t* __restrict__ labels,
                        void* __restrict__ dY, int dy_bf16, float* __restrict__ per_sample) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  __shared__ float red[NW];
  const int64_t b = blockIdx.x;
  const float* row = logits + b * d;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int G = VEC ? 4 : 1;                 // consecutive classes per group
  auto index = [&](int i) -> int64_t { return (static_cast<int64_t>(i / G) * NW * 32 + tid) * G + (i % G); };
  float v[VPT];
  float mx = -INFINITY;
  if (VEC) {
#pragma unroll
    for (int i = 0; i < VPT; i += 4) {
      const int64_t k = index(i);
      float4 q = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      if (k < d) q = __ldcs(reinterpret_cast<const float4*>(row + k));
      v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int64_t k = index(i);
      v[i] = k < d ? __ldcs(row + k) : -INFINITY;
    }
  }
#pragma unroll
  for (int i = 0; i < VPT; ++i) mx = fmaxf(mx, v[i]);
  mx = warp_max(mx);
  if (NW > 1) {
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) mx = fmaxf(mx, red[i]);
    __syncthreads();
  }
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < VPT; ++i) { v[i] = expf(v[i] - mx); sum += v[i]; }     // exp(-inf) = 0 past the end
  sum = warp_sum(sum);
  if (NW > 1) {
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    sum = red[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) sum += red[i];
  }
  const float inv = 1.f / sum;
  const int label = labels[b];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    v[i] *= inv;
    if (index(i) == label) v[i] -= 1.f;
  }
  if (VEC) {
#pragma unroll
    for (int i = 0; i < VPT; i += 4) {
      const int64_t k = index(i);
      if (k < d) {
        if (dy_bf16) {
          uint2 o;
          o.x = pack_bf16x2(v[i], v[i + 1]); o.y = pack_bf16x2(v[i + 2], v[i + 3]);
          *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(dY) + b * d + k) = o;
        } else {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(dY) + b * d + k) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        }
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int64_t k = index(i);
      if (k < d) {
        if (dy_bf16) reinterpret_cast<__nv_bfloat16*>(dY)[b * d + k] = __float2bfloat16_rn(v[i]);
        else reinterpret_cast<float*>(dY)[b * d + k] = v[i];
      }
    }
  }
  if (tid == 0) per_sample[b] = (label >= 0 && label < d) ? mx + logf(sum) - row[label] : __int_as_float(0x7fc00000);
}

// ------------------------------------------------------------------ fixed-order sum
__global__ void __launch_bounds__(1024)
sum_f32_kernel(const float* __restrict__ x, int64_t n, float scale, float* __restrict__ out) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  __shared__ float red[1024];
  float a = 0.f;
  for (int64_t i = threadIdx.x; i < n; i += 1024) a += x[i];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 512; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = red[0] * scale;
}

// ------------------------------------------------------------------ column sums (bias gradient)
// Stage 1: grid (ceil(N/256), row_splits); 256 threads = 8 warps; a lane owns 8 consecutive
// columns (one 16-byte load per row for bf16), a warp 256 columns, the 8 warps stride over the
// rows of this split.  Every warp stores its own partial row, scratch[(split * 8 + warp)][N];
// stage 2 adds the 8 * row_splits rows in a fixed order.  No shared memory: the CTAs fit on an SM next
// to a resident tensor-core GEMM CTA, so the kernel can run on the side stream under a product.
template <bool BF16>
__global__ void __launch_bounds__(256)
colsum_stage1(const void* __restrict__ dY, int64_t M, int64_t N, int row_splits, float* __restrict__ scratch) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t n0 = static_cast<int64_t>(blockIdx.x) * 256 + lane * 8;
  const int64_t r0 = (static_cast<int64_t>(blockIdx.y) * M) / row_splits;
  const int64_t r1 = (static_cast<int64_t>(blockIdx.y + 1) * M) / row_splits;
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = 0.f;
  const bool vec = (N % 8 == 0) && n0 + 8 <= N;
  for (int64_t m = r0 + warp; m < r1; m += 8) {
    if (vec) {
      if (BF16) {
        const uint4 q = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(dY) + m * N + n0));
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { a[2 * i] += bf16_bits_to_f32(w[i] & 0xFFFFu); a[2 * i + 1] += bf16_bits_to_f32(w[i] >> 16); }
      } else {
        const float* p = reinterpret_cast<const float*>(dY) + m * N + n0;
        const float4 u = *reinterpret_cast<const float4*>(p), v = *reinterpret_cast<const float4*>(p + 4);
        a[0] += u.x; a[1] += u.y; a[2] += u.z; a[3] += u.w; a[4] += v.x; a[5] += v.y; a[6] += v.z; a[7] += v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (n0 + i < N) {
          a[i] += BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(dY)[m * N + n0 + i])
                       : reinterpret_cast<const float*>(dY)[m * N + n0 + i];
        }
      }
    }
  }
  float* dst = scratch + (static_cast<int64_t>(blockIdx.y) * 8 + warp) * N + n0;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (n0 + i < N) dst[i] = a[i];
}

// Stage 2: a warp owns 4 columns; the partial rows of a column are shared out over 8 lanes (contiguous row
// ranges, each added in row order with eight loads in flight) and the 8 sub-sums are gathered by shuffles and
// added in lane order: a fixed order, a chain of rows / 64 dependent iterations instead of rows / 8, and still
// no shared memory (see stage 1).
__global__ void __launch_bounds__(256)
colsum_stage2(const float* __restrict__ scratch, int rows, int64_t N, float* __restrict__ db,
              float* __restrict__ bias, float scale) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col = lane & 3, grp = lane >> 2;
  const int64_t n = (blockIdx.x * 8ll + warp) * 4 + col;
  const int r0 = (grp * rows) / 8, r1 = ((grp + 1) * rows) / 8;
  float s = 0.f;
  if (n < N) {
    int r = r0;
    for (; r + 8 <= r1; r += 8) {
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = scratch[static_cast<int64_t>(r + j) * N + n];
#pragma unroll
      for (int j = 0; j < 8; ++j) s += v[j];
    }
    for (; r < r1; ++r) s += scratch[static_cast<int64_t>(r) * N + n];
  }
  float total = 0.f;
#pragma unroll
  for (int g = 0; g < 8; ++g) total += __shfl_sync(0xffffffffu, s, g * 4 + col);   // ascending group order
  if (grp != 0 || n >= N) return;
  if (db) db[n] = total;
  if (bias) bias[n] = fmaf(scale, total, bias[n]);
}

// ------------------------------------------------------------------ SGD update (Eq. 1)
__global__ void __launch_bounds__(256)
sgd_update_bf16_vec8(__nv_bfloat16* __restrict__ w, const float* __restrict__ g, int64_t n8, float scale) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n8;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(g + i * 8));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(g + i * 8 + 4));
    uint4* p = reinterpret_cast<uint4*>(w + i * 8);
    const uint4 q = *p;
    uint4 o;
    o.x = pack_bf16x2(fmaf(scale, a.x, bf16_bits_to_f32(q.x & 0xFFFFu)), fmaf(scale, a.y, bf16_bits_to_f32(q.x >> 16)));
    o.y = pack_bf16x2(fmaf(scale, a.z, bf16_bits_to_f32(q.y & 0xFFFFu)), fmaf(scale, a.w, bf16_bits_to_f32(q.y >> 16)));
    o.z = pack_bf16x2(fmaf(scale, b.x, bf16_bits_to_f32(q.z & 0xFFFFu)), fmaf(scale, b.y, bf16_bits_to_f32(q.z >> 16)));
    o.w = pack_bf16x2(fmaf(scale, b.z, bf16_bits_to_f32(q.w & 0xFFFFu)), fmaf(scale, b.w, bf16_bits_to_f32(q.w >> 16)));
    *p = o;
  }
}

__global__ void __launch_bounds__(256)
sgd_update_scalar(void* __restrict__ w, int w_bf16, const float* __restrict__ g, int64_t n, float scale) {
  pdl_wait();                            // everything this kernel reads or overwrites comes from earlier kernels
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    if (w_bf16) {
      __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(w) + i;
      *p = __float2bfloat16_rn(fmaf(scale, g[i], __bfloat162float(*p)));
    } else {
      float* p = reinterpret_cast<float*>(w) + i;
      *p = fmaf(scale, g[i], *p);
    }
  }
}

// Eq. 1 on fp32 master weights: w32 += scale * g, and the bf16 working copy the contractions read is the
// rounded master (updates smaller than half a bf16 ulp are kept in the master instead of being lost).
__global__ void __launch_bounds__(256)
sgd_master_update_kernel(float* __restrict__ w32, __nv_bfloat16* __restrict__ w, const float* __restrict__ g, int64_t n,
                         float scale) {
  pdl_wait();
  const int64_t n4 = n >> 2;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n4;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(g + i * 4));
    float4 m = *reinterpret_cast<const float4*>(w32 + i * 4);
    m.x = fmaf(scale, a.x, m.x); m.y = fmaf(scale, a.y, m.y); m.z = fmaf(scale, a.z, m.z); m.w = fmaf(scale, a.w, m.w);
    *reinterpret_cast<float4*>(w32 + i * 4) = m;
    uint2 o;
    o.x = pack_bf16x2(m.x, m.y);
    o.y = pack_bf16x2(m.z, m.w);
    *reinterpret_cast<uint2*>(w + i * 4) = o;
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {          // tail
    const int64_t i = (n4 << 2) + threadIdx.x;
    const float m = fmaf(scale, g[i], w32[i]);
    w32[i] = m;
    w[i] = __float2bfloat16_rn(m);
  }
}

__global__ void __launch_bounds__(256)
widen_bf16_kernel(const __nv_bfloat16* __restrict__ w, float* __restrict__ w32, int64_t n) {
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x)
    w32[i] = __bfloat162float(w[i]);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int grid_for(int64_t work_items, int num_sms, int per_sm) {
  int64_t blocks = (work_items + 255) / 256;
  const int64_t cap = static_cast<int64_t>(num_sms) * per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

}  // namespace

cudaError_t reduce_partials_launch(const float* parts, int S, int64_t M, int64_t N, const Epi& epi, int num_sms,
                                   cudaStream_t stream) {
  // 16-byte accesses need 16-byte aligned bases as well as leading dimensions that are multiples of 8; a
  // caller's view that starts at an odd offset goes through the element-wise kernel instead
  const bool vec = (N % 8 == 0) && (epi.ldo % 8 == 0) && (epi.mask == nullptr || epi.ldmask % 8 == 0) &&
                   aligned16(parts) && aligned16(epi.out) && aligned16(epi.mask) && aligned16(epi.bias) && aligned16(epi.master);
  if (vec) {
    // two planes of at least 8 MB: the two-piece kernel; small or many-plane sums: the plain one
    if (S == 2 && M * N >= (2 << 20))
      return launch_pdl(reduce_partials_vec8_two_planes, dim3(grid_for((M * (N / 8) + 1) / 2, num_sms, 8)), dim3(256), 0, stream, 0, parts, M, N, epi);
    return launch_pdl(reduce_partials_vec8, dim3(grid_for(M * (N / 8), num_sms, 8)), dim3(256), 0, stream, 0, parts, S, M, N, epi);
  }
  return launch_pdl(reduce_partials_scalar, dim3(grid_for(M * N, num_sms, 8)), dim3(256), 0, stream, 0, parts, S, M, N, epi);
}

cudaError_t softmax_xent_launch(const float* logits, int64_t B, int64_t d, const int32_t* labels, void* dY,
                                int dy_bf16, float* per_sample, cudaStream_t stream) {
  const unsigned nb = static_cast<unsigned>(B);
  const bool vec = d % 4 == 0 && aligned16(logits) && aligned16(dY);
  if (d <= 64) return launch_pdl(softmax_xent_reg_kernel<1, 2, false>, dim3(nb), dim3(32), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
  if (d <= 1024 && vec) return launch_pdl(softmax_xent_reg_kernel<4, 8, true>, dim3(nb), dim3(128), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
  if (d <= 1024) return launch_pdl(softmax_xent_reg_kernel<4, 8, false>, dim3(nb), dim3(128), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
  if (d <= 8192 && vec) return launch_pdl(softmax_xent_reg_kernel<8, 32, true>, dim3(nb), dim3(256), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
  if (d <= 8192) return launch_pdl(softmax_xent_reg_kernel<8, 32, false>, dim3(nb), dim3(256), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
  return launch_pdl(softmax_xent_kernel<8>, dim3(nb), dim3(256), 0, stream, 0, logits, d, labels, dY, dy_bf16, per_sample);
}

cudaError_t sum_f32_launch(const float* x, int64_t n, float scale, float* out, cudaStream_t stream) {
  return launch_pdl(sum_f32_kernel, dim3(1), dim3(1024), 0, stream, 0, x, n, scale, out);
}

// Row splits (<= 32) so that the first stage has about eight CTAs per SM and every warp of a CTA
// (each writes a partial row of its own) at least eight rows to add.
int colsum_row_splits(int64_t M, int64_t N, int num_sms) {
  const int64_t gx = (N + 255) / 256;
  int64_t r = (8 * static_cast<int64_t>(num_sms) + gx - 1) / gx;
  if (r > M / 64) r = M / 64;
  if (r > 32) r = 32;
  if (r < 1) r = 1;
  return static_cast<int>(r);
}

int colsum_launches(int64_t, int64_t, int) { return 2; }

cudaError_t colsum_launch(const void* dY, int dy_bf16, int64_t M, int64_t N, float* scratch, int row_splits,
                          float* db, float* bias, float scale, cudaStream_t stream) {
  dim3 g1(static_cast<unsigned>((N + 255) / 256), row_splits);
  cudaError_t e = dy_bf16 ? launch_pdl(colsum_stage1<true>, g1, dim3(256), 0, stream, 0, dY, M, N, row_splits, scratch)
                          : launch_pdl(colsum_stage1<false>, g1, dim3(256), 0, stream, 0, dY, M, N, row_splits, scratch);
  if (e != cudaSuccess) return e;
  return launch_pdl(colsum_stage2, dim3(static_cast<unsigned>((N + 31) / 32)), dim3(256), 0, stream, 0, static_cast<const float*>(scratch),
                    row_splits * 8, N, db, bias, scale);
}

// Heavy-ball momentum, the first-order method next to plain SGD (Section 2: the analysis holds for any of them):
//   v <- mu v + g / B ;  w <- w - eta v        (v starts at zero; mu = 0 is Eq. 1)
// on fp32 weights, bf16 weights (one rounding of the new weight) or an fp32 master whose rounding is the bf16 copy.
__global__ void __launch_bounds__(256)
sgd_momentum_update_kernel(void* __restrict__ w, int w_bf16, float* __restrict__ w32, float* __restrict__ v,
                           const float* __restrict__ g, int64_t n, float mu, float inv_B, float eta) {
  pdl_wait();
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const float vel = fmaf(mu, v[i], g[i] * inv_B);
    v[i] = vel;
    if (w_bf16) {
      __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(w) + i;
      const float old = w32 ? w32[i] : __bfloat162float(*p);
      const float nw = fmaf(-eta, vel, old);
      if (w32) w32[i] = nw;
      *p = __float2bfloat16_rn(nw);
    } else {
      float* p = reinterpret_cast<float*>(w) + i;
      *p = fmaf(-eta, vel, *p);
    }
  }
}

cudaError_t sgd_momentum_update_launch(void* w, int w_bf16, float* w32, float* v, const float* g, int64_t n, float mu,
                                       float inv_B, float eta, int num_sms, cudaStream_t stream) {
  return launch_pdl(sgd_momentum_update_kernel, dim3(grid_for(n, num_sms, 8)), dim3(256), 0, stream, 0, w, w_bf16, w32, v, g, n,
                    mu, inv_B, eta);
}

cudaError_t sgd_update_launch(void* w, int w_bf16, const float* g, int64_t n, float scale, int num_sms,
                              cudaStream_t stream) {
  if (w_bf16 && n % 8 == 0) {
    return launch_pdl(sgd_update_bf16_vec8, dim3(grid_for(n / 8, num_sms, 8)), dim3(256), 0, stream, 0, reinterpret_cast<__nv_bfloat16*>(w), g, n / 8, scale);
  }
  return launch_pdl(sgd_update_scalar, dim3(grid_for(n, num_sms, 8)), dim3(256), 0, stream, 0, w, w_bf16, g, n, scale);
}

cudaError_t sgd_master_update_launch(float* w32, void* w_bf16, const float* g, int64_t n, float scale, int num_sms,
                                     cudaStream_t stream) {
  return launch_pdl(sgd_master_update_kernel, dim3(grid_for((n + 3) / 4, num_sms, 8)), dim3(256), 0, stream, 0, w32,
                    reinterpret_cast<__nv_bfloat16*>(w_bf16), g, n, scale);
}

cudaError_t widen_bf16_launch(const void* w_bf16, float* w32, int64_t n, int num_sms, cudaStream_t stream) {
  widen_bf16_kernel<<<grid_for(n, num_sms, 8), 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(w_bf16), w32, n);
  return cudaGetLastError();
}

}  // namespace mbd
