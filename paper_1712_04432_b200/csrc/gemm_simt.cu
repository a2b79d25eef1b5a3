// fp32 contraction on the ordinary FP32 pipes (no tensor cores): the check mode whose
// results must agree with the fp64 oracle to 1e-5, and the path of the small fp32
// workload.  Same three products and the same K-range partial sums as the tensor-core
// kernel; operands are addressed through (row, k) strides so no transposed copy exists.
#include "epi.cuh"

namespace mbd {
namespace {

// 256 threads as 16 x 16; each thread owns an R x R micro-tile of a (16R) x (16R) CTA tile.
// R = 4 for large outputs, R = 2 (with a deeper K step, fewer load-sync round trips) when
// 64 x 64 tiles would leave most SMs idle.
template <int R>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(const SimtGemm g) {
  pdl_wait();                            // operands come from earlier kernels
  constexpr int TM = 16 * R, TN = 16 * R;
  constexpr int TK = R == 2 ? 64 : 16;
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM;
  const int64_t n0 = static_cast<int64_t>(blockIdx.x) * TN;
  const int s = blockIdx.z;
  const int k_lo = static_cast<int>((static_cast<int64_t>(s) * g.K) / g.k_splits);
  const int k_hi = static_cast<int>((static_cast<int64_t>(s + 1) * g.K) / g.k_splits);
  const bool a_kcontig = g.a_sk == 1, b_kcontig = g.b_sk == 1;

  float acc[R][R];
#pragma unroll
  for (int i = 0; i < R; ++i)
#pragma unroll
    for (int j = 0; j < R; ++j) acc[i][j] = 0.f;

  for (int k0 = k_lo; k0 < k_hi; k0 += TK) {
#pragma unroll
    for (int i = 0; i < (TM * TK) / 256; ++i) {
      const int e = tid + i * 256;
      int row, kk;
      if (a_kcontig) { row = e / TK; kk = e % TK; } else { row = e % TM; kk = e / TM; }
      const int64_t m = m0 + row;
      const int k = k0 + kk;
      As[kk][row] = (m < g.M && k < k_hi) ? g.A[m * g.a_sm + k * g.a_sk] : 0.f;
      if (b_kcontig) { row = e / TK; kk = e % TK; } else { row = e % TN; kk = e / TN; }
      const int64_t n = n0 + row;
      const int kb = k0 + kk;
      Bs[kk][row] = (n < g.N && kb < k_hi) ? g.B[n * g.b_sn + kb * g.b_sk] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[R], b[R];
#pragma unroll
      for (int i = 0; i < R; ++i) a[i] = As[kk][ty * R + i];
#pragma unroll
      for (int j = 0; j < R; ++j) b[j] = Bs[kk][tx * R + j];
#pragma unroll
      for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < R; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  float* part = g.k_splits > 1 ? g.partials + static_cast<int64_t>(s) * g.M * g.N : nullptr;
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int64_t m = m0 + ty * R + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < R; ++j) {
      const int64_t n = n0 + tx * R + j;
      if (n >= g.N) continue;
      if (part) part[m * g.N + n] = acc[i][j];
      else epi_apply1(g.epi, m, n, acc[i][j]);
    }
  }
}

}  // namespace

cudaError_t simt_gemm_launch(const SimtGemm& g, cudaStream_t stream) {
  const long long big = 1ll * ((g.N + 63) / 64) * ((g.M + 63) / 64) * g.k_splits;
  if (big >= 148) {
    dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, g.k_splits);
    return launch_pdl(simt_gemm_kernel<4>, grid, dim3(256), 0, stream, 1, g);
  }
  dim3 grid((g.N + 31) / 32, (g.M + 31) / 32, g.k_splits);
  return launch_pdl(simt_gemm_kernel<2>, grid, dim3(256), 0, stream, 1, g);
}

}  // namespace mbd
