// mbd_gemm_bf16_noalloc: the split-K tensor-core contraction of mbd_gemm_bf16 for callers
// that must not allocate device memory -- a service whose own memory pool was handed the
// whole GPU at start-up and is the only allocator permitted, or a plug-in called on a
// device whose memory is fully given out already, where cudaMalloc would fail or stall.
// The fp32 partial sums and the status word live in a fixed array that is part of this
// library's device image.  The call waits for the stream before it returns (it reads the
// status word back); the first call on a device also looks up the arrays' device addresses
// and sets the kernels' shared-memory attribute for that device.
#include "../../include/mbd.h"
#include "kernels.h"

using namespace mbd;

namespace {

constexpr size_t SCRATCH_FLOATS = size_t(4) << 20;     // 16 MiB of partial sums
constexpr int MAX_DEVICES = 64;

// Held by every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_scratch[SCRATCH_FLOATS];
static __device__ __align__(256) int g_status_word[64];

// Device addresses of the two arrays, looked up once per device.  In host code the names
// above are only handles for the runtime, not device pointers.
float* g_scratch_ptr[MAX_DEVICES] = {nullptr};
int* g_status_ptr[MAX_DEVICES] = {nullptr};

mbd_status setup_device(int dev) {
  if (g_scratch_ptr[dev] && g_status_ptr[dev]) return MBD_OK;
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  void* q = nullptr;
  if (cudaGetSymbolAddress(&q, g_status_word) != cudaSuccess || !q) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  g_scratch_ptr[dev] = static_cast<float*>(p);
  g_status_ptr[dev] = static_cast<int*>(q);
  return MBD_OK;
}

}  // namespace

extern "C" mbd_status mbd_gemm_bf16_noalloc(int variant, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                            const void* Bm, int64_t ldb, float* D, int64_t ldd, int k_splits,
                                            void* cuda_stream) {
  if (!A || !Bm || !D || variant < 0 || variant > 2 || M < 1 || N < 1 || K < 1 || k_splits < 1) return MBD_E_INVALID;
  if (lda % 8 || ldb % 8 || ldd % 8 || N % 8) return MBD_E_UNSUPPORTED;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return MBD_E_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(Bm) | reinterpret_cast<uintptr_t>(D)) & 15u)
    return MBD_E_UNSUPPORTED;                              // TMA and the 16-byte stores need 16-byte aligned bases
  const int64_t kb = (K + 63) / 64;
  const int64_t S = k_splits < kb ? k_splits : kb;
  if (S > 1 && static_cast<unsigned __int128>(S) * M * N > SCRATCH_FLOATS) return MBD_E_TOO_LARGE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MBD_E_CUDA;
  if (dev < 0 || dev >= MAX_DEVICES) return MBD_E_UNSUPPORTED;
  mbd_status st = setup_device(dev);
  if (st != MBD_OK) return st;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MBD_E_CUDA;
  float* scratch = g_scratch_ptr[dev];
  int* status = g_status_ptr[dev];
  // The arrays keep whatever the previous call left: the status word must start at zero;
  // the partial sums need no clearing because every element that is read is written first.
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  TcGemm g{};
  g.variant = variant;
  g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
  g.k_splits = static_cast<int>(S);
  g.status = status;
  if (tc_gemm_prepare(g, A, lda, Bm, ldb, sms, nullptr) != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  g.epi = Epi{};
  g.epi.op = EPI_ACT; g.epi.out = D; g.epi.ldo = ldd;
  g.partials = scratch;
  if (tc_gemm_launch(g, stream) != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  if (g.k_splits > 1 && reduce_partials_launch(scratch, g.k_splits, M, N, g.epi, sms, stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return MBD_E_CUDA;
  }
  if (cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  int h = 0;
  if (cudaMemcpy(&h, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { (void)cudaGetLastError(); return MBD_E_CUDA; }
  return h == 0 ? MBD_OK : MBD_E_TIMEOUT;
}
