// Stand-alone block operations on caller-owned device buffers: what ONE process of the P_r x P_c grid does
// between two collectives (Section 2.3; Appendix A.1 / A.2) -- a block product with its tail operation
// fused, the tail operation applied to a sum that arrived from a collective, and the loss.  They let a
// multi-process driver run the grid for real, every arithmetic step in these kernels and only the
// exchange outside.  With a caller-owned status word a call only enqueues (the caller reads the word when it
// likes: non-zero = a bounded wait gave up); without one the call allocates a word, waits for the stream and
// reports what it found.
#include "../../include/mbd.h"
#include "kernels.h"

using namespace mbd;

namespace {

bool to_epi(const mbd_tail* t, Epi* e) {
  if (!t || !t->out_dev || t->ldo < 1) return false;
  if (t->op != MBD_TAIL_STORE && t->op != MBD_TAIL_MASK && t->op != MBD_TAIL_SGD) return false;
  *e = Epi{};
  e->op = t->op == MBD_TAIL_STORE ? EPI_ACT : t->op == MBD_TAIL_MASK ? EPI_MASK : EPI_SGD;
  e->out_bf16 = t->out_bf16 != 0;
  e->relu = t->relu != 0;
  e->out = t->out_dev;
  e->ldo = t->ldo;
  e->bias = t->bias_dev;
  e->mask = t->mask_dev;
  e->ldmask = t->ldmask;
  e->scale = t->scale;
  return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct StatusWord {
  int* dev = nullptr;
  bool alloc(cudaStream_t s) {
    if (cudaMalloc(reinterpret_cast<void**>(&dev), sizeof(int)) != cudaSuccess) { (void)cudaGetLastError(); dev = nullptr; return false; }
    return cudaMemsetAsync(dev, 0, sizeof(int), s) == cudaSuccess;
  }
  mbd_status finish(cudaStream_t s, mbd_status ret) {
    if (ret == MBD_OK) {
      int h = 0;
      if (cudaStreamSynchronize(s) != cudaSuccess || cudaMemcpy(&h, dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) ret = MBD_E_CUDA;
      else if (h != 0) ret = h == DEV_SMEM_MISALIGNED ? MBD_E_CUDA : MBD_E_TIMEOUT;
    }
    (void)cudaGetLastError();
    cudaFree(dev);
    return ret;
  }
};

}  // namespace

extern "C" mbd_status mbd_block_gemm_bf16(int variant, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                          const void* Bm, int64_t ldb, const mbd_tail* tail, int32_t* status_dev,
                                          void* cuda_stream) {
  Epi epi;
  if (!A || !Bm || variant < 0 || variant > 2 || M < 1 || N < 1 || K < 1 || !to_epi(tail, &epi)) return MBD_E_INVALID;
  if (lda % 8 || ldb % 8 || epi.ldo % 8 || N % 8 || (epi.mask && epi.ldmask % 8)) return MBD_E_UNSUPPORTED;
  // TMA and the 16-byte accesses of the epilogue need 16-byte aligned bases (a view may start anywhere)
  if (!aligned16(A) || !aligned16(Bm) || !aligned16(epi.out) || !aligned16(epi.mask) || !aligned16(epi.bias)) return MBD_E_UNSUPPORTED;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return MBD_E_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return MBD_E_CUDA;
  }
  StatusWord st;
  if (status_dev) st.dev = status_dev;
  else if (!st.alloc(stream)) return MBD_E_ALLOC;
  TcGemm g{};
  g.variant = variant;
  g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
  g.k_splits = 1;
  g.status = st.dev;
  mbd_status ret = MBD_OK;
  if (tc_gemm_prepare(g, A, lda, Bm, ldb, sms, epi.out_bf16 ? &epi : nullptr) != cudaSuccess) ret = MBD_E_CUDA;
  if (ret == MBD_OK) {
    g.epi = epi;
    g.partials = nullptr;
    if (tc_gemm_launch(g, stream) != cudaSuccess) ret = MBD_E_CUDA;
  }
  if (status_dev) {                      // enqueue-only: the caller owns and reads the status word
    if (ret != MBD_OK) (void)cudaGetLastError();
    return ret;
  }
  return st.finish(stream, ret);
}

extern "C" mbd_status mbd_block_reduce(const float* parts, int S, int64_t M, int64_t N, const mbd_tail* tail,
                                       int sync, void* cuda_stream) {
  Epi epi;
  if (!parts || S < 1 || M < 1 || N < 1 || !to_epi(tail, &epi)) return MBD_E_INVALID;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      reduce_partials_launch(parts, S, M, N, epi, sms, stream) != cudaSuccess ||
      (sync && cudaStreamSynchronize(stream) != cudaSuccess)) {
    (void)cudaGetLastError();
    return MBD_E_CUDA;
  }
  return MBD_OK;
}

extern "C" mbd_status mbd_softmax_xent(const float* logits, int64_t B, int64_t d, const int32_t* labels, void* dY,
                                       int dY_bf16, float* per_sample, int sync, void* cuda_stream) {
  if (!logits || !labels || !dY || !per_sample || B < 1 || d < 1) return MBD_E_INVALID;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (softmax_xent_launch(logits, B, d, labels, dY, dY_bf16 != 0, per_sample, stream) != cudaSuccess ||
      (sync && cudaStreamSynchronize(stream) != cudaSuccess)) {
    (void)cudaGetLastError();
    return MBD_E_CUDA;
  }
  return MBD_OK;
}
