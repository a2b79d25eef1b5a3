// Internal interface between the host plan (net.cu) and the kernel files.
// Nothing here is exported; the C ABI lives in include/mbd.h.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace mbd {

// ---- programmatic dependent launch -------------------------------------------------------------
// A kernel launched with launch_pdl may be scheduled before its predecessor in the stream has
// finished (as soon as every CTA of the predecessor has called pdl_trigger() or exited); it must
// call pdl_wait() before it reads or writes anything the predecessor touches.  What comes before
// pdl_wait() -- barrier set-up, tensor-memory allocation, the launch itself -- then overlaps the
// predecessor's tail.  Both calls do nothing in a kernel launched the ordinary way.
// Only the GEMMs are launched this way (cluster_x >= 1; pass 0 for an ordinary launch): a
// memory-bound kernel that becomes resident early just waits beside the product it depends on and
// slowed the split products' steps by 4 % when it was tried.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
bool pdl_enabled();          // false if MBD_NO_PDL is set in the environment

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = static_cast<unsigned>(cluster_x); attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl_enabled() && cluster_x >= 1) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Device status word values (0 = fine).  A kernel that gives up a bounded wait
// stores one of these with atomicCAS(status, 0, code) and returns.
enum : int {
  DEV_OK = 0,
  DEV_TIMEOUT_PRODUCER = 101,   // TMA producer waited too long for a free stage
  DEV_TIMEOUT_MMA_FULL = 102,   // MMA issuer waited too long for operands
  DEV_TIMEOUT_MMA_TMEM = 103,   // MMA issuer waited too long for a drained accumulator
  DEV_TIMEOUT_EPILOGUE = 104,   // epilogue waited too long for a finished accumulator
  DEV_SMEM_MISALIGNED = 105,    // dynamic shared memory did not start on a 1024-byte boundary; nothing ran
  DEV_TIMEOUT_RUNNING_SUM = 106 // epilogue waited too long for the earlier pieces' sum of its tile
};

// What happens to a finished fp32 accumulator element acc at (m, n).
enum EpiOp : int {
  EPI_ACT = 0,    // v = acc (+ bias[n]); relu ? max(v,0) : v; store (bf16 or f32)
  EPI_MASK = 1,   // v = (mask == null || mask[m,n] > 0) ? acc : 0; store (bf16 or f32)
  EPI_SGD = 2     // out[m,n] = out[m,n] + scale * acc   (Eq. 1 with scale = -eta/B); see Epi::master
};

struct Epi {
  int op;
  int out_bf16;        // 1: out (and mask) are bf16, 0: float
  int relu;
  void* out;           // [M, ldo]
  int64_t ldo;
  const float* bias;   // [N] or null
  const void* mask;    // [M, ldmask] in out's dtype, or null
  int64_t ldmask;
  float scale;
  float* master;       // EPI_SGD on bf16 weights: fp32 master copy [M, ldo] (null: none).  The update is applied
                       // to the master and `out` receives the rounded master.
};

// ---- tcgen05 GEMM -----------------------------------------------------------
// variant 0: D[M,N] = A[M,K] B[N,K]^T      (A, B K-contiguous)          forward
// variant 1: D[M,N] = A[M,K] B[K,N]        (B N-contiguous)             backward-data
// variant 2: D[M,N] = A[K,M]^T B[K,N]      (A M-contiguous, B N-cont.)  backward-weight
// A convolution of k_h x k_w taps on tensors stored pixel-major ([pixels][channels], zero padding stored) is a
// contraction whose operand tiles are views of the same tensor shifted by whole pixel rows: tap t reads pixel
// p + off[t].  mode 1 (forward, variant 0): K index = (tap, input channel), padded to `Cp` per tap; the A tile of
// k-block (t, cb) starts at row m0 + off[t], column 64 cb.  mode 2 (backward-data, variant 1): K index = (tap,
// output channel); A tile at row m0 - off[t]; the B tile is rows 64 ob.. of the weight matrix [C_out][taps Cp] at
// column t Cp + n0.  mode 3 (backward-weight, variant 2): K = pixels; the B chunk of output columns n0.. = (tap t,
// channels n0 - t Cp ..) starts at pixel row k0 + off[t].  Rows outside the tensor read as zero (TMA fill).
// A strided layer reads phase-decimated copies of its input stored one after another (plane (a, b) holds the pixels
// (s h' + a, s w' + b)): its offsets then include the plane's start, and backward-data runs once per plane with the
// taps that read it -- `tap[j]` is the position in the weight matrix of the j-th tap of such a subset.
constexpr int MAX_TAPS = 121;      // kernels up to 11 x 11
struct ConvShift {
  int mode, taps, blocks, Cp;      // blocks: 64-wide k-blocks per tap (modes 1, 2)
  int off[MAX_TAPS];
  int tap[MAX_TAPS];               // mode 2: weight-matrix tap of the j-th tap of this product (identity for stride 1)
  int chan_major;                  // mode 2: k-block = (64-channel block, tap) instead of (tap, block): a cut of K into pieces
                                   // is then a cut of the output channels into blocks (model-parallel convolutions)
};

struct TcGemm {
  CUtensorMap tmA, tmB;
  CUtensorMap tmOut, tmAux;   // output / mask-source maps of the TMA epilogue (valid when te)
  int te;                     // plan allows the TMA epilogue for te_epi
  int te_planes;              // out: the S > 1 fp32 planes leave through TMA stores (short pieces on 128-row tiles)
  int te_ring;                // out: one work unit per CTA: the TMA epilogue's staging boxes lie in the idle operand ring
  Epi te_epi;
  int variant;
  int BN;               // CTA tile width: 256 or 128
  int MH;               // CTA tile height in units of 128 rows: 1 or 2
  int pair;             // two CTAs of a cluster share one 256 x 256 tile (cta_group::2)
  int allow_extra_split; // the planner may cut K further than asked (its pieces go through the same reduction)
  int allow_fix;        // in: the S pieces need not be kept as S planes
  int fix;              // out: pieces are added as a running sum in the epilogue (one plane in `partials`, words in
                        // `flags`), in ascending order like the reduction kernel; no reduction launch follows
  int join;             // out: > 1: that many pieces of K are accumulators of their own in tensor memory, added in ascending order by
                        // the epilogue (k_splits is 1 then: nothing is written to `partials`, no reduction launch follows)
  long long flag_words; // out: ints `flags` must hold (zero-initialised; the kernel leaves them zero)
  int* flags;
  int M, N, K;
  int k_splits;         // S >= 1; S > 1 writes partials[S][M][N] (fp32) and skips the epilogue op
  float* partials;
  Epi epi;
  int* status;
  int grid;
  // fp32 planes written by TMA (k_splits > 1 on 128-row tiles): the map over partials[S][M][N], encoded at the
  // first launch that sees `partials` (the workspace is the caller's and is known only then)
  mutable CUtensorMap tmPlanes;
  mutable const float* planes_base = nullptr;
  // Convolution as a contraction over shifted views (set before tc_gemm_prepare; cv.mode = 0: a plain product)
  ConvShift cv = {};
  int64_t cv_a_inner = 0;      // modes 1, 2: channels per pixel of the A tensor (its rows are pixels)
  int64_t cv_a_rows = 0;       // modes 1, 2: rows of the A tensor as stored, if more than M (phase planes); 0 = M
  int64_t cv_b_inner = 0, cv_b_rows = 0;   // modes 2, 3: extent of the B tensor as stored (inner, rows)
};

// The host-side part of tc_gemm_prepare: from M, N, K, variant, k_splits, allow_extra_split, allow_fix it fills BN, MH, pair,
// k_splits, join, fix, flag_words, te_planes, te (`want_te`: a bf16 result behind an epilogue operation), grid.  Touches no device.
void tc_gemm_plan(TcGemm& g, int num_sms, bool want_te);
// Plans (tc_gemm_plan), then fills the tensor maps.  Returns cudaSuccess or an error.
// `te_epi` (may be null): the epilogue this contraction will run with, if its output is bf16;
// lets the plan move the epilogue's global traffic with TMA.
cudaError_t tc_gemm_prepare(TcGemm& g, const void* A, int64_t lda, const void* B, int64_t ldb,
                            int num_sms, const Epi* te_epi);
cudaError_t tc_gemm_launch(const TcGemm& g, cudaStream_t stream);
cudaError_t selftest_timeout_launch(int* status, int limit_ms, cudaStream_t stream);
cudaError_t tc_gemm_init();   // driver entry point lookup + kernel attributes of the current device; idempotent per device

// ---- fp32 SIMT GEMM (check mode) ----------------------------------------------
struct SimtGemm {
  int M, N, K;
  const float* A; int64_t a_sm, a_sk;   // A(m,k) = A[m*a_sm + k*a_sk]
  const float* B; int64_t b_sn, b_sk;   // B(n,k) = B[n*b_sn + k*b_sk]
  int k_splits;                         // balanced ranges [floor(s K/S), floor((s+1) K/S))
  float* partials;                      // [S][M][N] when S > 1
  Epi epi;
};
cudaError_t simt_gemm_launch(const SimtGemm& g, cudaStream_t stream);

// ---- memory-bound kernels ---------------------------------------------------------
// out = sum_{s<S} parts[s] (ascending s), then the epilogue op.  parts is [S][M][N] dense.
cudaError_t reduce_partials_launch(const float* parts, int S, int64_t M, int64_t N, const Epi& epi,
                                   int num_sms, cudaStream_t stream);
cudaError_t softmax_xent_launch(const float* logits, int64_t B, int64_t d, const int32_t* labels,
                                void* dY, int dy_bf16, float* per_sample, cudaStream_t stream);
// sum of n floats in a fixed order into *out (single CTA, deterministic); scale applied.
cudaError_t sum_f32_launch(const float* x, int64_t n, float scale, float* out, cudaStream_t stream);
// db[n] = sum_m dY[m,n]; two deterministic stages through `scratch` [8 * row_splits][N]; the kernels
// use no shared memory, so their CTAs fit on an SM next to a resident tensor-core GEMM CTA.
// If bias != null: bias[n] += scale * db[n].  If db != null: db[n] stored.
cudaError_t colsum_launch(const void* dY, int dy_bf16, int64_t M, int64_t N, float* scratch,
                          int row_splits, float* db, float* bias, float scale, cudaStream_t stream);
int colsum_row_splits(int64_t M, int64_t N, int num_sms);   // at most 32
int colsum_launches(int64_t M, int64_t N, int num_sms);    // kernels one colsum_launch issues
// w[i] += scale * g[i]   (w bf16 or f32, g f32)
cudaError_t sgd_update_launch(void* w, int w_bf16, const float* g, int64_t n, float scale,
                              int num_sms, cudaStream_t stream);

// Heavy-ball momentum: v = mu v + g inv_B; w -= eta v (w fp32, bf16, or bf16 copy of the fp32 master w32).
cudaError_t sgd_momentum_update_launch(void* w, int w_bf16, float* w32, float* v, const float* g, int64_t n, float mu,
                                       float inv_B, float eta, int num_sms, cudaStream_t stream);
// fp32 master weights: w32[i] += scale * g[i]; w_bf16[i] = round(w32[i]).  widen: w32[i] = w_bf16[i].
cudaError_t sgd_master_update_launch(float* w32, void* w_bf16, const float* g, int64_t n, float scale,
                                     int num_sms, cudaStream_t stream);
cudaError_t widen_bf16_launch(const void* w_bf16, float* w32, int64_t n, int num_sms, cudaStream_t stream);

// ---- per-class event timing (host) ---------------------------------------------------------
struct Profiler {
  static constexpr int NCLS = 12;
  bool on = false;
  cudaStream_t stream = nullptr;
  struct Pending { cudaEvent_t a, b; int cls; };
  Pending* pending = nullptr;
  int n_pending = 0, cap = 0;
  cudaEvent_t* pool = nullptr;
  int n_pool = 0, pool_cap = 0;
  double ms[NCLS] = {0}, work[NCLS] = {0};
  long long launches[NCLS] = {0};
  int64_t total_launches = 0;

  cudaEvent_t get_event();
  cudaStream_t cur = nullptr;             // stream of the launch being bracketed
  void begin(int cls, double w, cudaStream_t launch_stream = nullptr);   // null: the main stream
  void end();
  void collect();          // synchronises the stream
  void reset();
  void destroy();
};

// ---- domain-parallel 3x3 convolution (conv.cu) ------------------------------------------
struct ConvNet;   // defined in conv.cu
}  // namespace mbd
