// Host plan and C ABI: owns the device state of one network, fixes the launch order of
// a training step (Section 1; Appendix A.1/A.2) and maps the logical P_r x P_c grid of
// Section 2.3 onto K-range partial sums.
//
//   forward   i = 1..L : Y_i = W_i X_i (+b), X_{i+1} = ReLU(Y_i); loss and dY_L
//   backward  i = L..1 : db_i; dX_i (i >= 2) as a sum over P_r row blocks of W_i, then the
//                        ReLU mask; dW_i as a sum over P_c batch blocks, then Eq. 1
// A sum over P blocks is taken as S = min(P, max_partials) fp32 partials (each chaining
// P/S consecutive blocks inside the accumulator) followed by reduce_partials.  The update
// of W_i is ordered after the dX_i product of the same layer, which still reads the old W_i.
#include <algorithm>
#include <new>
#include <stdlib.h>
#include <vector>

#include "../../include/mbd.h"
#include "conv.h"
#include "kernels.h"

using namespace mbd;

namespace {

enum { ST_IDLE = 0, ST_FWD = 1, ST_BWD_UNFUSED = 2, ST_BWD_FUSED = 3 };

struct Layer {
  mbd_layer spec;
  int64_t d_in = 0, d_out = 0, nW = 0;
  void* W = nullptr;
  float* bias = nullptr;
  float* dW = nullptr;
  float* W32 = nullptr;  // fp32 master weights (optional)
  float* V = nullptr;    // momentum: velocity of W (optional), fp32
  float* Vb = nullptr;   // momentum: velocity of the bias
  float* db = nullptr;
  void* act = nullptr;   // stored forward output [B, d_out]; float logits for the last FC layer
  void* dY = nullptr;    // [B, d_out] activation dtype
  TcGemm fwd, bwd_data, bwd_weight;
};

}  // namespace

struct mbd_net {
  int L = 0;                        // fully connected layers (n->layers); public layer index = Lc + index here
  int Lc = 0;                       // convolution layers below them (n->conv)
  bool mixed = false;               // convolutions first, fully connected layers after them (Section 2.4)
  void* X_fc = nullptr;             // [B, C*H*W]: output of the last convolution in NCHW order = input of the first FC layer
  void* dX_fc = nullptr;            // gradient w.r.t. X_fc after the mask of the last convolution's ReLU
  int64_t B = 0;
  int P_r = 1, P_c = 1, dtype = MBD_BF16, loss = 0, max_partials = 4;
  cudaStream_t stream = nullptr;
  int num_sms = 148;
  int device = 0;
  bool is_conv = false;
  bool master = false;              // fp32 master weights: the update leaves the contraction's epilogue
  bool momentum = false;            // heavy-ball momentum: the update is a kernel of its own after the gradient
  float mu = 0.f;
  std::vector<Layer> layers;
  float* partials = nullptr;
  size_t partial_elems = 0;
  float* colsum_scratch = nullptr;
  float* colsum_scratch_aux = nullptr;   // the side stream's own: sums on the two streams are not ordered
  // The bias gradients (column sums of dY_i) are small and independent of the contractions of
  // their layer: they run on a side stream, forked after dY_i exists and joined at the end of
  // the backward pass, next to the persistent GEMM CTAs (the column-sum kernels use no shared
  // memory and few registers, and the GEMM leaves room for them in every SM sub-partition).
  // The partial-sum reductions stay on the main stream: beside a product they reach about
  // 1 TB/s and slow that product by a third, which costs more than it hides (measured).
  cudaStream_t aux = nullptr;
  std::vector<cudaEvent_t> ev_fork;
  cudaEvent_t ev_join = nullptr;
  // Small networks (every backward-weight product under 0.2 TFLOP): the backward-weight products,
  // which nothing inside the step waits for, run on a stream of their own beside the chain of
  // backward-data products; their kernels leave SMs idle that the other stream's CTAs fill.
  // dW_i starts once the backward-data product of layer i (the last reader of the old W_i) is done.
  cudaStream_t wstream = nullptr;
  bool overlap_dw = false;
  std::vector<cudaEvent_t> ev_dx;           // per layer: dY_i final and W_i no longer read
  cudaEvent_t ev_wjoin = nullptr;
  float* partials_dw = nullptr;             // partials of the backward-weight products when they run beside the others
  // Running sums (a product's pieces added in its own epilogue instead of a reduction launch) hand over
  // through one word per (tile, epilogue warp); products that can run at the same time have words of their own.
  int* fix_flags = nullptr;
  int* fix_flags_dw = nullptr;
  size_t fix_words = 0, fix_words_dw = 0;
  size_t last_dw_elems = 0;
  bool last_red_dw = false;                 // the last reduction executed used partials_dw
  cudaEvent_t ev_loss = nullptr;            // forward done -> the sum of the per-sample losses may start
  bool defer_loss = false;                  // set by mbd_train_step: J is only needed when the step is over
  bool loss_pending = false;                // the loss sum runs on the side stream, not joined yet
  float* per_sample = nullptr;
  float* loss_dev = nullptr;
  int* status = nullptr;
  const void* X = nullptr;
  const void* X_mapped = nullptr;   // input pointer the layer-1 tensor maps were built for
  const int32_t* labels = nullptr;
  int state = ST_IDLE;
  Profiler prof;
  void* X_stage = nullptr;
  int32_t* labels_stage = nullptr;
  // pipelined host steps: two landing slots for the batch, filled on a copy stream
  cudaStream_t h2d = nullptr;
  void* X_in[2] = {nullptr, nullptr};
  int32_t* labels_in[2] = {nullptr, nullptr};
  float* loss_pinned = nullptr;             // two floats of pinned host memory
  cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_slot_free[2] = {nullptr, nullptr}, ev_step_done[2] = {nullptr, nullptr};
  bool slot_used[2] = {false, false};
  int pipe_head = 0, pipe_count = 0;
  ConvNet* conv = nullptr;
  // cached CUDA graph of one fused step and the arguments it was captured for
  cudaGraphExec_t graph_exec = nullptr;
  const void* g_X = nullptr;
  const int32_t* g_labels = nullptr;
  float* g_loss = nullptr;
  float g_eta = 0.f;
  int64_t graph_launches = 0;
  size_t elt() const { return dtype == MBD_BF16 ? 2 : 4; }
};

namespace {

#define CK(expr)                          \
  do {                                    \
    cudaError_t e_ = (expr);              \
    if (e_ != cudaSuccess) {              \
      (void)cudaGetLastError();           \
      return MBD_E_CUDA;                  \
    }                                     \
  } while (0)

mbd_status dev_alloc(void** p, size_t bytes) {
  if (bytes == 0) bytes = 16;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    *p = nullptr;
    return MBD_E_ALLOC;
  }
  return MBD_OK;
}

int splits_for(int P, int max_partials) { return P < max_partials ? P : max_partials; }

Epi epi_act(void* out, int64_t ldo, int out_bf16, const float* bias, int relu) {
  Epi e{};
  e.op = EPI_ACT; e.out_bf16 = out_bf16; e.relu = relu; e.out = out; e.ldo = ldo; e.bias = bias;
  return e;
}
Epi epi_mask(void* out, int64_t ldo, int out_bf16, const void* mask, int64_t ldmask) {
  Epi e{};
  e.op = EPI_MASK; e.out_bf16 = out_bf16; e.out = out; e.ldo = ldo; e.mask = mask; e.ldmask = ldmask;
  return e;
}
Epi epi_sgd(void* w, int64_t ldo, int out_bf16, float scale, float* master = nullptr) {
  Epi e{};
  e.op = EPI_SGD; e.out_bf16 = out_bf16; e.out = w; e.ldo = ldo; e.scale = scale; e.master = master;
  return e;
}

// One contraction on the path that matches the network dtype, followed by the reduction
// of its partials when the K range was split.
// `stream` / `parts`: null selects the network's stream and the common partial-sum workspace.
mbd_status run_gemm(mbd_net* n, TcGemm& tc, int variant, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                    const void* Bm, int64_t ldb, int S, const Epi& epi, cudaStream_t stream = nullptr, float* parts = nullptr) {
  const double flops = 2.0 * static_cast<double>(M) * static_cast<double>(N) * static_cast<double>(K);
  if (!stream) stream = n->stream;
  const bool own_parts = parts != nullptr;
  if (!parts) parts = n->partials;
  if (n->dtype == MBD_BF16) {
    tc.epi = epi;
    tc.partials = parts;
    tc.flags = own_parts ? n->fix_flags_dw : n->fix_flags;
    n->prof.begin(MBD_K_GEMM_FWD + variant, flops, stream);
    CK(tc_gemm_launch(tc, stream));
    n->prof.end();
    S = tc.fix ? 1 : tc.k_splits;          // a running sum leaves nothing to reduce
  } else {
    SimtGemm g{};
    g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
    g.A = static_cast<const float*>(A);
    g.B = static_cast<const float*>(Bm);
    if (variant == 0) { g.a_sm = lda; g.a_sk = 1; g.b_sn = ldb; g.b_sk = 1; }
    else if (variant == 1) { g.a_sm = lda; g.a_sk = 1; g.b_sn = 1; g.b_sk = ldb; }
    else { g.a_sm = 1; g.a_sk = lda; g.b_sn = 1; g.b_sk = ldb; }
    if (S > K) S = static_cast<int>(K);
    g.k_splits = S;
    g.partials = parts;
    g.epi = epi;
    n->prof.begin(MBD_K_GEMM_FWD + variant, flops, stream);
    CK(simt_gemm_launch(g, stream));
    n->prof.end();
  }
  if (S > 1) {
    // (S + 1) planes of M N floats cross HBM, plus what the tail operation touches
    const double esz = epi.out_bf16 ? 2.0 : 4.0;
    double bytes = static_cast<double>(M) * N * (4.0 * S + esz);
    if (epi.op == EPI_SGD || (epi.op == EPI_MASK && epi.mask)) bytes += static_cast<double>(M) * N * esz;
    n->prof.begin(MBD_K_REDUCE, bytes, stream);
    CK(reduce_partials_launch(parts, S, M, N, epi, n->num_sms, stream));
    n->prof.end();
    n->last_red_dw = own_parts;
  }
  return MBD_OK;
}

mbd_status prepare_tc(mbd_net* n, TcGemm& g, int variant, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                      const void* Bm, int64_t ldb, int S, const Epi* te_epi) {
  g = TcGemm{};
  g.variant = variant;
  g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
  g.k_splits = S;
  g.allow_extra_split = variant != 2;     // forward and backward-data: small outputs, cheap partials
  // max_partials >= P asks for every process's partial as a plane of its own (Appendix A.2 as the paper's
  // processes hold it); otherwise the pieces are intermediate and may be folded into a running sum
  const int P = variant == 1 ? n->P_r : variant == 2 ? n->P_c : 1;
  const bool no_fix = getenv("MBD_NO_FIXUP") != nullptr;             // tuning knob: always S planes + reduction launch
  g.allow_fix = !no_fix && (P == 1 || S < P);
  g.status = n->status;
  CK(tc_gemm_prepare(g, A, lda, Bm, ldb, n->num_sms, te_epi));
  return MBD_OK;
}

const void* layer_input(const mbd_net* n, int i) { return i == 0 ? n->X : n->layers[i - 1].act; }

// The epilogues of the three products of layer i (the scale of the update is set at launch).
Epi fwd_epi(mbd_net* n, int i) {
  Layer& l = n->layers[i];
  const bool last = i == n->L - 1;
  return epi_act(l.act, l.d_out, last ? 0 : (n->dtype == MBD_BF16), l.bias, (!last && l.spec.relu) ? 1 : 0);
}
Epi bwd_data_epi(mbd_net* n, int i) {
  Layer& l = n->layers[i];
  if (i == 0)     // below the first fully connected layer sits the last convolution
    return epi_mask(n->dX_fc, l.d_in, 1, conv_last_relu(n->conv) ? n->X_fc : nullptr, l.d_in);
  Layer& prev = n->layers[i - 1];
  return epi_mask(prev.dY, l.d_in, n->dtype == MBD_BF16, prev.spec.relu ? prev.act : nullptr, l.d_in);
}

// (Re)build the tensor maps that reference the caller's input buffer.
mbd_status map_input(mbd_net* n) {
  if (n->dtype != MBD_BF16 || n->is_conv || n->X_mapped == n->X) return MBD_OK;
  Layer& l = n->layers[0];
  const int S_c = splits_for(n->P_c, n->max_partials);
  const Epi ef = fwd_epi(n, 0), ew = epi_sgd(l.W, l.d_in, 1, 0.f);
  mbd_status s = prepare_tc(n, l.fwd, 0, n->B, l.d_out, l.d_in, n->X, l.d_in, l.W, l.d_in, 1, &ef);
  if (s != MBD_OK) return s;
  s = prepare_tc(n, l.bwd_weight, 2, l.d_out, l.d_in, n->B, l.dY, l.d_out, n->X, l.d_in, S_c, &ew);
  if (s != MBD_OK) return s;
  n->X_mapped = n->X;
  return MBD_OK;
}

void free_net(mbd_net* n) {
  if (!n) return;
  for (Layer& l : n->layers) {
    cudaFree(l.W); cudaFree(l.bias); cudaFree(l.dW); cudaFree(l.db); cudaFree(l.act); cudaFree(l.dY); cudaFree(l.W32); cudaFree(l.V); cudaFree(l.Vb);
  }
  cudaFree(n->partials); cudaFree(n->colsum_scratch); cudaFree(n->colsum_scratch_aux); cudaFree(n->per_sample); cudaFree(n->loss_dev);
  cudaFree(n->status); cudaFree(n->X_stage); cudaFree(n->labels_stage); cudaFree(n->X_fc); cudaFree(n->dX_fc);
  for (int k = 0; k < 2; ++k) {
    cudaFree(n->X_in[k]); cudaFree(n->labels_in[k]);
    if (n->ev_copied[k]) cudaEventDestroy(n->ev_copied[k]);
    if (n->ev_slot_free[k]) cudaEventDestroy(n->ev_slot_free[k]);
    if (n->ev_step_done[k]) cudaEventDestroy(n->ev_step_done[k]);
  }
  if (n->loss_pinned) cudaFreeHost(n->loss_pinned);
  if (n->h2d) cudaStreamDestroy(n->h2d);
  if (n->conv) conv_destroy(n->conv);
  if (n->graph_exec) cudaGraphExecDestroy(n->graph_exec);
  for (cudaEvent_t e : n->ev_fork) if (e) cudaEventDestroy(e);
  if (n->ev_join) cudaEventDestroy(n->ev_join);
  if (n->ev_loss) cudaEventDestroy(n->ev_loss);
  for (cudaEvent_t e : n->ev_dx) if (e) cudaEventDestroy(e);
  if (n->ev_wjoin) cudaEventDestroy(n->ev_wjoin);
  if (n->wstream) cudaStreamDestroy(n->wstream);
  cudaFree(n->partials_dw); cudaFree(n->fix_flags); cudaFree(n->fix_flags_dw);
  if (n->aux) cudaStreamDestroy(n->aux);
  n->prof.destroy();
  (void)cudaGetLastError();
  delete n;
}

}  // namespace

extern "C" mbd_status mbd_net_create(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, int dtype, int loss,
                                     int max_partials, void* cuda_stream, mbd_net** out) {
  if (!layers || !out || L < 1 || B < 1) return MBD_E_INVALID;
  if (dtype != MBD_F32 && dtype != MBD_BF16) return MBD_E_INVALID;
  if (loss != MBD_LOSS_SOFTMAX_CE && loss != MBD_LOSS_HALF_SSQ && loss != MBD_LOSS_NONE) return MBD_E_INVALID;
  if (max_partials < 0) return MBD_E_INVALID;
  *out = nullptr;
  if (P_r < 1 || P_c < 1 || P_c > B) return MBD_E_GRID;
  int Lc = 0;                                 // convolutions come first (L_D), fully connected layers after them (L_M)
  while (Lc < L && layers[Lc].kind == MBD_CONV3X3) ++Lc;
  const bool is_conv = Lc == L, mixed = Lc > 0 && Lc < L;
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    if (l.kind == MBD_CONV3X3 && i >= Lc) return MBD_E_UNSUPPORTED;      // a convolution above a fully connected layer
    if (l.kind == MBD_FC) {
      if (l.d_in < 1 || l.d_out < 1) return MBD_E_INVALID;
      if (l.split != MBD_SPLIT_MODEL) return MBD_E_INVALID;
      if (i > Lc && l.d_in != layers[i - 1].d_out) return MBD_E_INVALID;
      if (i == Lc && mixed) {
        const mbd_layer& lc = layers[Lc - 1];
        const int st = lc.stride > 1 ? lc.stride : 1;
        if (l.d_in != static_cast<int64_t>(lc.C_out) * (lc.H / st) * (lc.W / st)) return MBD_E_INVALID;
      }
      if (P_r > l.d_out) return MBD_E_GRID;
      if (dtype == MBD_BF16 && (l.d_in % 8 || l.d_out % 8)) return MBD_E_UNSUPPORTED;
      if (l.d_in > INT32_MAX || l.d_out > INT32_MAX || B > INT32_MAX) return MBD_E_UNSUPPORTED;
    } else if (l.kind == MBD_CONV3X3) {
      // "same" padding; odd kernel sizes up to 11, channel counts that are multiples of 8
      if (l.kh < 1 || l.kw < 1 || l.kh > 11 || l.kw > 11 || l.kh % 2 == 0 || l.kw % 2 == 0 || dtype != MBD_BF16) return MBD_E_UNSUPPORTED;
      if (l.C_in < 8 || l.C_out < 8 || l.C_in % 8 || l.C_out % 8) return MBD_E_UNSUPPORTED;
      if (i > 0 && l.C_in != layers[i - 1].C_out) return MBD_E_INVALID;
      if (l.split != MBD_SPLIT_DOMAIN && l.split != MBD_SPLIT_BATCH && l.split != MBD_SPLIT_MODEL) return MBD_E_INVALID;
      if (l.split == MBD_SPLIT_BATCH) {                                  // 1 x P: one sample per process at least
        if (l.H < 1 || l.W < 1 || static_cast<int64_t>(P_r) * P_c > B) return MBD_E_GRID;
      } else if (l.split == MBD_SPLIT_MODEL) {
        // L_M (Eq. 8): the P_r groups split the output channels.  A group's block must be whole 64-channel k-blocks of
        // the backward-data product, whose K range is cut over these blocks; stride 1 only
        if (l.H < 1 || l.W < 1) return MBD_E_GRID;
        if (P_r > l.C_out) return MBD_E_GRID;
        if (l.stride > 1 || (P_r > 1 && l.C_out % (64 * P_r) != 0)) return MBD_E_UNSUPPORTED;
      } else if (l.H < 1 || l.W < 1 || P_r > l.H || (P_r > 1 && l.H / P_r < l.kh / 2)) {
        return MBD_E_GRID;   // a strip needs >= 1 row, and its halo rows come from the adjacent strip only
      }
      const int st = l.stride > 1 ? l.stride : 1;
      if (st > 4 || l.H % st || l.W % st) return l.stride > 4 ? MBD_E_UNSUPPORTED : MBD_E_INVALID;
      if (i > 0) {                                                       // the image sizes chain through the strides
        const int ps = layers[i - 1].stride > 1 ? layers[i - 1].stride : 1;
        if (l.H != layers[i - 1].H / ps || l.W != layers[i - 1].W / ps) return MBD_E_INVALID;
      }
      if (l.split == MBD_SPLIT_DOMAIN && P_r > l.H / st) return MBD_E_GRID;
    } else {
      return MBD_E_INVALID;
    }
  }
  if (is_conv && loss != MBD_LOSS_HALF_SSQ && loss != MBD_LOSS_NONE) return MBD_E_UNSUPPORTED;
  if (!is_conv && loss != MBD_LOSS_SOFTMAX_CE) return MBD_E_UNSUPPORTED;
  if (mixed && dtype != MBD_BF16) return MBD_E_UNSUPPORTED;

  mbd_net* n = new (std::nothrow) mbd_net();
  if (!n) return MBD_E_ALLOC;
  n->L = L - Lc; n->Lc = Lc; n->mixed = mixed;
  n->B = B; n->P_r = P_r; n->P_c = P_c; n->dtype = dtype; n->loss = loss;
  n->max_partials = max_partials == 0 ? 4 : max_partials;
  n->stream = static_cast<cudaStream_t>(cuda_stream);
  n->prof.stream = n->stream;
  n->is_conv = is_conv;
  mbd_status st = MBD_OK;
  cudaDeviceProp prop;
  if (cudaGetDevice(&n->device) != cudaSuccess || cudaGetDeviceProperties(&prop, n->device) != cudaSuccess) {
    (void)cudaGetLastError();
    delete n;
    return MBD_E_CUDA;
  }
  n->num_sms = prop.multiProcessorCount;
  if (dtype == MBD_BF16 && prop.major != 10) {   // tcgen05 kernels need compute capability 10.x
    delete n;
    return MBD_E_UNSUPPORTED;
  }

#define ALLOC(ptr, bytes)                                                   \
  do {                                                                      \
    st = dev_alloc(reinterpret_cast<void**>(&(ptr)), (bytes));              \
    if (st != MBD_OK) { free_net(n); return st; }                           \
  } while (0)

  ALLOC(n->status, sizeof(int));
  ALLOC(n->loss_dev, sizeof(float));
  if (cudaMemsetAsync(n->status, 0, sizeof(int), n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }

  if (Lc > 0) {
    // how each convolution uses the grid follows from its split kind (strips, batch blocks on 1 x P, groups over the
    // output channels): conv_create works that out, layer by layer
    st = conv_create(layers, Lc, B, P_r, P_c, n->max_partials, n->num_sms, n->status, n->stream, &n->prof, mixed || loss == MBD_LOSS_NONE, &n->conv);
    if (st != MBD_OK) { free_net(n); return st; }
    if (is_conv) {
      *out = n;
      return MBD_OK;
    }
  }
  layers += Lc;                      // from here on: the fully connected layers
  L -= Lc;

  const size_t es = n->elt();
  const int S_r = splits_for(P_r, n->max_partials), S_c = splits_for(P_c, n->max_partials);
  n->layers.resize(L);
  size_t part_elems = 0, max_d = 0;
  for (int i = 0; i < L; ++i) {
    Layer& l = n->layers[i];
    l.spec = layers[i];
    l.d_in = layers[i].d_in; l.d_out = layers[i].d_out; l.nW = l.d_in * l.d_out;
    ALLOC(l.W, l.nW * es);
    ALLOC(l.dW, l.nW * sizeof(float));
    if (l.spec.bias) {
      ALLOC(l.bias, l.d_out * sizeof(float));
      ALLOC(l.db, l.d_out * sizeof(float));
      if (cudaMemsetAsync(l.bias, 0, l.d_out * sizeof(float), n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }
    }
    const bool last = i == L - 1;
    ALLOC(l.act, static_cast<size_t>(B) * l.d_out * (last ? sizeof(float) : es));
    ALLOC(l.dY, static_cast<size_t>(B) * l.d_out * es);
    if (cudaMemsetAsync(l.W, 0, l.nW * es, n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }
    if (dtype != MBD_BF16) {
      if (S_c > 1) part_elems = std::max(part_elems, static_cast<size_t>(S_c) * l.nW);
      if (i > 0 && S_r > 1) part_elems = std::max(part_elems, static_cast<size_t>(S_r) * B * l.d_in);
    }
    max_d = std::max(max_d, static_cast<size_t>(l.d_out));
  }
  if (mixed) {
    ALLOC(n->X_fc, static_cast<size_t>(B) * n->layers[0].d_in * es);
    ALLOC(n->dX_fc, static_cast<size_t>(B) * n->layers[0].d_in * es);
    n->X = n->X_fc;
    n->X_mapped = n->X_fc;           // the plans below are built on the real input buffer
  }
  if (dtype == MBD_BF16) {
    // Plan every contraction now (tile width, number of K pieces); the partial-sum workspace is
    // sized from the plans.  The first layer's maps are rebuilt once the caller's X is known.
    for (int i = 0; i < L; ++i) {
      Layer& l = n->layers[i];
      const void* x_in = i > 0 ? n->layers[i - 1].act : (mixed ? n->X_fc : l.W);   // placeholder address for layer 1
      const Epi ef = fwd_epi(n, i), ew = epi_sgd(l.W, l.d_in, 1, 0.f);
      st = prepare_tc(n, l.fwd, 0, B, l.d_out, l.d_in, x_in, l.d_in, l.W, l.d_in, 1, &ef);
      if (st == MBD_OK && (i > 0 || mixed)) {
        const Epi ed = bwd_data_epi(n, i);
        st = prepare_tc(n, l.bwd_data, 1, B, l.d_in, l.d_out, l.dY, l.d_out, l.W, l.d_in, S_r, &ed);
      }
      if (st == MBD_OK) st = prepare_tc(n, l.bwd_weight, 2, l.d_out, l.d_in, B, l.dY, l.d_out, x_in, l.d_in, S_c, &ew);
      if (st != MBD_OK) { free_net(n); return st; }
      auto planes = [](const TcGemm& g) { return static_cast<size_t>(g.fix ? 1 : g.k_splits); };
      if (l.fwd.k_splits > 1) part_elems = std::max(part_elems, planes(l.fwd) * B * l.d_out);
      if ((i > 0 || mixed) && l.bwd_data.k_splits > 1) part_elems = std::max(part_elems, planes(l.bwd_data) * B * l.d_in);
      if (l.bwd_weight.k_splits > 1) part_elems = std::max(part_elems, planes(l.bwd_weight) * l.nW);
      n->fix_words = std::max(n->fix_words, static_cast<size_t>(std::max(l.fwd.flag_words, l.bwd_weight.flag_words)));
      if (i > 0 || mixed) n->fix_words = std::max(n->fix_words, static_cast<size_t>(l.bwd_data.flag_words));
    }
  }
  n->partial_elems = part_elems;
  if (part_elems) ALLOC(n->partials, part_elems * sizeof(float));
  {
    // backward-weight products beside the backward-data chain: only where every one of them is small
    // (a product that fills the GPU for a long time gains nothing from a neighbour), bf16 path only
    bool small = dtype == MBD_BF16 && L > 1 && !getenv("MBD_NO_DW_OVERLAP");
    size_t dw_elems = 0;
    for (int i = 0; i < L && small; ++i) {
      const Layer& l = n->layers[i];
      if (2.0 * static_cast<double>(l.nW) * static_cast<double>(B) > 2e11) small = false;
      if (l.bwd_weight.k_splits > 1) dw_elems = std::max(dw_elems, static_cast<size_t>(l.bwd_weight.fix ? 1 : l.bwd_weight.k_splits) * l.nW);
      n->fix_words_dw = std::max(n->fix_words_dw, static_cast<size_t>(l.bwd_weight.flag_words));
    }
    n->overlap_dw = small;
    if (small && dw_elems) ALLOC(n->partials_dw, dw_elems * sizeof(float));
    n->last_dw_elems = dw_elems;
    if (n->fix_words) {
      ALLOC(n->fix_flags, n->fix_words * sizeof(int));
      if (cudaMemsetAsync(n->fix_flags, 0, n->fix_words * sizeof(int), n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }
    }
    if (small && n->fix_words_dw) {
      ALLOC(n->fix_flags_dw, n->fix_words_dw * sizeof(int));
      if (cudaMemsetAsync(n->fix_flags_dw, 0, n->fix_words_dw * sizeof(int), n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }
    }
  }
  ALLOC(n->colsum_scratch, static_cast<size_t>(8 * 32) * max_d * sizeof(float));
  ALLOC(n->colsum_scratch_aux, static_cast<size_t>(8 * 32) * max_d * sizeof(float));
  ALLOC(n->per_sample, B * sizeof(float));
#undef ALLOC
  {
    bool ok = cudaStreamCreateWithFlags(&n->aux, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&n->ev_join, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&n->ev_loss, cudaEventDisableTiming) == cudaSuccess;
    n->ev_fork.assign(L, nullptr);
    for (int i = 0; i < L && ok; ++i) ok = cudaEventCreateWithFlags(&n->ev_fork[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok && n->overlap_dw) {
      ok = cudaStreamCreateWithFlags(&n->wstream, cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&n->ev_wjoin, cudaEventDisableTiming) == cudaSuccess;
      n->ev_dx.assign(L, nullptr);
      for (int i = 0; i < L && ok; ++i) ok = cudaEventCreateWithFlags(&n->ev_dx[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) { free_net(n); return MBD_E_CUDA; }
  }
  if (cudaStreamSynchronize(n->stream) != cudaSuccess) { free_net(n); return MBD_E_CUDA; }
  *out = n;
  return MBD_OK;
}

extern "C" mbd_status mbd_net_destroy(mbd_net* n) {
  if (!n) return MBD_E_INVALID;
  cudaStreamSynchronize(n->stream);
  free_net(n);
  return MBD_OK;
}

extern "C" mbd_status mbd_set_weights(mbd_net* n, int layer, const void* W_dev, const float* bias_dev) {
  if (!n || !W_dev || layer < 0 || layer >= n->Lc + n->L) return MBD_E_INVALID;
  if (layer < n->Lc) return bias_dev ? MBD_E_INVALID : conv_set_weights(n->conv, layer, W_dev);
  Layer& l = n->layers[layer - n->Lc];
  CK(cudaMemcpyAsync(l.W, W_dev, l.nW * n->elt(), cudaMemcpyDeviceToDevice, n->stream));
  if (l.W32) CK(widen_bf16_launch(l.W, l.W32, l.nW, n->num_sms, n->stream));
  if (bias_dev) {
    if (!l.bias) return MBD_E_INVALID;
    CK(cudaMemcpyAsync(l.bias, bias_dev, l.d_out * sizeof(float), cudaMemcpyDeviceToDevice, n->stream));
  }
  return MBD_OK;
}

extern "C" mbd_status mbd_enable_master_weights(mbd_net* n) {
  if (!n) return MBD_E_INVALID;
  if (n->dtype != MBD_BF16) return MBD_E_UNSUPPORTED;
  if (n->master) return MBD_OK;
  if (n->conv) {
    const mbd_status s = conv_enable_master(n->conv);
    if (s != MBD_OK) return s;
  }
  for (Layer& l : n->layers) {
    const mbd_status s = dev_alloc(reinterpret_cast<void**>(&l.W32), l.nW * sizeof(float));
    if (s != MBD_OK) return s;
    CK(widen_bf16_launch(l.W, l.W32, l.nW, n->num_sms, n->stream));
  }
  n->master = true;
  if (n->graph_exec) { cudaGraphExecDestroy(n->graph_exec); n->graph_exec = nullptr; }   // the step's launches change
  return MBD_OK;
}

extern "C" mbd_status mbd_enable_momentum(mbd_net* n, float mu) {
  if (!n || !(mu >= 0.f && mu < 1.f)) return MBD_E_INVALID;
  if (n->conv) {
    const mbd_status s = conv_enable_momentum(n->conv, mu);
    if (s != MBD_OK) return s;
  }
  for (Layer& l : n->layers) {
    if (!l.V) {
      mbd_status s = dev_alloc(reinterpret_cast<void**>(&l.V), l.nW * sizeof(float));
      if (s == MBD_OK && l.bias) s = dev_alloc(reinterpret_cast<void**>(&l.Vb), l.d_out * sizeof(float));
      if (s != MBD_OK) return s;
    }
    CK(cudaMemsetAsync(l.V, 0, l.nW * sizeof(float), n->stream));
    if (l.Vb) CK(cudaMemsetAsync(l.Vb, 0, l.d_out * sizeof(float), n->stream));
  }
  n->momentum = true;
  n->mu = mu;
  if (n->graph_exec) { cudaGraphExecDestroy(n->graph_exec); n->graph_exec = nullptr; }   // the step's launches change
  return MBD_OK;
}

extern "C" mbd_status mbd_get_weights(mbd_net* n, int layer, void* W_dev, float* bias_dev) {
  if (!n || !W_dev || layer < 0 || layer >= n->Lc + n->L) return MBD_E_INVALID;
  if (layer < n->Lc) return bias_dev ? MBD_E_INVALID : conv_get_weights(n->conv, layer, W_dev);
  Layer& l = n->layers[layer - n->Lc];
  CK(cudaMemcpyAsync(W_dev, l.W, l.nW * n->elt(), cudaMemcpyDeviceToDevice, n->stream));
  if (bias_dev) {
    if (!l.bias) return MBD_E_INVALID;
    CK(cudaMemcpyAsync(bias_dev, l.bias, l.d_out * sizeof(float), cudaMemcpyDeviceToDevice, n->stream));
  }
  return MBD_OK;
}

extern "C" mbd_status mbd_forward(mbd_net* n, const void* X_dev, const int32_t* labels_dev, float* loss_sum_dev) {
  if (!n || !X_dev) return MBD_E_INVALID;
  if (n->is_conv) {
    mbd_status s = conv_forward(n->conv, X_dev, loss_sum_dev);
    if (s == MBD_OK) n->state = ST_FWD;
    return s;
  }
  if (!labels_dev) return MBD_E_INVALID;
  mbd_status s;
  if (n->mixed) {
    // domain-parallel layers, then the activation leaves the strips as the [B, C*H*W] input of the model-parallel ones
    if ((s = conv_forward(n->conv, X_dev, nullptr)) != MBD_OK) return s;
    if ((s = conv_output_to_nchw(n->conv, n->X_fc)) != MBD_OK) return s;
  } else {
    n->X = X_dev;
  }
  n->labels = labels_dev;
  s = map_input(n);
  if (s != MBD_OK) return s;
  const int bf = n->dtype == MBD_BF16;
  for (int i = 0; i < n->L; ++i) {
    Layer& l = n->layers[i];
    const Epi e = fwd_epi(n, i);
    s = run_gemm(n, l.fwd, 0, n->B, l.d_out, l.d_in, layer_input(n, i), l.d_in, l.W, l.d_in, 1, e);
    if (s != MBD_OK) return s;
  }
  Layer& top = n->layers[n->L - 1];
  n->prof.begin(MBD_K_SOFTMAX, static_cast<double>(n->B) * top.d_out * (4.0 + (bf ? 2.0 : 4.0)));
  CK(softmax_xent_launch(static_cast<const float*>(top.act), n->B, top.d_out, labels_dev, top.dY, bf, n->per_sample, n->stream));
  n->prof.end();
  if (loss_sum_dev) {
    // inside a whole step nothing waits for J: its (single-CTA) sum goes to the side stream
    cudaStream_t ls = n->stream;
    if (n->defer_loss && n->aux) {
      CK(cudaEventRecord(n->ev_loss, n->stream));
      CK(cudaStreamWaitEvent(n->aux, n->ev_loss, 0));
      ls = n->aux;
      n->loss_pending = true;
    }
    n->prof.begin(MBD_K_OTHER, static_cast<double>(n->B) * 4.0, ls);
    CK(sum_f32_launch(n->per_sample, n->B, 1.f, loss_sum_dev, ls));
    n->prof.end();
  }
  n->state = ST_FWD;
  return MBD_OK;
}

extern "C" mbd_status mbd_backward(mbd_net* n, float fused_eta) {
  if (!n || fused_eta < 0.f) return MBD_E_INVALID;
  if (n->state != ST_FWD) return MBD_E_STATE;
  if (n->is_conv) {
    mbd_status s = conv_backward(n->conv, fused_eta);
    if (s == MBD_OK) n->state = fused_eta > 0.f ? ST_BWD_FUSED : ST_BWD_UNFUSED;
    return s;
  }
  const int bf = n->dtype == MBD_BF16;
  const bool fused = fused_eta > 0.f;
  const float scale = -fused_eta / static_cast<float>(n->B);
  const int S_r = splits_for(n->P_r, n->max_partials), S_c = splits_for(n->P_c, n->max_partials);
  static const bool no_side = getenv("MBD_NO_SIDE") != nullptr;      // tuning knob: column sums on the main stream
  const bool side = n->aux != nullptr && !no_side;
  bool forked = false, dw_forked = false;
  for (int i = n->L - 1; i >= 0; --i) {
    Layer& l = n->layers[i];
    if (l.bias) {
      cudaStream_t cs = n->stream;
      // Small sums are launch-bound and hide entirely beside the products; a large one (cfg5: 134 MB)
      // slows the product it runs beside by more than its own 0.04 ms, so it stays in line.
      const bool small = static_cast<double>(n->B) * l.d_out * (bf ? 2.0 : 4.0) <= 32.0 * 1024 * 1024;
      if (side && small) {
        CK(cudaEventRecord(n->ev_fork[i], n->stream));
        CK(cudaStreamWaitEvent(n->aux, n->ev_fork[i], 0));
        cs = n->aux;
        forked = true;
      }
      n->prof.begin(MBD_K_COLSUM, static_cast<double>(n->B) * l.d_out * (bf ? 2.0 : 4.0), cs);
      const bool fused_b = fused && !n->momentum;          // momentum: db first, then the update kernel
      CK(colsum_launch(l.dY, bf, n->B, l.d_out, cs == n->aux ? n->colsum_scratch_aux : n->colsum_scratch, colsum_row_splits(n->B, l.d_out, n->num_sms), fused_b ? nullptr : l.db,
                       fused_b ? l.bias : nullptr, scale, cs));
      n->prof.end();
      n->prof.total_launches += colsum_launches(n->B, l.d_out, n->num_sms) - 1;
      if (fused && n->momentum) {
        n->prof.begin(MBD_K_SGD, static_cast<double>(l.d_out) * 20.0, cs);
        CK(sgd_momentum_update_launch(l.bias, 0, nullptr, l.Vb, l.db, l.d_out, n->mu, 1.f / static_cast<float>(n->B), fused_eta, n->num_sms, cs));
        n->prof.end();
      }
    }
    if (i > 0 || n->mixed) {   // nothing is propagated below the first layer of the network
      const Epi e = bwd_data_epi(n, i);
      mbd_status s = run_gemm(n, l.bwd_data, 1, n->B, l.d_in, l.d_out, l.dY, l.d_out, l.W, l.d_in, S_r, e);
      if (s != MBD_OK) return s;
    }
    // With master weights: a split product updates the fp32 master in the tail of its reduction (which streams
    // the sum through registers anyway); an unsplit one materialises the gradient and a streaming kernel applies
    // Eq. 1 to the master (measured equal to doing it in the product's epilogue, whose loads would be exposed).
    const bool master_tail = fused && n->master && !n->momentum && bf && l.bwd_weight.k_splits > 1;
    const bool master_kernel = fused && (n->master || n->momentum) && !master_tail;     // momentum: always a kernel of its own
    const Epi e = (fused && !master_kernel) ? epi_sgd(l.W, l.d_in, bf, scale, master_tail ? l.W32 : nullptr)
                                            : epi_act(l.dW, l.d_in, 0, nullptr, 0);
    cudaStream_t ws = nullptr;
    if (n->overlap_dw) {
      // dY_i is final and the last reader of the old W_i has been enqueued: dW_i may start beside
      // the backward-data products of the layers below
      CK(cudaEventRecord(n->ev_dx[i], n->stream));
      CK(cudaStreamWaitEvent(n->wstream, n->ev_dx[i], 0));
      ws = n->wstream;
      dw_forked = true;
    }
    mbd_status s = run_gemm(n, l.bwd_weight, 2, l.d_out, l.d_in, n->B, l.dY, l.d_out, layer_input(n, i), l.d_in, S_c, e, ws,
                            ws ? n->partials_dw : nullptr);
    if (s != MBD_OK) return s;
    if (master_kernel) {
      cudaStream_t us = ws ? ws : n->stream;
      n->prof.begin(MBD_K_SGD, static_cast<double>(l.nW) * (n->momentum ? 12.0 + 2.0 * n->elt() + (l.W32 ? 8.0 : 0.0) : 14.0), us);
      if (n->momentum)
        CK(sgd_momentum_update_launch(l.W, bf, l.W32, l.V, l.dW, l.nW, n->mu, 1.f / static_cast<float>(n->B), fused_eta, n->num_sms, us));
      else
        CK(sgd_master_update_launch(l.W32, l.W, l.dW, l.nW, scale, n->num_sms, us));
      n->prof.end();
    }
  }
  if (dw_forked) {
    CK(cudaEventRecord(n->ev_wjoin, n->wstream));
    CK(cudaStreamWaitEvent(n->stream, n->ev_wjoin, 0));
  }
  if (n->loss_pending) { forked = true; n->loss_pending = false; }
  if (forked) {
    CK(cudaEventRecord(n->ev_join, n->aux));
    CK(cudaStreamWaitEvent(n->stream, n->ev_join, 0));
  }
  if (n->mixed) {
    // the gradient of the first fully connected layer's input goes back into strips and down the convolutions
    mbd_status s = conv_top_grad_from_nchw(n->conv, n->dX_fc);
    if (s == MBD_OK) s = conv_backward(n->conv, fused_eta);
    if (s != MBD_OK) return s;
  }
  n->state = fused ? ST_BWD_FUSED : ST_BWD_UNFUSED;
  return MBD_OK;
}

extern "C" mbd_status mbd_sgd_step(mbd_net* n, float eta) {
  if (!n || eta < 0.f) return MBD_E_INVALID;
  if (n->state != ST_BWD_UNFUSED) return MBD_E_STATE;
  if (n->is_conv) {
    mbd_status s = conv_sgd_step(n->conv, eta);
    if (s == MBD_OK) n->state = ST_IDLE;
    return s;
  }
  const float scale = -eta / static_cast<float>(n->B);
  if (n->mixed) {
    mbd_status s = conv_sgd_step(n->conv, eta);
    if (s != MBD_OK) return s;
  }
  for (int i = 0; i < n->L; ++i) {
    Layer& l = n->layers[i];
    n->prof.begin(MBD_K_SGD, static_cast<double>(l.nW) * (n->master ? 14.0 : 4.0 + 2.0 * n->elt()));
    const float inv_B = 1.f / static_cast<float>(n->B);
    if (n->momentum) CK(sgd_momentum_update_launch(l.W, n->dtype == MBD_BF16, l.W32, l.V, l.dW, l.nW, n->mu, inv_B, eta, n->num_sms, n->stream));
    else if (n->master) CK(sgd_master_update_launch(l.W32, l.W, l.dW, l.nW, scale, n->num_sms, n->stream));
    else CK(sgd_update_launch(l.W, n->dtype == MBD_BF16, l.dW, l.nW, scale, n->num_sms, n->stream));
    n->prof.end();
    if (l.bias) {
      n->prof.begin(MBD_K_SGD, static_cast<double>(l.d_out) * 12.0);
      if (n->momentum) CK(sgd_momentum_update_launch(l.bias, 0, nullptr, l.Vb, l.db, l.d_out, n->mu, inv_B, eta, n->num_sms, n->stream));
      else CK(sgd_update_launch(l.bias, 0, l.db, l.d_out, scale, n->num_sms, n->stream));
      n->prof.end();
    }
  }
  n->state = ST_IDLE;
  return MBD_OK;
}

extern "C" mbd_status mbd_train_step(mbd_net* n, const void* X_dev, const int32_t* labels_dev, float eta, float* loss_sum_dev) {
  if (!n || !X_dev || eta <= 0.f) return MBD_E_INVALID;
  // per-kernel events cannot be recorded inside a graph, and the default stream cannot be captured
  if (n->prof.on || n->stream == nullptr || n->stream == cudaStreamLegacy || n->stream == cudaStreamPerThread) {
    n->defer_loss = !n->is_conv;
    mbd_status s = mbd_forward(n, X_dev, labels_dev, loss_sum_dev);
    n->defer_loss = false;
    return s != MBD_OK ? s : mbd_backward(n, eta);
  }
  const bool same = n->graph_exec && n->g_X == X_dev && n->g_labels == labels_dev && n->g_loss == loss_sum_dev && n->g_eta == eta;
  if (!same) {
    if (n->graph_exec) { cudaGraphExecDestroy(n->graph_exec); n->graph_exec = nullptr; }
    // first use of these buffers: build the tensor maps that refer to X outside the capture
    if (!n->mixed) n->X = X_dev;
    mbd_status s = map_input(n);
    if (s != MBD_OK) return s;
    const int64_t launches_before = n->prof.total_launches;
    CK(cudaStreamBeginCapture(n->stream, cudaStreamCaptureModeThreadLocal));
    n->defer_loss = !n->is_conv;
    s = mbd_forward(n, X_dev, labels_dev, loss_sum_dev);
    n->defer_loss = false;
    if (s == MBD_OK) s = mbd_backward(n, eta);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(n->stream, &graph);
    n->graph_launches = n->prof.total_launches - launches_before;   // kernels of one step
    n->prof.total_launches = launches_before;                        // nothing has run yet
    if (s != MBD_OK || ce != cudaSuccess || !graph) {
      if (graph) cudaGraphDestroy(graph);
      (void)cudaGetLastError();
      return s != MBD_OK ? s : MBD_E_CUDA;
    }
    const cudaError_t ie = cudaGraphInstantiate(&n->graph_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) { n->graph_exec = nullptr; (void)cudaGetLastError(); return MBD_E_CUDA; }
    n->g_X = X_dev; n->g_labels = labels_dev; n->g_loss = loss_sum_dev; n->g_eta = eta;
  }
  CK(cudaGraphLaunch(n->graph_exec, n->stream));
  n->prof.total_launches += n->graph_launches;
  n->state = ST_BWD_FUSED;
  return MBD_OK;
}

extern "C" mbd_status mbd_train_step_host(mbd_net* n, const void* X_host, const int32_t* labels_host, float eta,
                                          float* loss_host) {
  if (!n || !X_host || !loss_host || eta <= 0.f) return MBD_E_INVALID;
  const size_t x_bytes = n->conv ? conv_input_bytes(n->conv) : static_cast<size_t>(n->B) * n->layers[0].d_in * n->elt();
  if (!n->X_stage) {
    mbd_status s = dev_alloc(&n->X_stage, x_bytes);
    if (s != MBD_OK) return s;
    s = dev_alloc(reinterpret_cast<void**>(&n->labels_stage), n->B * sizeof(int32_t));
    if (s != MBD_OK) return s;
  }
  CK(cudaMemcpyAsync(n->X_stage, X_host, x_bytes, cudaMemcpyHostToDevice, n->stream));
  if (!n->is_conv) {
    if (!labels_host) return MBD_E_INVALID;
    CK(cudaMemcpyAsync(n->labels_stage, labels_host, n->B * sizeof(int32_t), cudaMemcpyHostToDevice, n->stream));
  }
  mbd_status s = mbd_train_step(n, n->X_stage, n->is_conv ? nullptr : n->labels_stage, eta, n->loss_dev);
  if (s != MBD_OK) return s;
  CK(cudaMemcpyAsync(loss_host, n->loss_dev, sizeof(float), cudaMemcpyDeviceToHost, n->stream));
  CK(cudaStreamSynchronize(n->stream));
  return MBD_OK;
}

namespace {
size_t input_bytes(const mbd_net* n) {
  return n->conv ? conv_input_bytes(n->conv) : static_cast<size_t>(n->B) * n->layers[0].d_in * n->elt();
}

mbd_status pipe_setup(mbd_net* n) {
  if (n->h2d) return MBD_OK;
  const size_t x_bytes = input_bytes(n);
  mbd_status s;
  if (!n->X_stage) {
    if ((s = dev_alloc(&n->X_stage, x_bytes)) != MBD_OK) return s;
    if ((s = dev_alloc(reinterpret_cast<void**>(&n->labels_stage), n->B * sizeof(int32_t))) != MBD_OK) return s;
  }
  for (int k = 0; k < 2; ++k) {
    if ((s = dev_alloc(&n->X_in[k], x_bytes)) != MBD_OK) return s;
    if ((s = dev_alloc(reinterpret_cast<void**>(&n->labels_in[k]), n->B * sizeof(int32_t))) != MBD_OK) return s;
    CK(cudaEventCreateWithFlags(&n->ev_copied[k], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&n->ev_slot_free[k], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&n->ev_step_done[k], cudaEventDisableTiming));
  }
  CK(cudaMallocHost(reinterpret_cast<void**>(&n->loss_pinned), 2 * sizeof(float)));
  CK(cudaStreamCreateWithFlags(&n->h2d, cudaStreamNonBlocking));
  return MBD_OK;
}
}  // namespace

extern "C" mbd_status mbd_train_step_host_begin(mbd_net* n, const void* X_host, const int32_t* labels_host, float eta) {
  if (!n || !X_host || eta <= 0.f || (!n->is_conv && !labels_host)) return MBD_E_INVALID;
  if (n->pipe_count == 2) return MBD_E_STATE;
  mbd_status s = pipe_setup(n);
  if (s != MBD_OK) return s;
  const size_t x_bytes = input_bytes(n), l_bytes = n->B * sizeof(int32_t);
  const int k = (n->pipe_head + n->pipe_count) & 1;
  // copy stream: the slot must have been drained by the step that used it last
  if (n->slot_used[k]) CK(cudaStreamWaitEvent(n->h2d, n->ev_slot_free[k], 0));
  CK(cudaMemcpyAsync(n->X_in[k], X_host, x_bytes, cudaMemcpyHostToDevice, n->h2d));
  if (!n->is_conv) CK(cudaMemcpyAsync(n->labels_in[k], labels_host, l_bytes, cudaMemcpyHostToDevice, n->h2d));
  CK(cudaEventRecord(n->ev_copied[k], n->h2d));
  // compute stream: move the batch to the buffer the (graph-captured) step reads, free the slot, run
  CK(cudaStreamWaitEvent(n->stream, n->ev_copied[k], 0));
  CK(cudaMemcpyAsync(n->X_stage, n->X_in[k], x_bytes, cudaMemcpyDeviceToDevice, n->stream));
  if (!n->is_conv) CK(cudaMemcpyAsync(n->labels_stage, n->labels_in[k], l_bytes, cudaMemcpyDeviceToDevice, n->stream));
  CK(cudaEventRecord(n->ev_slot_free[k], n->stream));
  n->slot_used[k] = true;
  s = mbd_train_step(n, n->X_stage, n->is_conv ? nullptr : n->labels_stage, eta, n->loss_dev);
  if (s != MBD_OK) return s;
  CK(cudaMemcpyAsync(n->loss_pinned + k, n->loss_dev, sizeof(float), cudaMemcpyDeviceToHost, n->stream));
  CK(cudaEventRecord(n->ev_step_done[k], n->stream));
  n->pipe_count++;
  return MBD_OK;
}

extern "C" mbd_status mbd_train_step_host_end(mbd_net* n, float* loss_host) {
  if (!n || !loss_host) return MBD_E_INVALID;
  if (n->pipe_count == 0) return MBD_E_STATE;
  const int k = n->pipe_head;
  CK(cudaEventSynchronize(n->ev_step_done[k]));
  *loss_host = n->loss_pinned[k];
  n->pipe_head ^= 1;
  n->pipe_count--;
  return MBD_OK;
}

extern "C" mbd_status mbd_get_tensor(mbd_net* n, int which, int layer, void* dst, size_t bytes) {
  if (!n || !dst) return MBD_E_INVALID;
  if (n->is_conv) return conv_get_tensor(n->conv, which, layer, dst, bytes);
  if (n->mixed && which != MBD_T_LOSS && which != MBD_T_PARTIALS) {
    if (layer >= 0 && layer < n->Lc) return conv_get_tensor(n->conv, which, layer, dst, bytes);
    layer -= n->Lc;
  }
  const void* src = nullptr;
  size_t size = 0;
  if (which == MBD_T_LOSS) {
    src = n->per_sample; size = n->B * sizeof(float);
  } else if (which == MBD_T_PARTIALS) {
    src = n->last_red_dw ? n->partials_dw : n->partials; size = bytes;
    if (bytes > (n->last_red_dw ? n->last_dw_elems : n->partial_elems) * sizeof(float)) return MBD_E_INVALID;
  } else {
    if (layer < 0 || layer >= n->L) return MBD_E_INVALID;
    Layer& l = n->layers[layer];
    const bool last = layer == n->L - 1;
    switch (which) {
      case MBD_T_ACT: src = l.act; size = static_cast<size_t>(n->B) * l.d_out * (last ? sizeof(float) : n->elt()); break;
      case MBD_T_DY: src = l.dY; size = static_cast<size_t>(n->B) * l.d_out * n->elt(); break;
      case MBD_T_DW: src = l.dW; size = l.nW * sizeof(float); break;
      case MBD_T_MASTER: src = l.W32; size = l.nW * sizeof(float); break;
      case MBD_T_VELOCITY: src = l.V; size = l.nW * sizeof(float); break;
      case MBD_T_VELOCITY_BIAS: src = l.Vb; size = l.d_out * sizeof(float); break;
      case MBD_T_DB: src = l.db; size = l.d_out * sizeof(float); break;
      default: return MBD_E_INVALID;
    }
  }
  if (!src || bytes != size) return MBD_E_INVALID;
  CK(cudaMemcpyAsync(dst, src, size, cudaMemcpyDeviceToDevice, n->stream));
  return MBD_OK;
}

extern "C" mbd_status mbd_set_tensor(mbd_net* n, int which, int layer, const void* src, size_t bytes) {
  if (!n || !src) return MBD_E_INVALID;
  if (n->is_conv) return which == MBD_T_DW ? conv_set_dw(n->conv, layer, src, bytes) : conv_set_tensor(n->conv, which, layer, src, bytes);
  if (n->mixed) {
    if (layer >= 0 && layer < n->Lc) {
      const mbd_status s = conv_set_tensor(n->conv, which, layer, src, bytes);
      // the last convolution's stored output is also the first fully connected layer's input
      if (s == MBD_OK && which == MBD_T_ACT && layer == n->Lc - 1)
        CK(cudaMemcpyAsync(n->X_fc, src, bytes, cudaMemcpyDeviceToDevice, n->stream));
      return s;
    }
    layer -= n->Lc;
  }
  if (layer < 0 || layer >= n->L) return MBD_E_INVALID;
  Layer& l = n->layers[layer];
  const bool last = layer == n->L - 1;
  void* dst = nullptr;
  size_t size = 0;
  if (which == MBD_T_ACT) { dst = l.act; size = static_cast<size_t>(n->B) * l.d_out * (last ? sizeof(float) : n->elt()); }
  else if (which == MBD_T_DY) { dst = l.dY; size = static_cast<size_t>(n->B) * l.d_out * n->elt(); }
  else return MBD_E_INVALID;
  if (bytes != size) return MBD_E_INVALID;
  CK(cudaMemcpyAsync(dst, src, size, cudaMemcpyDeviceToDevice, n->stream));
  return MBD_OK;
}

// ---- the convolution step piece by piece (pure convolution stacks; one process per strip, Section 2.2) ----
extern "C" mbd_status mbd_conv_stage_input(mbd_net* n, const void* X_dev) {
  if (!n || !X_dev) return MBD_E_INVALID;
  if (!n->is_conv) return MBD_E_UNSUPPORTED;
  n->state = ST_IDLE;
  return conv_stage_input(n->conv, X_dev);
}

extern "C" mbd_status mbd_conv_forward_layer_rows(mbd_net* n, int layer, int rows, float* loss_sum_dev) {
  if (!n) return MBD_E_INVALID;
  if (!n->is_conv) return MBD_E_UNSUPPORTED;
  if (layer < 0 || layer >= n->Lc || rows < MBD_ROWS_ALL || rows > MBD_ROWS_BOUNDARY) return MBD_E_INVALID;
  const mbd_status s = conv_forward_layer(n->conv, layer, loss_sum_dev, rows);
  if (s == MBD_OK && layer == n->Lc - 1 && rows != MBD_ROWS_INTERIOR) n->state = ST_FWD;
  return s;
}

extern "C" mbd_status mbd_conv_forward_layer(mbd_net* n, int layer, float* loss_sum_dev) {
  return mbd_conv_forward_layer_rows(n, layer, MBD_ROWS_ALL, loss_sum_dev);
}

extern "C" mbd_status mbd_conv_backward_layer_rows(mbd_net* n, int layer, int rows, float fused_eta) {
  if (!n || fused_eta < 0.f) return MBD_E_INVALID;
  if (!n->is_conv) return MBD_E_UNSUPPORTED;
  if (layer < 0 || layer >= n->Lc || rows < MBD_ROWS_ALL || rows > MBD_ROWS_BOUNDARY) return MBD_E_INVALID;
  if (n->state != ST_FWD) return MBD_E_STATE;
  const mbd_status s = conv_backward_layer(n->conv, layer, fused_eta, rows);
  if (s == MBD_OK && layer == 0 && rows != MBD_ROWS_INTERIOR) n->state = fused_eta > 0.f ? ST_BWD_FUSED : ST_BWD_UNFUSED;
  return s;
}

extern "C" mbd_status mbd_conv_backward_layer(mbd_net* n, int layer, float fused_eta) {
  return mbd_conv_backward_layer_rows(n, layer, MBD_ROWS_ALL, fused_eta);
}

extern "C" mbd_status mbd_conv_outer_rows(mbd_net* n, int which, int layer, int side, void* rows_dev, size_t bytes, int set) {
  if (!n || !rows_dev) return MBD_E_INVALID;
  if (!n->is_conv) return MBD_E_UNSUPPORTED;
  return conv_outer_rows(n->conv, which, layer, side, rows_dev, bytes, set);
}

extern "C" mbd_status mbd_poll_status(mbd_net* n) {
  if (!n) return MBD_E_INVALID;
  CK(cudaStreamSynchronize(n->stream));
  int h = 0;
  CK(cudaMemcpy(&h, n->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (h != 0) {
    CK(cudaMemset(n->status, 0, sizeof(int)));
    // a kernel that gave up may have left hand-over words of a running sum behind
    if (n->fix_flags) CK(cudaMemset(n->fix_flags, 0, n->fix_words * sizeof(int)));
    if (n->fix_flags_dw) CK(cudaMemset(n->fix_flags_dw, 0, n->fix_words_dw * sizeof(int)));
    return h == DEV_SMEM_MISALIGNED ? MBD_E_CUDA : MBD_E_TIMEOUT;
  }
  return MBD_OK;
}

extern "C" int64_t mbd_launch_count(const mbd_net* n) { return n ? n->prof.total_launches : -1; }

namespace {
void fill_plan(const TcGemm& g, mbd_plan* out) {
  out->tile_m = 128 * g.MH * (g.pair ? 2 : 1);
  out->tile_n = g.BN;
  out->cta_pair = g.pair;
  out->k_pieces = g.join > 1 ? g.join : g.k_splits;
  out->tma_epilogue = g.te_planes ? 2 : g.te;
  out->ctas = g.grid;
  out->running_sum = g.join > 1 ? 2 : g.fix;
  out->k_blocks = (g.K + 63) / 64;
}
}  // namespace

extern "C" mbd_status mbd_get_plan(const mbd_net* n, int layer, int product, mbd_plan* out) {
  if (!n || !out || product < 0 || product > 2) return MBD_E_INVALID;
  if (layer < 0 || layer >= n->Lc + n->L) return MBD_E_INVALID;
  if (n->dtype != MBD_BF16) return MBD_E_UNSUPPORTED;
  const TcGemm* gp = nullptr;
  if (layer < n->Lc) {
    const mbd_status s = conv_get_product(n->conv, layer, product, &gp);     // general convolution layers only
    if (s != MBD_OK) return s;
  } else {
    const int i = layer - n->Lc;
    if (product == 1 && i == 0 && !n->mixed) return MBD_E_INVALID;
    const Layer& l = n->layers[i];
    gp = product == 0 ? &l.fwd : product == 1 ? &l.bwd_data : &l.bwd_weight;
  }
  fill_plan(*gp, out);
  return MBD_OK;
}

extern "C" mbd_status mbd_plan_product(int variant, int64_t M, int64_t N, int64_t K, int k_pieces, int flags, int num_sms,
                                       mbd_plan* out) {
  if (!out || variant < 0 || variant > 2 || M < 1 || N < 1 || K < 1 || k_pieces < 1 || num_sms < 2) return MBD_E_INVALID;
  if (flags & ~(MBD_PLAN_EXTRA_CUTS | MBD_PLAN_INTERMEDIATE | MBD_PLAN_BF16_RESULT)) return MBD_E_INVALID;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return MBD_E_UNSUPPORTED;
  TcGemm g{};
  g.variant = variant;
  g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
  g.k_splits = k_pieces;
  g.allow_extra_split = (flags & MBD_PLAN_EXTRA_CUTS) != 0;
  g.allow_fix = (flags & MBD_PLAN_INTERMEDIATE) != 0;
  tc_gemm_plan(g, num_sms, (flags & MBD_PLAN_BF16_RESULT) != 0);
  fill_plan(g, out);
  return MBD_OK;
}

extern "C" mbd_status mbd_profile_enable(mbd_net* n, int on) {
  if (!n) return MBD_E_INVALID;
  n->prof.reset();
  n->prof.on = on != 0;
  return MBD_OK;
}

extern "C" mbd_status mbd_profile_read(mbd_net* n, int kclass, double* ms_total, int64_t* launches, double* work_total) {
  if (!n || kclass < 0 || kclass >= MBD_K_COUNT) return MBD_E_INVALID;
  n->prof.collect();
  if (ms_total) *ms_total = n->prof.ms[kclass];
  if (launches) *launches = n->prof.launches[kclass];
  if (work_total) *work_total = n->prof.work[kclass];
  return MBD_OK;
}

extern "C" mbd_status mbd_gemm_bf16(int variant, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                    const void* Bm, int64_t ldb, float* D, int64_t ldd, int k_splits, float* partials,
                                    void* cuda_stream) {
  if (!A || !Bm || !D || variant < 0 || variant > 2 || M < 1 || N < 1 || K < 1 || k_splits < 1) return MBD_E_INVALID;
  if (lda % 8 || ldb % 8 || ldd % 8 || N % 8) return MBD_E_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(Bm) | reinterpret_cast<uintptr_t>(D) |
       reinterpret_cast<uintptr_t>(partials)) & 15u) return MBD_E_UNSUPPORTED;      // 16-byte aligned bases
  if (k_splits > 1 && !partials) return MBD_E_INVALID;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return MBD_E_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  int* status = nullptr;
  if (dev_alloc(reinterpret_cast<void**>(&status), sizeof(int)) != MBD_OK) return MBD_E_ALLOC;
  cudaMemsetAsync(status, 0, sizeof(int), stream);
  TcGemm g{};
  g.variant = variant;
  g.M = static_cast<int>(M); g.N = static_cast<int>(N); g.K = static_cast<int>(K);
  g.k_splits = k_splits;
  g.status = status;
  mbd_status ret = MBD_OK;
  do {
    if (tc_gemm_prepare(g, A, lda, Bm, ldb, sms, nullptr) != cudaSuccess) { ret = MBD_E_CUDA; break; }
    g.epi = epi_act(D, ldd, 0, nullptr, 0);
    g.partials = partials;
    if (tc_gemm_launch(g, stream) != cudaSuccess) { ret = MBD_E_CUDA; break; }
    if (g.k_splits > 1 && reduce_partials_launch(partials, g.k_splits, M, N, g.epi, sms, stream) != cudaSuccess) { ret = MBD_E_CUDA; break; }
    if (cudaStreamSynchronize(stream) != cudaSuccess) { ret = MBD_E_CUDA; break; }
    int h = 0;
    if (cudaMemcpy(&h, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { ret = MBD_E_CUDA; break; }
    if (h != 0) ret = MBD_E_TIMEOUT;
  } while (0);
  (void)cudaGetLastError();
  cudaFree(status);
  return ret;
}

extern "C" mbd_status mbd_selftest_timeout(int limit_ms, void* cuda_stream) {
  if (limit_ms < 1 || limit_ms > 2000) return MBD_E_INVALID;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* status = nullptr;
  if (dev_alloc(reinterpret_cast<void**>(&status), sizeof(int)) != MBD_OK) return MBD_E_ALLOC;
  mbd_status ret = MBD_OK;
  int h = 0;
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess || selftest_timeout_launch(status, limit_ms, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess || cudaMemcpy(&h, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    ret = MBD_E_CUDA;
  } else if (h != 0) {
    ret = MBD_E_TIMEOUT;
  }
  (void)cudaGetLastError();
  cudaFree(status);
  return ret;
}
