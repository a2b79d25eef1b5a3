/* mbd.h -- C ABI of libmbd: one minibatch-SGD training step in matrix form,
 * computed on one B200 over a logical P_r x P_c block grid.
 *
 * Per layer i = 1..L (Section 1 and Appendix A.1/A.2 of the paper):
 *     forward          Y_i  = W_i X_i (+ b_i),  X_{i+1} = ReLU(Y_i)
 *     backward-data    dX_i = W_i^T dY_i            (i >= 2)
 *     backward-weight  dW_i = dY_i X_i^T = sum_b dY_i[:,b] X_i[:,b]^T
 *     update (Eq. 1)   W_i <- W_i - (eta/B) dW_i
 * The grid (Section 2.3): P_r splits the model dimension d_i (or, for a
 * domain-split convolution layer, the image height into row strips with halo
 * rows, Section 2.2/2.4); P_c splits the batch.  The sum over the P_r row
 * blocks that forms dX and the sum over the P_c batch blocks that forms dW
 * (the paper's all-reduces) are taken on the device: consecutive logical
 * blocks are either chained in the tensor-memory accumulator or written as
 * fp32 partials and added, in ascending block order, by a reduction kernel.
 * The last part of this file holds the calls a multi-process driver needs to
 * run the same grid with one process per position (block operations, the
 * convolution step piece by piece).
 *
 * Conventions
 *   - Every pointer named *_dev is DEVICE memory, every *_host is HOST memory.
 *   - Activations are [B, d] row-major (row = sample = one column of the
 *     paper's X_i); weights are [d_i, d_{i-1}] row-major; convolution input is
 *     NCHW, its kernel [C_out, C_in, 3, 3] (or [C_out, C_in, 1, 1]).
 *   - dtype MBD_BF16: X, W, activations and dY are bfloat16 bit patterns,
 *     accumulation, logits, loss, partials, dW, biases are float.
 *     dtype MBD_F32: everything float (no tensor cores; the <=1e-5 check mode).
 *   - Calls only enqueue work on the stream given at creation (the bias-gradient
 *     column sums use a side stream of the library that is forked from and joined
 *     back into that stream inside mbd_backward; the pipelined host step copies
 *     its batches on a copy stream of the library); nothing synchronises except
 *     mbd_poll_status, mbd_train_step_host, mbd_train_step_host_end, creation /
 *     destruction, and the stand-alone calls that say so (mbd_gemm_bf16*, the block
 *     operations in their synchronous form).  The library owns weights, activations, gradients and
 *     workspace; the caller owns every buffer it passes in.
 *   - Errors are return codes; nothing aborts, throws or traps.
 */
#ifndef MBD_H
#define MBD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MBD_API __attribute__((visibility("default")))
#else
#define MBD_API
#endif

typedef struct mbd_net mbd_net; /* opaque */

typedef enum {
  MBD_OK = 0,
  MBD_E_INVALID = 1,     /* null pointer, bad enum, bad size                        */
  MBD_E_GRID = 2,        /* grid not realisable for these layers / batch            */
  MBD_E_ALLOC = 3,       /* device or host allocation failed                        */
  MBD_E_CUDA = 4,        /* a CUDA runtime / driver call failed                     */
  MBD_E_STATE = 5,       /* call order violated (forward -> backward -> sgd_step)   */
  MBD_E_TIMEOUT = 6,     /* a bounded device-side wait gave up (see mbd_poll_status)*/
  MBD_E_UNSUPPORTED = 7, /* shape / layer kind outside what the kernels cover       */
  MBD_E_TOO_LARGE = 8    /* beyond the fixed scratch of an allocation-free entry    */
} mbd_status;

enum { MBD_FC = 0, MBD_CONV3X3 = 1 };                 /* mbd_layer.kind                      */
enum { MBD_SPLIT_MODEL = 0, MBD_SPLIT_DOMAIN = 1,     /* mbd_layer.split: L_M or L_D, Eq. 9  */
       MBD_SPLIT_BATCH = 2 };  /* Section 3's improved case: this layer runs batch-parallel on a 1 x P grid
                                  (P = P_r P_c) whatever the grid of the other layers -- "we force P_r = 1,
                                  P_c = P for the convolutional layers and use varying P_r x P_c grids for the
                                  fully connected layers"; convolution layers only, and all of them alike */
enum { MBD_F32 = 0, MBD_BF16 = 1 };                   /* dtype                               */
enum { MBD_LOSS_SOFTMAX_CE = 0, MBD_LOSS_HALF_SSQ = 1,
       MBD_LOSS_NONE = 2 };   /* convolution stacks only: no loss here.  The last layer applies its ReLU like
                                 any other, and the caller supplies dJ/dY of the last layer with
                                 mbd_set_tensor(MBD_T_DY, L-1) between the forward and the backward pass
                                 (the stack is the lower part of a larger network). */

/* One layer.  FC: d_in, d_out.  Convolution (kh x kw, both odd, zero pad floor(k/2), NCHW; see mbd_net_create
 * for the shapes that exist): C_in, C_out, kh, kw, the INPUT image size H x W and the stride (0 or 1: every
 * position; s: the positions (s h', s w') of the stride-1 result, an H/s x W/s output -- H and W must be multiples of
 * s); d_in = C_in*H*W, d_out = C_out*(H/s)*(W/s); |W_i| = kh kw C_in C_out (Eq. 2).
 * relu: apply f = ReLU after this layer (ignored for the last layer).
 * bias: FC only. */
typedef struct {
  int32_t kind, split, relu, bias;
  int64_t d_in, d_out;
  int32_t C_in, C_out, H, W, kh, kw;
  int32_t stride, reserved;
} mbd_layer;

/* Words (matrix elements) one process moves for one layer under the chosen
 * grid: the bandwidth terms of Eq. 8 (model-split layers) and Eq. 9
 * (domain-split layers). */
typedef struct {
  int64_t allgather_y;   /* Eq. 8 term 1:  B/P_c (P_r-1)/P_r d_i                    */
  int64_t allreduce_dx;  /* Eq. 8 term 2:  2 B/P_c (P_r-1)/P_r d_{i-1}, 0 for i = 1 */
  int64_t allreduce_dw;  /* Eq. 8 term 3:  2 (P_c-1)/P_c |W_i|/P_r ; Eq. 9 term 6:  */
                         /*                2 (P-1)/P |W_i| for a domain-split layer; */
                         /* Eq. 4: the same 2 (P-1)/P |W_i| for a batch-split layer  */
                         /* (its only term)                                          */
  int64_t halo_fwd;      /* Eq. 9 term 4:  B/P_c X_W X_C floor(k_h/2), 0 if P_r = 1 */
  int64_t halo_bwd;      /* Eq. 9 term 5:  B/P_c Y_W Y_C floor(k_h/2), 0 if P_r = 1 */
} mbd_words;

/* Tensors readable through mbd_get_tensor. */
enum {
  MBD_T_ACT = 0,      /* stored forward output of `layer`: ReLU(Y_i) in the activation dtype,
                         or the raw fp32 logits Y_L for the last FC layer; [B, d_i]          */
  MBD_T_DY = 1,       /* dJ/dY_i, activation dtype, [B, d_i]                                 */
  MBD_T_DW = 2,       /* dW_i, float, weight shape (valid after mbd_backward(net, 0))        */
  MBD_T_DB = 3,       /* db_i, float [d_i]                                                   */
  MBD_T_LOSS = 4,     /* per-sample loss, float [B] (softmax-CE); layer ignored              */
  MBD_T_PARTIALS = 5, /* fp32 partial-sum workspace as left by the LAST reduction executed   */
  MBD_T_MASTER = 6,   /* fp32 master weights, weight shape (get only; after mbd_enable_master_weights) */
  MBD_T_VELOCITY = 7, /* momentum velocity of W_i, float, weight shape (get only; after mbd_enable_momentum) */
  MBD_T_VELOCITY_BIAS = 8 /* momentum velocity of b_i, float [d_i] (fully connected layers with a bias)    */
};

/* Section 2.3 / 2.4.  Builds the plan for an L-layer network on batch B over a
 * logical P_r x P_c grid and allocates all device state (weights start at zero).
 *   max_partials  how many separate fp32 partial sums a reduction over P blocks is
 *                 formed from: S = min(P, max_partials) partials, each chaining
 *                 P/S consecutive logical blocks in the accumulator; 0 selects
 *                 the default (4); 1 never leaves the accumulator; >= P keeps every
 *                 block's partial as a plane of its own, exactly as the paper's
 *                 processes would hold it, and a reduction kernel adds the planes.
 *                 With 1 < S < P the partials are intermediate: they are either
 *                 written as S planes and reduced the same way, or (two long pieces
 *                 of a product with more output tiles than SMs) added as a running sum inside the
 *                 product -- the CTA that finishes piece s of a tile adds it to the
 *                 sum of pieces 0..s-1 that the CTA before it left in one fp32 plane
 *                 and the last one applies the tail operation -- or (two or four short
 *                 pieces) kept as S accumulators of one tile in tensor memory, which the
 *                 product's epilogue adds before its tail operation.  All three forms add
 *                 in ascending block order and give bit-identical results; mbd_get_plan
 *                 tells which one a product uses.
 *   cuda_stream   a cudaStream_t (may be NULL for the default stream).
 * Layer order (Section 2.4, Eq. 9): domain-split convolutions first (L_D), model-split
 * fully connected layers after them (L_M); either group may be empty.  With both present
 * the input is NCHW, the first fully connected layer reads the last convolution's output
 * as [B, C*H*W] (row index c*H*W + h*W + w; its d_in must equal that), the loss is
 * softmax-CE, the dtype bf16, and the public layer index counts the convolutions first.
 * On a P_r x P_c grid a convolution is cut into P_r row strips (the balanced ranges
 * [floor(s H / P_r), floor((s + 1) H / P_r)): heights differ by at most one row) and P_c batch blocks, a
 * fully connected layer into P_r row blocks of W_i and the same P_c batch blocks.
 * MBD_E_GRID if P_r < 1, P_c < 1, P_c > B, P_r > min d_i over model-split layers,
 * a strip would be shorter than its halo, or (batch-split convolutions) P_r P_c > B.
 * Batch-split convolutions (MBD_SPLIT_BATCH) are cut into P_r P_c batch blocks and no strips; between them
 * and the fully connected layers on P_r x P_c lies the re-distribution of Eq. 6 (mbd_redistribute_time).
 * Model-split convolutions (MBD_SPLIT_MODEL: convolutions in L_M, Eq. 8 with |W| = k_h k_w C_in C_out) are cut like
 * a fully connected layer: the P_r groups split the output channels, the P_c groups the batch, no strips; dX is the
 * sum over the groups' partial results (min(P_r, max_partials) partial sums, added in ascending group order), dK a
 * sum over the batch blocks.  Stride 1, and C_out a multiple of 64 P_r (a group's channels are whole 64-channel
 * blocks of the backward-data product's K range): MBD_E_UNSUPPORTED otherwise.
 * The convolutions of one network may be split in different ways, each layer in L_M or L_D on its own (Section 2.4):
 * between two runs of layers with different kinds the activation and, backward, its gradient change their
 * distribution (the re-distribution of Eq. 6; here a pass through the NCHW form).  Such a network runs on the
 * contraction kernel whatever its shapes; the row-range calls are then unsupported.
 * Convolutions (kind MBD_CONV3X3 whatever the kernel size; Section 2.2): zero padding floor(k/2), k_h and
 * k_w odd and at most 11, stride 1 to 4 (the same in both directions), C_in and C_out multiples of 8, C_in of a layer =
 * C_out of the layer below, H x W of a layer = the output size of the layer below (H/s x W/s of its input);
 * weights [C_out][C_in][k_h][k_w] ([C_out][C_in] for 1x1).  A strip needs floor(k_h/2) halo rows
 * from each neighbour, which must be the adjacent strip's own rows: MBD_E_GRID when a strip is shorter than that.  The
 * stride-1 layers with 64 channels and 3x3 or 1x1 kernels run on kernels of their own; every other shape runs as
 * products of row-shifted views on the contraction kernel of the fully connected layers; there the interior /
 * boundary calls and mbd_conv_outer_rows are MBD_E_UNSUPPORTED, and so are strips of unequal height under a strided
 * layer (H and H / s of a strided layer must be multiples of P_r).
 * MBD_E_UNSUPPORTED for other convolutions (even or larger kernels, other channel counts, larger strides),
 * a convolution above a fully connected layer, half-SSQ with
 * fully connected layers or softmax-CE without them, or bf16 FC dims that are not
 * multiples of 8. */
MBD_API mbd_status mbd_net_create(const mbd_layer* layers_host, int L, int64_t B, int P_r, int P_c,
                          int dtype, int loss, int max_partials, void* cuda_stream, mbd_net** out);
MBD_API mbd_status mbd_net_destroy(mbd_net* net);

/* Optional, bf16 networks: keep an fp32 master copy of every weight.  Eq. 1 is then applied to the
 * master (w32 += -(eta/B) dW, from the fp32 gradient) and the bf16 weights the contractions read are
 * the rounded master, so updates below half a bf16 ulp accumulate instead of being lost.  Costs
 * 4 + 4 + 2 bytes of update traffic per weight plus the fp32 gradient instead of 2 + 2 (the update
 * leaves the contraction's epilogue).  The masters start from the current weights and follow every
 * later mbd_set_weights.  MBD_E_UNSUPPORTED for an fp32 network (its weights are fp32 already). */
MBD_API mbd_status mbd_enable_master_weights(mbd_net* net);

/* Optional: heavy-ball momentum in place of the plain step of Eq. 1 (Section 2: SGD stands for any first-order
 * method; forward pass, back-propagation and their communication are the same).  Per parameter
 *     v <- mu v + dW / B ,   w <- w - eta v ,        0 <= mu < 1, v = 0 when this call returns;
 * mu = 0 is Eq. 1.  The velocities are fp32 (4 more bytes per parameter, biases included).  The update no longer
 * rides in a product's epilogue or a reduction's tail: with fused_eta > 0 mbd_backward materialises dW_i (as with
 * fused_eta = 0) and one streaming kernel per layer applies the two lines above -- to the fp32 master when
 * master weights are on, the bf16 weights being its rounding.  mbd_sgd_step does the same from the stored
 * gradients.  Calling it again resets the velocities and sets a new mu.  MBD_E_INVALID for mu outside [0, 1). */
MBD_API mbd_status mbd_enable_momentum(mbd_net* net, float mu);

/* Copy weights (network dtype) and bias (float, may be NULL) device -> library / back. */
MBD_API mbd_status mbd_set_weights(mbd_net* net, int layer, const void* W_dev, const float* bias_dev);
MBD_API mbd_status mbd_get_weights(mbd_net* net, int layer, void* W_dev, float* bias_dev);

/* Forward pass (Section 1, Appendix A.1) and loss.  X_dev [B, d_0] (or NCHW) in the
 * network dtype must stay valid and unchanged until the following mbd_backward has
 * finished on the stream.  labels_dev: int32 [B] in [0, d_L) (softmax-CE; NULL for
 * half-SSQ).  loss_sum_dev (may be NULL) receives J = sum over the batch. */
MBD_API mbd_status mbd_forward(mbd_net* net, const void* X_dev, const int32_t* labels_dev,
                       float* loss_sum_dev);

/* Backward pass (Section 1, Appendix A.2) over the grid.  fused_eta == 0: dW_i and
 * db_i are materialised in float and weights are left alone.  fused_eta > 0: the update
 * of Eq. 1 with eta = fused_eta is applied inside the backward-weight epilogue (or the
 * tail of its reduction) and dW is not kept. */
MBD_API mbd_status mbd_backward(mbd_net* net, float fused_eta);

/* Eq. 1 from the materialised gradients.  MBD_E_STATE if there was no backward since
 * the last forward, or if that backward already applied the update. */
MBD_API mbd_status mbd_sgd_step(mbd_net* net, float eta);

/* One whole step on DEVICE buffers: mbd_forward + mbd_backward(eta) with the fused update, J
 * written to loss_sum_dev (may be NULL).  The launch sequence is captured into a CUDA graph at the
 * first call with a given (X_dev, labels_dev, eta, loss_sum_dev) and replayed afterwards, which
 * removes the per-kernel launch cost that dominates small networks; any change of these arguments
 * re-captures.  While profiling is enabled, or if the network was created on the default stream
 * (which cannot be captured), the kernels are launched directly.  Enqueue only. */
MBD_API mbd_status mbd_train_step(mbd_net* net, const void* X_dev, const int32_t* labels_dev, float eta,
                          float* loss_sum_dev);

/* One whole step from HOST buffers: copies X_host / labels_host to the device, runs
 * forward, backward with the fused update, copies J back to *loss_host and waits. */
MBD_API mbd_status mbd_train_step_host(mbd_net* net, const void* X_host, const int32_t* labels_host,
                               float eta, float* loss_host);

/* The same step, pipelined over two batches: _begin enqueues the host-to-device copy of this
 * batch on a copy stream of the library (into one of two device staging slots), then the step
 * and the device-to-host copy of J on the network's stream, and returns at once; _end waits
 * for the OLDEST step begun and returns its J.  With two steps in flight the copy of batch
 * k+1 runs under the compute of batch k.  X_host / labels_host must stay unchanged until the
 * matching _end has returned; pinned host memory keeps the copies asynchronous.
 * MBD_E_STATE: _begin with two steps already in flight, _end with none. */
MBD_API mbd_status mbd_train_step_host_begin(mbd_net* net, const void* X_host, const int32_t* labels_host, float eta);
MBD_API mbd_status mbd_train_step_host_end(mbd_net* net, float* loss_host);

/* Eq. 8 / Eq. 9 bandwidth terms, one row per layer, exact integers (a term that is not
 * integral is rounded up).  Host only: needs no GPU and no network object. */
MBD_API mbd_status mbd_comm_words(const mbd_layer* layers_host, int L, int64_t B, int P_r, int P_c,
                          mbd_words* out_host);

/* ---- Communication time model and choice of the grid (Eq. 3-9 with their latency terms;
 * Section 3).  Host only, no GPU.  A collective costs alpha * messages + beta * words:
 * all-gather of Y_i over P_r: ceil(log2 P_r) messages; all-reduce of dX_i (layers >= 2) over
 * P_r: 2 ceil(log2 P_r); all-reduce of dW_i over P_c: 2 ceil(log2 P_c); a domain-split layer:
 * one message per halo exchange (none for a single strip or a 1 x 1 kernel) and 2 ceil(log2 P) for its
 * all-reduce over all P processes.  The words are those of mbd_comm_words before rounding. */
typedef struct {
  double alpha;   /* latency per message, seconds                           */
  double beta;    /* inverse bandwidth, seconds per word (one matrix element) */
} mbd_machine;

typedef struct { double allgather_y, allreduce_dx, allreduce_dw, halo_fwd, halo_bwd; } mbd_times;  /* seconds */

typedef enum {
  MBD_GRID_UNIFORM = 0,     /* every layer on the same P_r x P_c grid, split as its `split` field says     */
  MBD_GRID_CONV_BATCH = 1   /* convolutions batch-parallel on 1 x P, fully connected layers on P_r x P_c   */
} mbd_grid_policy;

typedef struct {
  int P_r, P_c;
  double comm_fwd;   /* all-gathers, forward halos, redistribution (Eq. 6) */
  double comm_bwd;   /* all-reduces, backward halos                        */
  double comm;       /* comm_fwd + comm_bwd                                */
  double total;      /* with the compute time, see mbd_total_time          */
} mbd_grid_row;

/* Per-layer terms of Eq. 9 (Eq. 8 if no layer is domain-split) in seconds; out_host has L rows.
 * MBD_E_GRID as for mbd_comm_words. */
MBD_API mbd_status mbd_comm_time(const mbd_layer* layers_host, int L, int64_t B, int P_r, int P_c,
                                 const mbd_machine* machine, mbd_times* out_host);

/* Eq. 6 for a grid: all-gather of a (B / P_c) x d block over the P_r processes of a group,
 * paid when a batch-parallel layer feeds a layer on a P_r x P_c grid (P_c = 1: Eq. 6 itself). */
MBD_API mbd_status mbd_redistribute_time(int64_t B, int P_r, int P_c, int64_t d, const mbd_machine* machine,
                                         double* out_host);

/* compute + comm_fwd + comm_bwd; with overlap != 0 the backward communication hides behind
 * the backward compute, taken as two thirds of `compute` (two of the three products per
 * layer): compute + comm_fwd + max(0, comm_bwd - 2/3 compute).  The paper shows this variant
 * only as a figure; the formula is this library's reading of it. */
MBD_API mbd_status mbd_total_time(double compute, double comm_fwd, double comm_bwd, int overlap, double* out_host);

/* One row per feasible factorisation P = P_r * P_c, ascending P_r.  Feasible: P_c <= B; P_r
 * at most the outputs of every model-split layer and at most the rows H of every domain-split
 * layer; MBD_GRID_CONV_BATCH also needs P <= B and charges Eq. 6 at the first fully connected
 * layer that follows a convolution when P_r > 1 and charge_redistribution != 0.
 * rows_host may be NULL (cap 0) to ask for the count; *n_rows is always the full count;
 * MBD_E_INVALID if cap is smaller than that and rows_host is not NULL. */
MBD_API mbd_status mbd_grid_table(const mbd_layer* layers_host, int L, int64_t B, int P, const mbd_machine* machine,
                                  int policy, double compute, int overlap, int charge_redistribution,
                                  mbd_grid_row* rows_host, int cap, int* n_rows);

/* The row of mbd_grid_table with the least `total`; ties go to the smaller P_r.  MBD_E_GRID if
 * no factorisation is feasible. */
MBD_API mbd_status mbd_choose_grid(const mbd_layer* layers_host, int L, int64_t B, int P, const mbd_machine* machine,
                                   int policy, double compute, int overlap, int charge_redistribution,
                                   mbd_grid_row* best_host);

/* Copy an internal tensor to dst_dev; `bytes` must equal the tensor's size. */
MBD_API mbd_status mbd_get_tensor(mbd_net* net, int which, int layer, void* dst_dev, size_t bytes);

/* Overwrite an internal tensor (MBD_T_ACT or MBD_T_DY; MBD_T_DW on a convolution stack) from
 * src_dev, same shapes and types as mbd_get_tensor.  Writing the stored activations between
 * mbd_forward and mbd_backward fixes the ReLU decisions [X_{i+1} > 0] the backward pass will take
 * (the parity tests do); MBD_T_DY of the last layer is how a MBD_LOSS_NONE stack receives its top
 * gradient; MBD_T_DW is how a multi-process driver puts back a summed weight gradient. */
MBD_API mbd_status mbd_set_tensor(mbd_net* net, int which, int layer, const void* src_dev, size_t bytes);

/* Waits for the stream and reads the device status word: MBD_OK, or MBD_E_TIMEOUT if
 * a kernel's bounded barrier wait ran out, or MBD_E_CUDA. */
MBD_API mbd_status mbd_poll_status(mbd_net* net);

/* Per-kernel-class device timing with CUDA events on the network's stream.  While enabled,
 * every launch is bracketed by two events; mbd_profile_read waits for the stream and returns,
 * for one class, the summed duration (ms), the number of launches and the summed ALGORITHMIC
 * work of those launches: flops (2 M N K) for the contraction classes, bytes for the others.
 * mbd_profile_enable(net, 1) also clears the counters.  MBD_K_HALO: the passes between NCHW and the
 * strip layout (they also fill the halo rows of what they write; the halo rows of a tensor a
 * convolution produces are stored by that convolution's epilogue and have no launch of their own). */
enum {
  MBD_K_GEMM_FWD = 0, MBD_K_GEMM_BWD_DATA = 1, MBD_K_GEMM_BWD_WEIGHT = 2, MBD_K_REDUCE = 3,
  MBD_K_SOFTMAX = 4, MBD_K_COLSUM = 5, MBD_K_SGD = 6, MBD_K_HALO = 7, MBD_K_CONV_FWD = 8,
  MBD_K_CONV_BWD_DATA = 9, MBD_K_CONV_BWD_WEIGHT = 10, MBD_K_OTHER = 11, MBD_K_COUNT = 12
};
MBD_API mbd_status mbd_profile_enable(mbd_net* net, int on);
MBD_API mbd_status mbd_profile_read(mbd_net* net, int kclass, double* ms_total, int64_t* launches,
                            double* work_total);

/* Kernels launched by this network since creation (host counter). */
MBD_API int64_t mbd_launch_count(const mbd_net* net);

/* How one of the three products of Section 1 is launched for fully connected layer `layer` (public
 * index) of a bf16 network: product 0 = forward, 1 = backward-data, 2 = backward-weight.  Lets a test
 * or a benchmark state which kernel variant it ran.  tile_m x tile_n is the output tile of one work
 * unit (of the CTA pair when cta_pair != 0); k_pieces the number of fp32 partial sums the K range is
 * cut into (the grid's S = min(P, max_partials) times any further cut the planner added); running_sum != 0:
 * the pieces are added inside the product's own epilogue (see max_partials of mbd_net_create; 1: as a running sum
 * through one fp32 plane, 2: as accumulators of their own in tensor memory), otherwise
 * k_pieces > 1 means a reduce_partials launch follows; tma_epilogue = 1: the tail operation the plan was made for (bias +
 * ReLU, ReLU mask, fused update) moves its global data by TMA; tma_epilogue = 2: the k_pieces fp32 partial sums are
 * stored by TMA (short pieces on 128-row tiles); ctas: CTAs launched.
 * k_blocks: 64-deep blocks of the product's K range (for a general convolution layer (taps x channel blocks), or its
 * tap runs when a first layer with few input channels folds several taps into one block).
 * MBD_E_UNSUPPORTED for fp32 networks and for the convolution layers that run on kernels of their own (64 channels,
 * 3x3 / 1x1, stride 1), MBD_E_INVALID for a product the layer does not have (backward-data of the network's first
 * layer). */
typedef struct { int32_t tile_m, tile_n, cta_pair, k_pieces, tma_epilogue, ctas, running_sum, k_blocks; } mbd_plan;
MBD_API mbd_status mbd_get_plan(const mbd_net* net, int layer, int product, mbd_plan* out_host);

/* The same plan for a stand-alone bf16 product of Section 1 (variant as in mbd_gemm_bf16: 0 = forward Y = W X,
 * 1 = backward-data, 2 = backward-weight; output M x N, reduction length K), computed on the host without touching a
 * device: the planner is a cost model over tile shapes and cuts of K for `num_sms` SMs (>= 2), so its choices can be
 * inspected and tested where there is no GPU.  k_pieces >= 1: the pieces of K the caller's grid asks for (Appendix A.2:
 * the partial sums over a process group).  flags: MBD_PLAN_EXTRA_CUTS: the planner may cut K further to fill the SMs
 * (what a network allows for its forward and backward-data products and for the weight gradients of general
 * convolutions); MBD_PLAN_INTERMEDIATE: the pieces need not be kept as planes of their own (max_partials < P), so
 * they may be joined in tensor memory or added as a running sum; MBD_PLAN_BF16_RESULT: the result is bf16 behind a
 * tail operation, so the TMA epilogue is possible.  k_blocks = ceil(K / 64).  The environment's tuning knobs apply
 * as they do to a network.  MBD_E_INVALID for bad arguments, MBD_E_UNSUPPORTED for an extent beyond 2^31 - 1. */
enum { MBD_PLAN_EXTRA_CUTS = 1, MBD_PLAN_INTERMEDIATE = 2, MBD_PLAN_BF16_RESULT = 4 };
MBD_API mbd_status mbd_plan_product(int variant, int64_t M, int64_t N, int64_t K, int k_pieces, int flags, int num_sms,
                                    mbd_plan* out_host);

/* Stand-alone dense contraction on the tensor cores, used by the unit tests:
 *   variant 0 (forward)          D[M,N] = A[M,K]   * B[N,K]^T   A, B row-major, K contiguous
 *   variant 1 (backward-data)    D[M,N] = A[M,K]   * B[K,N]     B row-major, N contiguous
 *   variant 2 (backward-weight)  D[M,N] = A[K,M]^T * B[K,N]     A, B row-major
 * bf16 inputs, fp32 accumulation.  The K range is cut into k_splits balanced pieces;
 * k_splits == 1 writes D_dev [M,N] float directly, otherwise partials_dev
 * [k_splits][M][N] float receives the pieces and D_dev their sum (ascending order).
 * Leading dimensions are in elements and, like M/N/K offsets, multiples of 8; every base pointer is
 * 16-byte aligned (MBD_E_UNSUPPORTED otherwise: nothing is launched). */
MBD_API mbd_status mbd_gemm_bf16(int variant, int64_t M, int64_t N, int64_t K, const void* A_dev,
                         int64_t lda, const void* B_dev, int64_t ldb, float* D_dev, int64_t ldd,
                         int k_splits, float* partials_dev, void* cuda_stream);

/* ---- Block operations for a multi-process driver of the grid (Section 2.3; Appendix A.1 / A.2) ----
 * What one process (r, c) does between two collectives, on caller-owned device buffers: a block product
 * with its tail operation fused, the tail operation applied to a sum that a collective delivered, and
 * the loss.  All of them enqueue on cuda_stream.  mbd_block_gemm_bf16 with status_dev == NULL, and the
 * other two with sync != 0, return after the stream has drained (MBD_E_TIMEOUT if a bounded wait inside a
 * kernel gave up); with a caller-owned, zero-initialised device word status_dev (resp. sync == 0) they only
 * enqueue, so that a driver can overlap them with its collectives on other streams -- the caller then reads
 * the word when it likes: non-zero means a bounded wait gave up and the results are not valid.
 *
 * mbd_tail: what happens to a finished fp32 element acc at (m, n):
 *   MBD_TAIL_STORE  out = acc (+ bias_dev[n]); relu != 0: max(., 0)
 *   MBD_TAIL_MASK   out = (mask_dev == NULL || mask_dev[m, n] > 0) ? acc : 0      (ReLU derivative)
 *   MBD_TAIL_SGD    out = out + scale * acc                                          (Eq. 1, scale = -eta/B)
 * out_dev is [M, ldo] bf16 (out_bf16 != 0) or float; mask_dev has out's element type and ldmask.
 * Leading dimensions in elements, multiples of 8 for the contraction, and its bases (operands, out, mask,
 * bias) 16-byte aligned (MBD_E_UNSUPPORTED otherwise, nothing is launched).  mbd_block_reduce and
 * mbd_softmax_xent accept any alignment: they move 16 bytes per access when bases and leading dimensions
 * allow it and fall back to element-wise kernels otherwise. */
enum { MBD_TAIL_STORE = 0, MBD_TAIL_MASK = 1, MBD_TAIL_SGD = 2 };
typedef struct {
  int32_t op, out_bf16, relu, reserved;
  void* out_dev;
  int64_t ldo;
  const float* bias_dev;
  const void* mask_dev;
  int64_t ldmask;
  float scale;
} mbd_tail;

/* One block product (variants and operand layouts of mbd_gemm_bf16, K not split) with `tail` fused. */
MBD_API mbd_status mbd_block_gemm_bf16(int variant, int64_t M, int64_t N, int64_t K, const void* A_dev,
                               int64_t lda, const void* B_dev, int64_t ldb, const mbd_tail* tail,
                               int32_t* status_dev, void* cuda_stream);
/* sum_{s < S} parts_dev[s] (planes of M x N floats, ascending s), then `tail`.  S = 1 applies the tail
 * operation to a sum that is already complete (e.g. after an all-reduce). */
MBD_API mbd_status mbd_block_reduce(const float* parts_dev, int S, int64_t M, int64_t N, const mbd_tail* tail,
                            int sync, void* cuda_stream);
/* Softmax cross-entropy of float logits [B, d]: per_sample_dev[b] = loss of sample b (natural log),
 * dY_dev [B, d] = softmax - onehot (bf16 if dY_bf16 != 0, else float).  labels_dev: int32 in [0, d); a label
 * outside that range is never used as an index: the sample's loss comes back as NaN and its dY row is the
 * plain softmax (mbd_forward treats labels the same way). */
MBD_API mbd_status mbd_softmax_xent(const float* logits_dev, int64_t B, int64_t d, const int32_t* labels_dev,
                            void* dY_dev, int dY_bf16, float* per_sample_dev, int sync, void* cuda_stream);

/* ---- The convolution step piece by piece, for a driver with one process per row strip (Section 2.2) ----
 * A process holds its strip of every image as a network of its own (H = its rows) and exchanges the
 * strips' outer rows with its neighbours between the pieces: mbd_conv_stage_input, then per layer
 * [outer halo rows of the layer's input, if its kernel is 3x3] mbd_conv_forward_layer; backward per layer
 * from the top [outer halo rows of dY_layer, if 3x3 and layer > 0] mbd_conv_backward_layer (the gradient
 * with respect to the layer's input, then the layer's weight gradient).  mbd_forward / mbd_backward are
 * exactly these pieces in a row.  Pure convolution stacks only (MBD_E_UNSUPPORTED otherwise).
 *
 * mbd_conv_outer_rows: rows_dev is [B][W][C] bf16 (bytes = B*W*C*2).  set == 0 reads the first (side 0) or
 * last (side 1) OWN row of every image of the tensor -- what the process above / below needs as its halo
 * row; set != 0 writes the upper (side 0) or lower (side 1) HALO row, which is zero (the image border)
 * unless written.  which = MBD_T_ACT (output of `layer`; layer -1 = the staged input) or MBD_T_DY.
 * mbd_set_tensor(MBD_T_DW) on a convolution stack replaces the materialised weight gradient (e.g. by its
 * sum over all processes) before mbd_sgd_step.
 *
 * Section 2.2's overlap of the halo exchange with the interior computation: the _rows forms compute part of a
 * layer.  MBD_ROWS_INTERIOR = the own rows 2 .. H - 1, which read no halo row of the layer's input (forward) or of
 * dY_layer (backward): they can be enqueued while the halo rows are still travelling; MBD_ROWS_BOUNDARY = rows 1 and
 * H, after the halo rows have been written -- and, in the backward form, the layer's weight gradient (and update)
 * after them.  A 1x1 layer reads no halo: all of its rows are interior, its boundary call only finishes the layer.
 * INTERIOR then BOUNDARY leaves bit for bit the tensors MBD_ROWS_ALL (= the plain call) leaves (the loss sum adds
 * the same squares in another order).  One strip per network only
 * (P_r = 1: the network of one process), MBD_E_UNSUPPORTED otherwise. */
enum { MBD_ROWS_ALL = 0, MBD_ROWS_INTERIOR = 1, MBD_ROWS_BOUNDARY = 2 };
MBD_API mbd_status mbd_conv_stage_input(mbd_net* net, const void* X_dev);
MBD_API mbd_status mbd_conv_forward_layer(mbd_net* net, int layer, float* loss_sum_dev);
MBD_API mbd_status mbd_conv_backward_layer(mbd_net* net, int layer, float fused_eta);
MBD_API mbd_status mbd_conv_forward_layer_rows(mbd_net* net, int layer, int rows, float* loss_sum_dev);
MBD_API mbd_status mbd_conv_backward_layer_rows(mbd_net* net, int layer, int rows, float fused_eta);
MBD_API mbd_status mbd_conv_outer_rows(mbd_net* net, int which, int layer, int side, void* rows_dev,
                               size_t bytes, int set);

/* Failure-detection self test: launches one small kernel whose only job is to wait, with a
 * limit of `limit_ms` milliseconds, on a barrier that nothing will ever signal.  The kernel
 * gives up when the limit runs out, records a status code and returns normally; the call then
 * reports MBD_E_TIMEOUT (MBD_OK would mean the bounded wait did not fire).  The device context
 * stays usable.  This is the same bounded-wait path every pipeline barrier of the tensor-core
 * kernels uses (their limit is 4 s). */
MBD_API mbd_status mbd_selftest_timeout(int limit_ms, void* cuda_stream);

/* No counterpart in the paper: a convenience for callers that cannot allocate device memory
 * themselves and cannot let a library do it -- a service whose own pool owns all of the GPU's
 * memory, a plug-in that runs where cudaMalloc would stall or fail (memory exhausted, or an
 * environment that forbids implicit synchronisation), or code that wants a fixed footprint.
 * Same contraction, operand layouts, splitting and result as mbd_gemm_bf16, but the fp32
 * partial sums (k_splits > 1) and the status word live in a fixed 16 MiB array inside the
 * library's device image (present on every GPU that loads the library, until exit) and the
 * call makes no cudaMalloc / cudaFree nor any other allocating call.
 *   - MBD_E_TOO_LARGE if min(k_splits, ceil(K/64)) * M * N exceeds 4 Mi floats (k_splits > 1).
 *   - The first call on each device looks up the array's device address and opts the kernels into
 *     their shared-memory size on that device (the device must be current, as for every call); make
 *     that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     entry clears what has to start at zero.  Calls whose GPU work overlaps -- different
 *     streams or threads -- race on it: serialise them.  The call waits for cuda_stream (it reads the
 *     status word back) and returns after its work is done.
 *   - Bases 16-byte aligned, leading dimensions multiples of 8 (MBD_E_UNSUPPORTED otherwise). */
MBD_API mbd_status mbd_gemm_bf16_noalloc(int variant, int64_t M, int64_t N, int64_t K, const void* A_dev,
                                 int64_t lda, const void* B_dev, int64_t ldb, float* D_dev, int64_t ldd,
                                 int k_splits, void* cuda_stream);

MBD_API const char* mbd_strerror(mbd_status s);

#ifdef __cplusplus
}
#endif
#endif /* MBD_H */
