// Domain-parallel 3x3 convolution stack (Section 2.2 / 2.4): interface used by net.cu.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/mbd.h"
#include "kernels.h"

namespace mbd {
struct ConvNet;
mbd_status conv_create(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, int max_partials, int num_sms, int* status,
                       cudaStream_t stream, Profiler* prof, bool fc_above, ConvNet** out);
void conv_destroy(ConvNet* c);
mbd_status conv_set_weights(ConvNet* c, int layer, const void* K_dev);
mbd_status conv_get_weights(ConvNet* c, int layer, void* K_dev);
mbd_status conv_forward(ConvNet* c, const void* X_nchw, float* loss_sum_dev);
mbd_status conv_backward(ConvNet* c, float fused_eta);
mbd_status conv_sgd_step(ConvNet* c, float eta);
mbd_status conv_get_tensor(ConvNet* c, int which, int layer, void* dst, size_t bytes);
mbd_status conv_set_tensor(ConvNet* c, int which, int layer, const void* src, size_t bytes);
size_t conv_input_bytes(const ConvNet* c);
// fully connected layers above the convolutions: activation out / gradient in, [B, C*H*W] in NCHW order
mbd_status conv_output_to_nchw(ConvNet* c, void* dst);
mbd_status conv_top_grad_from_nchw(ConvNet* c, const void* src);
int conv_last_relu(const ConvNet* c);
mbd_status conv_enable_master(ConvNet* c);     // fp32 master weights from now on
mbd_status conv_enable_momentum(ConvNet* c, float mu);   // heavy-ball momentum from now on (velocities start at zero)
// the step piece by piece, and the outer rows of the images (for a driver with one process per strip)
mbd_status conv_stage_input(ConvNet* c, const void* X_nchw);
// rows: MBD_ROWS_ALL, or (one strip per network only) MBD_ROWS_INTERIOR / MBD_ROWS_BOUNDARY -- see include/mbd.h
mbd_status conv_forward_layer(ConvNet* c, int layer, float* loss_sum_dev, int rows);
mbd_status conv_backward_layer(ConvNet* c, int layer, float fused_eta, int rows);
mbd_status conv_outer_rows(ConvNet* c, int which, int layer, int side, void* rows, size_t bytes, int set);
mbd_status conv_set_dw(ConvNet* c, int layer, const void* src, size_t bytes);
// the contraction a general convolution layer launches for `product` (0 forward, 1 backward-data, 2 backward-weight);
// MBD_E_UNSUPPORTED for the layers that run on the convolution kernels of their own
mbd_status conv_get_product(const ConvNet* c, int layer, int product, const TcGemm** out);
}  // namespace mbd
