// General convolution layers on the contraction kernel (conv_general.cu): interface used by conv.cu, which
// forwards the calls of a network whose layers its own 64-channel 3 x 3 / 1 x 1 kernels do not cover.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/mbd.h"
#include "kernels.h"

namespace mbd {
struct GenConv;
bool gconv_needed(const mbd_layer* layers, int L);
mbd_status gconv_create(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, int max_partials, int num_sms, int* status,
                        cudaStream_t stream, Profiler* prof, bool fc_above, int model_P_r, bool need_dx0, int in_relu, GenConv** out);
void gconv_destroy(GenConv* c);
mbd_status gconv_set_weights(GenConv* c, int layer, const void* K_dev);     // K[C_out][C_in][k_h][k_w] bf16
mbd_status gconv_get_weights(GenConv* c, int layer, void* K_dev);
mbd_status gconv_stage_input(GenConv* c, const void* X_nchw);
mbd_status gconv_forward_layer(GenConv* c, int layer, float* loss_sum_dev);
mbd_status gconv_forward(GenConv* c, const void* X_nchw, float* loss_sum_dev);
mbd_status gconv_backward_layer(GenConv* c, int layer, float fused_eta);
mbd_status gconv_backward(GenConv* c, float fused_eta);
mbd_status gconv_sgd_step(GenConv* c, float eta);
mbd_status gconv_enable_master(GenConv* c);                 // fp32 master weights from now on
mbd_status gconv_enable_momentum(GenConv* c, float mu);     // heavy-ball momentum from now on, velocities zero
mbd_status gconv_get_tensor(GenConv* c, int which, int layer, void* dst, size_t bytes);
mbd_status gconv_set_tensor(GenConv* c, int which, int layer, const void* src, size_t bytes);
mbd_status gconv_set_dw(GenConv* c, int layer, const void* src, size_t bytes);
mbd_status gconv_get_product(const GenConv* c, int layer, int product, const TcGemm** out);
mbd_status gconv_output_to_nchw(GenConv* c, void* dst);
mbd_status gconv_input_grad_to_nchw(GenConv* c, void* dst_nchw);
mbd_status gconv_top_grad_from_nchw(GenConv* c, const void* src);
size_t gconv_input_bytes(const GenConv* c);
int gconv_last_relu(const GenConv* c);
}  // namespace mbd
