#include "conv.h"
namespace mbd {
struct ConvNet { int dummy; };
mbd_status conv_create(const mbd_layer*, int, int64_t, int, int, int, int*, cudaStream_t, Profiler*, ConvNet**) { return MBD_E_UNSUPPORTED; }
void conv_destroy(ConvNet*) {}
mbd_status conv_set_weights(ConvNet*, int, const void*) { return MBD_E_UNSUPPORTED; }
mbd_status conv_get_weights(ConvNet*, int, void*) { return MBD_E_UNSUPPORTED; }
mbd_status conv_forward(ConvNet*, const void*, float*) { return MBD_E_UNSUPPORTED; }
mbd_status conv_backward(ConvNet*, float) { return MBD_E_UNSUPPORTED; }
mbd_status conv_sgd_step(ConvNet*, float) { return MBD_E_UNSUPPORTED; }
mbd_status conv_get_tensor(ConvNet*, int, int, void*, size_t) { return MBD_E_UNSUPPORTED; }
mbd_status conv_set_tensor(ConvNet*, int, int, const void*, size_t) { return MBD_E_UNSUPPORTED; }
size_t conv_input_bytes(const ConvNet*) { return 0; }
}  // namespace mbd
