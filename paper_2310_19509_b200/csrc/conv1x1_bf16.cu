// bf16 tensor-core variant of the group-sparse 1x1 convolution (placeholder until the kernel lands).
#include "common.h"
namespace sbnn {
sbnn_status conv1x1_bf16(const sbnn_packed*, const float*, float*, int, int, cudaStream_t) {
    return fail(SBNN_ERR_UNSUPPORTED, "bf16 tensor-core mode not built yet");
}
void free_stream_bf16(sbnn_packed*) {}
}  // namespace sbnn
