// Group-sparse 3x3 convolution (placeholder until the kernel lands).
#include "common.h"
namespace sbnn {
sbnn_status prepare_default_3x3(const sbnn_packed*) { return SBNN_OK; }
void free_streams_3x3(sbnn_packed*) {}
}  // namespace sbnn
using namespace sbnn;
extern "C" sbnn_status sbnn_conv3x3_gs(const sbnn_packed*, const float*, float*, int, int, int, int, void*) {
    clear_error();
    return fail(SBNN_ERR_UNSUPPORTED, "3x3 kernel not built yet");
}
