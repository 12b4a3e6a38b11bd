// Classifier head (global average pool -> 1x1 classifier) that allocates nothing.
//
// The ordinary route through sbnn_avgpool + sbnn_conv1x1_gs needs a pooled [N][C] buffer between
// the two kernels, which the caller (or sbnn_mobilenet_v1_create) has to allocate.  Code that runs
// where cudaMalloc is off limits -- inside a latency-critical serving loop, in a process whose
// memory pool is owned and capped by someone else, after the application has frozen its device
// memory map -- cannot do that.  Here the pooled buffer lives in a fixed array that is part of the
// loaded library image on every GPU.
#include "common.h"

namespace sbnn {
namespace {

constexpr int kHeadScratchFloats = SBNN_HEAD_NOALLOC_MAX_FLOATS;

// Pooled activations [N][C].  Shared by every call on this device; holds the previous call's values.
static __device__ __align__(256) float g_head_scratch[kHeadScratchFloats];

// Mean over HW positions, 4 channels per thread: x [N][HW][C] -> pooled [N][C].
__global__ void __launch_bounds__(256)
head_pool_kernel(const float* __restrict__ x, float* __restrict__ pooled, int N, int HW, int C) {
    const int C4 = C >> 2;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= N * C4) return;
    const int c4 = t % C4, n = t / C4;
    const float4* p = reinterpret_cast<const float4*>(x + (size_t)n * HW * C) + c4;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = 0; i < HW; ++i) {
        const float4 v = __ldg(p + (size_t)i * C4);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    const float inv = 1.0f / (float)HW;
    reinterpret_cast<float4*>(pooled + (size_t)n * C)[c4] = make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);
}

// Device address of the scratch array on the current device (the array's name is only a host-side
// handle; kernels must be given the address the runtime reports for it).
sbnn_status scratch_address(float** out) {
    static std::mutex mu;
    static std::map<int, float*> addr;
    int dev = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    auto it = addr.find(dev);
    if (it == addr.end()) {
        float* p = nullptr;
        SBNN_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_head_scratch));
        if (!p) return fail(SBNN_ERR_CUDA, "no device address for the head scratch array");
        it = addr.emplace(dev, p).first;
    }
    *out = it->second;
    return SBNN_OK;
}

}  // namespace
}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_head_noalloc(const sbnn_packed* fc, const float* x_dev, float* logits_dev, int N, int HW,
                                         void* cuda_stream) {
    clear_error();
    if (!fc || !x_dev || !logits_dev) return fail(SBNN_ERR_NULL, "fc, x_dev and logits_dev must not be NULL");
    if (fc->KH != 1 || fc->KW != 1) return fail(SBNN_ERR_SHAPE, "classifier must be a packed 1x1 layer");
    if (N < 0 || HW <= 0) return fail(SBNN_ERR_SHAPE, "bad shape N=%d HW=%d", N, HW);
    if (fc->Cin % 4) return fail(SBNN_ERR_UNSUPPORTED, "Cin=%d is not a multiple of 4", fc->Cin);
    if ((int64_t)N * fc->Cin > kHeadScratchFloats)
        return fail(SBNN_ERR_SHAPE, "N*Cin = %lld exceeds the fixed scratch of %d floats (SBNN_HEAD_NOALLOC_MAX_FLOATS)",
                    (long long)N * fc->Cin, kHeadScratchFloats);
    if (!aligned16(x_dev) || !aligned16(logits_dev)) return fail(SBNN_ERR_ALIGN, "x_dev and logits_dev must be 16-byte aligned");
    if (N == 0) return SBNN_OK;
    // everything that can fail is checked before the first launch: on error nothing has been enqueued
    sbnn_status st = check_packed_device(fc);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    float* pooled = nullptr;
    if ((st = scratch_address(&pooled)) != SBNN_OK) return st;
    const int total = N * (fc->Cin / 4);
    // Every pooled value the classifier reads is rewritten here first, so nothing needs clearing.
    head_pool_kernel<<<(total + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(x_dev, pooled, N, HW, fc->Cin);
    SBNN_CUDA_TRY(cudaGetLastError());
    return sbnn_conv1x1_gs(fc, pooled, logits_dev, N, 1, 1, 0, cuda_stream);
}
