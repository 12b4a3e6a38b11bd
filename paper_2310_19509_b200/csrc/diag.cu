// Set-up and diagnostic entry points: sbnn_prepare (does ahead of time what compute calls otherwise do on first
// use), a register-only FMA kernel that measures the FP32 rate the roofline is quoted against, and a test hook for
// the device-ownership check.
#include "common.h"
#include "pipeline.cuh"

namespace sbnn {
namespace {

__device__ float g_fma_sink[32];

// Every thread runs `iters` rounds of 32 packed FMAs on 16 independent accumulator pairs, all operands in
// registers: nothing but the FMA pipe is exercised.  The result is stored only if it takes a value it cannot
// take, which keeps the loop alive without any memory traffic.
__global__ void __launch_bounds__(512) fma_rate_kernel(int iters, float seed) {
    f32x2 acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = pack2(seed + (float)i, seed - (float)i);
    const f32x2 a = pack2(0.999f, 1.001f), b = pack2(seed * 0.5f, seed * 0.25f);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) fma2(acc[i], a, b);
#pragma unroll
        for (int i = 0; i < 16; ++i) fma2(acc[i], b, a);
    }
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float lo, hi;
        unpack2(acc[i], lo, hi);
        s += lo + hi;
    }
    if (s == 123456.789f) g_fma_sink[threadIdx.x & 31] = s;
}

// Device-side consistency check of a packed layer's device copies: one thread per group walks its index list.
// A violation is recorded in the status word (first one wins); nothing traps, the kernel always returns normally.
__global__ void __launch_bounds__(128)
check_packed_kernel(const int32_t* __restrict__ group_ptr, const int32_t* __restrict__ idx, int ngroups, int Cin, long long nnz,
                    int* status) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= ngroups) return;
    const long long lo = group_ptr[g], hi = group_ptr[g + 1];
    bool ok = lo >= 0 && lo <= hi && hi <= nnz && (g > 0 || lo == 0) && (g + 1 < ngroups || hi == nnz);
    for (long long u = lo; ok && u < hi; ++u) {
        const int c = idx[u];
        ok = c >= 0 && c < Cin && (u == lo || c > idx[u - 1]);
    }
    if (!ok) atomicCAS(status, 0, (int)SBNN_ERR_SHAPE);
}

}  // namespace

// defined in conv1x1_cm.cu: builds the weight streams of every tile shape the default choice can take for this layer
sbnn_status prepare_all_cm(const sbnn_packed* p);

}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_prepare(const sbnn_packed* w, int N, int H, int W, int flags) {
    clear_error();
    if (!w) return fail(SBNN_ERR_NULL, "packed weights must not be NULL");
    if (N < 0 || H < 0 || W < 0) return fail(SBNN_ERR_SHAPE, "negative activation shape %dx%dx%d", N, H, W);
    if ((int64_t)N * H * W > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "N*H*W exceeds 2^31-1");
    if ((int64_t)N * H * W == 0) return SBNN_OK;
    PrepareScope scope;   // the entry points below run their host side only
    // Stand-ins for the activation pointers: aligned, non-NULL, never dereferenced while preparing.
    const float* x = reinterpret_cast<const float*>(uintptr_t(256));
    float* y = reinterpret_cast<float*>(uintptr_t(512));
    if (w->KH == 3) return sbnn_conv3x3_gs(w, x, y, N, H, W, flags & SBNN_RELU, nullptr);
    sbnn_status st = sbnn_conv1x1_gs(w, x, y, N, H, W, flags & (SBNN_RELU | SBNN_BF16_TC | SBNN_BF16_GATHER), nullptr);
    if (st != SBNN_OK || (flags & SBNN_BF16_TC)) return st;
    return prepare_all_cm(w);
}

extern "C" sbnn_status sbnn_selftest_fma_rate(int iterations, double* flop_out, void* cuda_stream) {
    clear_error();
    if (iterations <= 0) return fail(SBNN_ERR_SHAPE, "iterations=%d must be positive", iterations);
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    int dev = 0, sms = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    SBNN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int ctas = 4 * sms, threads = 512;
    fma_rate_kernel<<<ctas, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(iterations, 1.0f);
    SBNN_CUDA_TRY(cudaGetLastError());
    // 32 packed FMAs per round, 2 lanes per packed FMA, 2 flop per FMA
    if (flop_out) *flop_out = (double)ctas * threads * (double)iterations * 32.0 * 2.0 * 2.0;
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_debug_set_packed_device(sbnn_packed* w, int device, int* previous) {
    clear_error();
    if (!w) return fail(SBNN_ERR_NULL, "packed weights must not be NULL");
    if (previous) *previous = w->device;
    w->device = device;
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_debug_check_packed(const sbnn_packed* w, void* cuda_stream) {
    clear_error();
    if (!w) return fail(SBNN_ERR_NULL, "packed weights must not be NULL");
    sbnn_status st = check_packed_device(w);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    int* status = nullptr;
    if ((st = async_status_word(&status)) != SBNN_OK) return st;
    check_packed_kernel<<<(w->ngroups + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        w->d_group_ptr, w->d_idx, w->ngroups, w->Cin, (long long)w->nnz, status);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_debug_poke_device_index(sbnn_packed* w, long long unit, int value, int* previous) {
    clear_error();
    if (!w) return fail(SBNN_ERR_NULL, "packed weights must not be NULL");
    if (unit < 0 || unit >= w->nnz) return fail(SBNN_ERR_SHAPE, "unit %lld outside [0, %lld)", unit, (long long)w->nnz);
    sbnn_status st = check_packed_device(w);
    if (st != SBNN_OK) return st;
    if (previous) SBNN_CUDA_TRY(cudaMemcpy(previous, w->d_idx + unit, sizeof(int), cudaMemcpyDeviceToHost));
    SBNN_CUDA_TRY(cudaMemcpy(w->d_idx + unit, &value, sizeof(int), cudaMemcpyHostToDevice));
    return SBNN_OK;
}
