// Dense supporting layers of the MobileNet-v1 chain: depthwise 3x3, the thin-input first 3x3
// convolution and the global average pool.  All are bandwidth-bound: every kernel reads and
// writes NHWC rows with float4 accesses that are contiguous across a warp.
#include "common.h"

namespace sbnn {
namespace {

// ---- depthwise 3x3 --------------------------------------------------------------------------
// One thread: 4 channels x TW consecutive output columns of one output row.  The 3 x (S*(TW-1)+3)
// input window is read once into registers and slides across the TW outputs.
template <int S, int TW>
__global__ void __launch_bounds__(256)
dwconv3x3_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x,
                 float* __restrict__ y, int N, int H, int W, int C, int Ho, int Wo, int relu) {
    const int C4 = C >> 2;
    const int strips = (Wo + TW - 1) / TW;
    const int64_t total = (int64_t)N * Ho * strips * C4;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int c4 = (int)(t % C4);
    int64_t r = t / C4;
    const int sx = (int)(r % strips); r /= strips;
    const int oy = (int)(r % Ho);
    const int n = (int)(r / Ho);
    const int ox0 = sx * TW;
    constexpr int IW = S * (TW - 1) + 3;

    const float4* w4 = reinterpret_cast<const float4*>(w);
    float4 wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w4 + i * C4 + c4);
    const float4 bias = b ? __ldg(reinterpret_cast<const float4*>(b) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
    float4 acc[TW];
#pragma unroll
    for (int i = 0; i < TW; ++i) acc[i] = bias;

    const int ix0 = ox0 * S - 1;
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;
        const float4* row = reinterpret_cast<const float4*>(x + ((size_t)n * H + iy) * W * C) + c4;
        float4 in[IW];
#pragma unroll
        for (int j = 0; j < IW; ++j) {
            const int ix = ix0 + j;
            in[j] = (ix >= 0 && ix < W) ? __ldg(row + (size_t)ix * C4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int i = 0; i < TW; ++i)
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const float4 v = in[i * S + kw], k = wk[kh * 3 + kw];
                acc[i].x = fmaf(v.x, k.x, acc[i].x);
                acc[i].y = fmaf(v.y, k.y, acc[i].y);
                acc[i].z = fmaf(v.z, k.z, acc[i].z);
                acc[i].w = fmaf(v.w, k.w, acc[i].w);
            }
    }
    float4* out = reinterpret_cast<float4*>(y + (((size_t)n * Ho + oy) * Wo) * C) + c4;
#pragma unroll
    for (int i = 0; i < TW; ++i) {
        const int ox = ox0 + i;
        if (ox >= Wo) break;
        float4 v = acc[i];
        if (relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
        out[(size_t)ox * C4] = v;
    }
}

// ---- first layer: dense 3x3 on a thin input ---------------------------------------------------
// One thread: 4 consecutive output columns x 8 output channels.  Weights sit in shared memory as
// [tap][cin][Cout] so the 8 channels of a thread are two broadcast float4 reads.
template <int S>
__global__ void __launch_bounds__(256)
conv3x3_thin_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x,
                    float* __restrict__ y, int N, int H, int W, int Cin, int Cout, int Ho, int Wo, int relu) {
    extern __shared__ __align__(16) float ws[];  // [9][Cin][Cout]
    for (int i = threadIdx.x; i < 9 * Cin * Cout; i += blockDim.x) {
        const int o = i % Cout, tc = i / Cout;  // tc = tap*Cin + c
        ws[i] = w[(size_t)o * 9 * Cin + tc];
    }
    __syncthreads();
    constexpr int TW = 4, IW = S * (TW - 1) + 3;
    const int CG = Cout >> 3;
    const int strips = (Wo + TW - 1) / TW;
    const int64_t total = (int64_t)N * Ho * strips * CG;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int cg = (int)(t % CG);
    int64_t r = t / CG;
    const int sx = (int)(r % strips); r /= strips;
    const int oy = (int)(r % Ho);
    const int n = (int)(r / Ho);
    const int ox0 = sx * TW, ix0 = ox0 * S - 1;

    float acc[TW][8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float bv = b ? __ldg(b + cg * 8 + j) : 0.f;
#pragma unroll
        for (int i = 0; i < TW; ++i) acc[i][j] = bv;
    }
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;
        const float* row = x + ((size_t)n * H + iy) * W * Cin;
        for (int c = 0; c < Cin; ++c) {
            float in[IW];
#pragma unroll
            for (int j = 0; j < IW; ++j) {
                const int ix = ix0 + j;
                in[j] = (ix >= 0 && ix < W) ? __ldg(row + (size_t)ix * Cin + c) : 0.f;
            }
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const float4* wp = reinterpret_cast<const float4*>(ws + ((kh * 3 + kw) * Cin + c) * Cout + cg * 8);
                const float4 w0 = wp[0], w1 = wp[1];
                const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                for (int i = 0; i < TW; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(in[i * S + kw], wv[j], acc[i][j]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < TW; ++i) {
        const int ox = ox0 + i;
        if (ox >= Wo) break;
        float4* out = reinterpret_cast<float4*>(y + (((size_t)n * Ho + oy) * Wo + ox) * Cout + cg * 8);
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = relu ? fmaxf(acc[i][j], 0.f) : acc[i][j];
        out[0] = make_float4(v[0], v[1], v[2], v[3]);
        out[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
}

// ---- global average pool ------------------------------------------------------------------
__global__ void __launch_bounds__(256)
avgpool_kernel(const float* __restrict__ x, float* __restrict__ y, int N, int HW, int C) {
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
    reinterpret_cast<float4*>(y + (size_t)n * C)[c4] = make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);
}

}  // namespace
}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_dwconv3x3(const float* w_dev, const float* b_dev, const float* x_dev, float* y_dev, int N,
                                      int H, int W, int C, int stride, int flags, void* cuda_stream) {
    clear_error();
    if (!w_dev || !x_dev || !y_dev) return fail(SBNN_ERR_NULL, "w_dev, x_dev and y_dev must not be NULL");
    if (N < 0 || H < 0 || W < 0 || C <= 0) return fail(SBNN_ERR_SHAPE, "bad shape N=%d H=%d W=%d C=%d", N, H, W, C);
    if (stride != 1 && stride != 2) return fail(SBNN_ERR_SHAPE, "stride %d: only 1 and 2", stride);
    if (flags & ~SBNN_RELU) return fail(SBNN_ERR_UNSUPPORTED, "unknown flag bits 0x%x", flags);
    if (C % 4) return fail(SBNN_ERR_UNSUPPORTED, "C=%d is not a multiple of 4", C);
    if (!aligned16(w_dev) || !aligned16(x_dev) || !aligned16(y_dev) || (b_dev && !aligned16(b_dev)))
        return fail(SBNN_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if ((int64_t)N * H * W == 0) return SBNN_OK;
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    constexpr int TW = 4;
    const int64_t total = (int64_t)N * Ho * ((Wo + TW - 1) / TW) * (C / 4);
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "tensor too large");
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int relu = flags & SBNN_RELU;
    if (stride == 1)
        dwconv3x3_kernel<1, TW><<<(unsigned)blocks, 256, 0, s>>>(w_dev, b_dev, x_dev, y_dev, N, H, W, C, Ho, Wo, relu);
    else
        dwconv3x3_kernel<2, TW><<<(unsigned)blocks, 256, 0, s>>>(w_dev, b_dev, x_dev, y_dev, N, H, W, C, Ho, Wo, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_conv3x3_dense(const float* w_dev, const float* b_dev, const float* x_dev, float* y_dev,
                                          int N, int H, int W, int Cin, int Cout, int stride, int flags,
                                          void* cuda_stream) {
    clear_error();
    if (!w_dev || !x_dev || !y_dev) return fail(SBNN_ERR_NULL, "w_dev, x_dev and y_dev must not be NULL");
    if (N < 0 || H < 0 || W < 0 || Cin <= 0 || Cout <= 0) return fail(SBNN_ERR_SHAPE, "bad shape");
    if (stride != 1 && stride != 2) return fail(SBNN_ERR_SHAPE, "stride %d: only 1 and 2", stride);
    if (flags & ~SBNN_RELU) return fail(SBNN_ERR_UNSUPPORTED, "unknown flag bits 0x%x", flags);
    if (Cin > 4 || Cout % 8 || Cout > 64)
        return fail(SBNN_ERR_UNSUPPORTED, "thin-input conv needs Cin <= 4, Cout %% 8 == 0, Cout <= 64 (got %d, %d)", Cin, Cout);
    if (!aligned16(y_dev)) return fail(SBNN_ERR_ALIGN, "y_dev must be 16-byte aligned");
    if ((int64_t)N * H * W == 0) return SBNN_OK;
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const int64_t total = (int64_t)N * Ho * ((Wo + 3) / 4) * (Cout / 8);
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "tensor too large");
    const size_t smem = sizeof(float) * 9 * Cin * Cout;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int relu = flags & SBNN_RELU;
    if (stride == 1)
        conv3x3_thin_kernel<1><<<(unsigned)blocks, 256, smem, s>>>(w_dev, b_dev, x_dev, y_dev, N, H, W, Cin, Cout, Ho, Wo, relu);
    else
        conv3x3_thin_kernel<2><<<(unsigned)blocks, 256, smem, s>>>(w_dev, b_dev, x_dev, y_dev, N, H, W, Cin, Cout, Ho, Wo, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_avgpool(const float* x_dev, float* y_dev, int N, int HW, int C, void* cuda_stream) {
    clear_error();
    if (!x_dev || !y_dev) return fail(SBNN_ERR_NULL, "x_dev and y_dev must not be NULL");
    if (N < 0 || HW <= 0 || C <= 0) return fail(SBNN_ERR_SHAPE, "bad shape N=%d HW=%d C=%d", N, HW, C);
    if (C % 4) return fail(SBNN_ERR_UNSUPPORTED, "C=%d is not a multiple of 4", C);
    if (!aligned16(x_dev) || !aligned16(y_dev)) return fail(SBNN_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (N == 0) return SBNN_OK;
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    const int total = N * (C / 4);
    avgpool_kernel<<<(total + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(x_dev, y_dev, N, HW, C);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}
