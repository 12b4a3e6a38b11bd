// Depthwise 3x3 with 3:9 kernel patterns (Section 3.2, "DwConv3x3"; Section 3.3, Algorithm 2).
//
// Every kernel loses three of its nine weights: in each of the three rows either the first or the third
// column, which gives 2^3 patterns; a block of `go` consecutive channels shares one pattern (the paper's
// PatternInfo, go = 16, else 8 or 4).  The compact form keeps per channel and row the middle weight and the
// surviving side weight, so the kernel does 6 loads and 6 FMAs per output instead of 9, and which neighbour
// column it reads is a per-thread address offset, not a branch.
#include <string.h>

#include "common.h"

namespace sbnn {
namespace {

__device__ __forceinline__ void fma4(float4& acc, const float4& a, const float4& w) {
    acc.x = fmaf(a.x, w.x, acc.x);
    acc.y = fmaf(a.y, w.y, acc.y);
    acc.z = fmaf(a.z, w.z, acc.z);
    acc.w = fmaf(a.w, w.w, acc.w);
}

// a if p else b, as four select instructions (lanes of a warp hold different patterns, so this must not become a branch).
__device__ __forceinline__ float4 sel4(int p, const float4& a, const float4& b) {
    float4 r;
    asm("{\n\t.reg .pred q;\n\tsetp.ne.s32 q, %8, 0;\n\t"
        "selp.f32 %0, %4, %9, q;\n\tselp.f32 %1, %5, %10, q;\n\tselp.f32 %2, %6, %11, q;\n\tselp.f32 %3, %7, %12, q;\n\t}"
        : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
        : "f"(a.x), "f"(a.y), "f"(a.z), "f"(a.w), "r"(p), "f"(b.x), "f"(b.y), "f"(b.z), "f"(b.w));
    return r;
}

// One thread: TW consecutive output columns x 4 consecutive channels (a float4; go is a multiple of 4, so the four
// share the pattern).  Consecutive threads take consecutive channel quads, then consecutive strips.  The input
// window of a row is loaded whole, whatever the pattern, so that no load address waits for the pattern byte;
// the pattern only selects which neighbour enters the side FMA.  The layer is bound by memory traffic, which the
// pattern does not change (neighbouring outputs read the pruned column anyway): it saves a third of the FMAs.
template <int S, int TW>
__global__ void __launch_bounds__(256)
dwconv3x3_pattern_kernel(const float* __restrict__ w6, const uint8_t* __restrict__ pattern, int go, const float* __restrict__ b,
                         const float* __restrict__ x, float* __restrict__ y, int N, int H, int W, int C, int Ho, int Wo,
                         int relu) {
    constexpr int IW = S * (TW - 1) + 3;
    const int C4 = C >> 2, strips = (Wo + TW - 1) / TW;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)N * Ho * strips * C4;
    if (t >= total) return;
    const int c = (int)(t % C4) * 4;
    long long r = t / C4;
    const int ox0 = (int)(r % strips) * TW;
    r /= strips;
    const int oy = (int)(r % Ho), n = (int)(r / Ho);
    const unsigned pat = pattern[c / go];
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 wk[6];
#pragma unroll
    for (int i = 0; i < 6; ++i) wk[i] = __ldg(reinterpret_cast<const float4*>(w6 + (size_t)i * C + c));
    const float4 bias = b ? __ldg(reinterpret_cast<const float4*>(b + c)) : zero;
    float4 acc[TW];
#pragma unroll
    for (int i = 0; i < TW; ++i) acc[i] = bias;
    const int ix0 = ox0 * S - 1;
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;
        const float* row = x + (((size_t)n * H + iy) * W) * C + c;
        float4 in[IW];                                          // columns ix0 .. ix0 + IW - 1
#pragma unroll
        for (int j = 0; j < IW; ++j) {
            const int ix = ix0 + j;
            in[j] = (ix >= 0 && ix < W) ? __ldg(reinterpret_cast<const float4*>(row + (size_t)ix * C)) : zero;
        }
        const int left = (int)((pat >> kh) & 1u);               // bit set: the third column is pruned, the first is read
#pragma unroll
        for (int i = 0; i < TW; ++i) {
            fma4(acc[i], in[i * S + 1], wk[kh * 2 + 1]);
            fma4(acc[i], sel4(left, in[i * S], in[i * S + 2]), wk[kh * 2]);
        }
    }
    float* yp = y + (((size_t)n * Ho + oy) * Wo + ox0) * C + c;
#pragma unroll
    for (int i = 0; i < TW; ++i) {
        if (ox0 + i >= Wo) break;
        float4 v = acc[i];
        if (relu) v = make_float4(fmaxf(v.x, 0.f), fmaxf(v.y, 0.f), fmaxf(v.z, 0.f), fmaxf(v.w, 0.f));
        *reinterpret_cast<float4*>(yp + (size_t)i * C) = v;
    }
}

}  // namespace
}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_pack_dw_pattern(const float* W, const uint8_t* mask, int C, int go, uint8_t* pattern_out,
                                            float* w6_out) {
    clear_error();
    if (!W || !mask || !pattern_out || !w6_out) return fail(SBNN_ERR_NULL, "all pointers must be non-NULL");
    if (C <= 0) return fail(SBNN_ERR_SHAPE, "C=%d must be positive", C);
    if (go != 4 && go != 8 && go != 16) return fail(SBNN_ERR_GROUP, "go=%d not in {4,8,16}", go);
    if (C % go) return fail(SBNN_ERR_GROUP, "C=%d is not a multiple of go=%d", C, go);
    for (int blk = 0; blk < C / go; ++blk) {
        unsigned pat = 0;
        for (int kh = 0; kh < 3; ++kh) {
            const uint8_t* m = mask + (size_t)kh * 3 * C;          // [kw][C] of this row
            const int c0 = blk * go;
            const uint8_t first = m[0 * C + c0], mid = m[1 * C + c0], third = m[2 * C + c0];
            if (first > 1 || third > 1 || mid != 1 || first + third != 1)
                return fail(SBNN_ERR_MASK_NOT_GROUP_UNIFORM,
                            "row %d of channel %d is not a 3:9 pattern row (middle kept, exactly one side pruned)", kh, c0);
            for (int c = c0; c < c0 + go; ++c)
                if (m[c] != first || m[C + c] != mid || m[2 * C + c] != third)
                    return fail(SBNN_ERR_MASK_NOT_GROUP_UNIFORM, "channel %d deviates from the pattern of its block of %d in row %d",
                                c, go, kh);
            if (third == 0) pat |= 1u << kh;
            const int side = third == 0 ? 0 : 2;                   // the surviving side column
            for (int c = c0; c < c0 + go; ++c) {
                w6_out[(size_t)(kh * 2 + 0) * C + c] = W[(size_t)(kh * 3 + side) * C + c];
                w6_out[(size_t)(kh * 2 + 1) * C + c] = W[(size_t)(kh * 3 + 1) * C + c];
            }
        }
        pattern_out[blk] = (uint8_t)pat;
    }
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_dwconv3x3_pattern(const float* w6_dev, const uint8_t* pattern_dev, int go, const float* b_dev,
                                              const float* x_dev, float* y_dev, int N, int H, int W, int C, int stride,
                                              int flags, void* cuda_stream) {
    clear_error();
    if (!w6_dev || !pattern_dev || !x_dev || !y_dev) return fail(SBNN_ERR_NULL, "w6_dev, pattern_dev, x_dev and y_dev must not be NULL");
    if (N < 0 || H < 0 || W < 0 || C <= 0) return fail(SBNN_ERR_SHAPE, "bad shape N=%d H=%d W=%d C=%d", N, H, W, C);
    if (stride != 1 && stride != 2) return fail(SBNN_ERR_SHAPE, "stride %d: only 1 and 2", stride);
    if (go != 4 && go != 8 && go != 16) return fail(SBNN_ERR_GROUP, "go=%d not in {4,8,16}", go);
    if (C % go) return fail(SBNN_ERR_GROUP, "C=%d is not a multiple of go=%d", C, go);
    if (flags & ~SBNN_RELU) return fail(SBNN_ERR_UNSUPPORTED, "unknown flag bits 0x%x", flags);
    if (!aligned16(w6_dev) || !aligned16(x_dev) || !aligned16(y_dev) || (b_dev && !aligned16(b_dev)))
        return fail(SBNN_ERR_ALIGN, "w6_dev, b_dev, x_dev and y_dev must be 16-byte aligned");
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
        dwconv3x3_pattern_kernel<1, TW><<<(unsigned)blocks, 256, 0, s>>>(w6_dev, pattern_dev, go, b_dev, x_dev, y_dev, N, H, W, C, Ho, Wo, relu);
    else
        dwconv3x3_pattern_kernel<2, TW><<<(unsigned)blocks, 256, 0, s>>>(w6_dev, pattern_dev, go, b_dev, x_dev, y_dev, N, H, W, C, Ho, Wo, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}
