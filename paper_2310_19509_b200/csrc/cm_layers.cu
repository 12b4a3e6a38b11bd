// Dense supporting layers on channel-major activations ([C][ld], the pixels of a channel contiguous):
// depthwise 3x3, the thin-input first convolution (NHWC image in, channel-major out), the global
// average pool (channel-major in, [N][C] out) and a general 2-D transpose between the two layouts.
// The MobileNet chain keeps every intermediate activation in this layout so that the group-sparse
// 1x1 kernel can fill its shared-memory tiles with plain row copies.
#include "common.h"

namespace sbnn {
namespace {

// out[c][r] = in[r][c] for an R x Ccols matrix; 32 x 32 tiles through padded shared memory.
__global__ void __launch_bounds__(256)
transpose_kernel(const float* __restrict__ in, int ld_in, float* __restrict__ out, int ld_out, int R, int Ccols) {
    __shared__ float t[32][33];
    const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty + 8 * i, c = c0 + tx;
        if (r < R && c < Ccols) t[ty + 8 * i][tx] = in[(size_t)r * ld_in + c];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, r = r0 + tx;
        if (r < R && c < Ccols) out[(size_t)c * ld_out + r] = t[tx][ty + 8 * i];
    }
}

// ---- depthwise 3x3 on channel-major planes ------------------------------------------------------
// Rows of the whole batch are numbered f = n*Ho + oy on the output side and g = n*H + iy on the input
// side; with H = S*Ho the input rows of output row f are S*f - 1 .. S*f + 1, so a CTA's block of TR
// output rows needs one contiguous span of input rows, which it stages in shared memory with
// coalesced loads.  A thread then computes up to 4 consecutive outputs of one row from a 3 x (3S+3)
// register window.  Rows that belong to a neighbouring image are masked by the row index inside the
// image (top padding; bottom padding for stride 1).
template <int S>
__global__ void __launch_bounds__(256)
dwconv3x3_cm_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                    float* __restrict__ y, int ldy, int N, int H, int W, int Ho, int Wo, int TR, int SPR, int relu) {
    extern __shared__ float xs[];   // (S*TR + 2) rows x W
    const int c = blockIdx.y;
    const int f0 = blockIdx.x * TR;
    const long long NHo = (long long)N * Ho, NH = (long long)N * H;
    const int in_rows = S * TR + 2;
    const long long g0 = (long long)S * f0 - 1;          // first staged input row (may be -1)
    const float* xc = x + (size_t)c * ldx;
    for (int i = threadIdx.x; i < in_rows * W; i += blockDim.x) {
        const long long g = g0 + i / W;
        xs[i] = (g >= 0 && g < NH) ? __ldg(xc + g * W + (i % W)) : 0.0f;
    }
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * gridDim.y + c);   // weights are [3][3][C]
    const float bias = b ? __ldg(b + c) : 0.0f;
    __syncthreads();

    const int lr = threadIdx.x / SPR, strip = threadIdx.x % SPR;
    const long long f = (long long)f0 + lr;
    if (lr >= TR || f >= NHo) return;
    const int oy = (int)(f % Ho);
    const int ox0 = strip * 4;
    constexpr int IW = 3 * S + 3;
    float acc[4] = {bias, bias, bias, bias};
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;                 // row of another image or outside: zero padding
        const float* row = xs + (S * lr + kh) * W;       // staged row g0 + S*lr + kh = S*f + kh - 1
        float in[IW];
#pragma unroll
        for (int j = 0; j < IW; ++j) {
            const int ix = ox0 * S - 1 + j;
            in[j] = (ix >= 0 && ix < W) ? row[ix] : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) acc[i] = fmaf(in[i * S + kw], wk[kh * 3 + kw], acc[i]);
    }
    float* yp = y + (size_t)c * ldy + f * Wo + ox0;
    if (relu) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaxf(acc[i], 0.0f);
    }
    if (ox0 + 3 < Wo && ((f * Wo + ox0) & 3) == 0) {
        *reinterpret_cast<float4*>(yp) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (ox0 + i < Wo) yp[i] = acc[i];
    }
}

// ---- first layer: NHWC image with Cin <= 4 in, channel-major out --------------------------------
// One thread: 4 consecutive output columns of one row x 8 output channels; consecutive lanes take
// consecutive column strips, so each channel's stores are contiguous across the warp.
template <int S>
__global__ void __launch_bounds__(256)
conv3x3_thin_cm_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x,
                       float* __restrict__ y, int ldy, int N, int H, int W, int Cin, int Cout, int Ho, int Wo, int relu) {
    extern __shared__ __align__(16) float ws[];   // [9][Cin][Cout]
    for (int i = threadIdx.x; i < 9 * Cin * Cout; i += blockDim.x) {
        const int o = i % Cout, tc = i / Cout;
        ws[i] = w[(size_t)o * 9 * Cin + tc];
    }
    __syncthreads();
    constexpr int TW = 4, IW = S * (TW - 1) + 3;
    const int strips = (Wo + TW - 1) / TW;
    const long long total = (long long)N * Ho * strips;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int cg = blockIdx.y;
    const int sx = (int)(t % strips);
    const long long f = t / strips;                      // n*Ho + oy
    const int oy = (int)(f % Ho);
    const int n = (int)(f / Ho);
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
    const long long p0 = f * Wo + ox0;
    const bool vec = (ox0 + 3 < Wo) && ((p0 & 3) == 0);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float v[TW];
#pragma unroll
        for (int i = 0; i < TW; ++i) v[i] = relu ? fmaxf(acc[i][j], 0.f) : acc[i][j];
        float* yp = y + (size_t)(cg * 8 + j) * ldy + p0;
        if (vec) {
            *reinterpret_cast<float4*>(yp) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int i = 0; i < TW; ++i)
                if (ox0 + i < Wo) yp[i] = v[i];
        }
    }
}

// ---- global average pool: channel-major in ([C][ld], pixel index n*HW + p), [N][C] out -----------
// One warp per (channel, image): the HW values are contiguous; lanes stride over them and reduce.
__global__ void __launch_bounds__(256)
avgpool_cm_kernel(const float* __restrict__ x, int ldx, float* __restrict__ y, int N, int HW, int C) {
    const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (wid >= N * C) return;
    const int n = wid % N, c = wid / N;
    const float* p = x + (size_t)c * ldx + (size_t)n * HW;
    float s = 0.f;
    for (int i = lane; i < HW; i += 32) s += __ldg(p + i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) y[(size_t)n * C + c] = s * (1.0f / (float)HW);
}

}  // namespace

// ---- launchers used by the chain (arguments are validated by the callers) ---------------------
sbnn_status launch_transpose(const float* in, int ld_in, float* out, int ld_out, int R, int Ccols, cudaStream_t st) {
    if (R <= 0 || Ccols <= 0) return SBNN_OK;
    dim3 grid((R + 31) / 32, (Ccols + 31) / 32);
    if (grid.y > 65535) return fail(SBNN_ERR_SHAPE, "transpose: too many columns");
    transpose_kernel<<<grid, 256, 0, st>>>(in, ld_in, out, ld_out, R, Ccols);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

sbnn_status launch_dwconv3x3_cm(const float* w, const float* b, const float* x, int ldx, float* y, int ldy, int N, int H,
                                int W, int C, int stride, int relu, cudaStream_t st) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (H != stride * Ho) return fail(SBNN_ERR_UNSUPPORTED, "channel-major depthwise needs H divisible by the stride");
    const int SPR = (Wo + 3) / 4;
    if (SPR > 256) return fail(SBNN_ERR_UNSUPPORTED, "channel-major depthwise: row of %d pixels too wide", Wo);
    int TR = 256 / SPR;
    // keep the staged input span within the default shared-memory budget
    while (TR > 1 && (size_t)(stride * TR + 2) * W * sizeof(float) > 40 * 1024) TR /= 2;
    const size_t smem = (size_t)(stride * TR + 2) * W * sizeof(float);
    if (smem > 48 * 1024) return fail(SBNN_ERR_UNSUPPORTED, "channel-major depthwise: row of %d pixels too wide", W);
    const long long NHo = (long long)N * Ho;
    dim3 grid((unsigned)((NHo + TR - 1) / TR), C);
    if (C > 65535) return fail(SBNN_ERR_SHAPE, "too many channels");
    if (stride == 1)
        dwconv3x3_cm_kernel<1><<<grid, 256, smem, st>>>(w, b, x, ldx, y, ldy, N, H, W, Ho, Wo, TR, SPR, relu);
    else
        dwconv3x3_cm_kernel<2><<<grid, 256, smem, st>>>(w, b, x, ldx, y, ldy, N, H, W, Ho, Wo, TR, SPR, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

sbnn_status launch_conv3x3_thin_cm(const float* w, const float* b, const float* x, float* y, int ldy, int N, int H, int W,
                                   int Cin, int Cout, int stride, int relu, cudaStream_t st) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const long long total = (long long)N * Ho * ((Wo + 3) / 4);
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "tensor too large");
    dim3 grid((unsigned)blocks, Cout / 8);
    const size_t smem = sizeof(float) * 9 * Cin * Cout;
    if (stride == 1)
        conv3x3_thin_cm_kernel<1><<<grid, 256, smem, st>>>(w, b, x, y, ldy, N, H, W, Cin, Cout, Ho, Wo, relu);
    else
        conv3x3_thin_cm_kernel<2><<<grid, 256, smem, st>>>(w, b, x, y, ldy, N, H, W, Cin, Cout, Ho, Wo, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

sbnn_status launch_avgpool_cm(const float* x, int ldx, float* y, int N, int HW, int C, cudaStream_t st) {
    const long long threads = (long long)N * C * 32;
    avgpool_cm_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(x, ldx, y, N, HW, C);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

}  // namespace sbnn
