// Dense supporting layers on channel-major activations ([C][ld], the pixels of a channel contiguous):
// depthwise 3x3, the thin-input first convolution (NHWC image in, channel-major out), the global
// average pool (channel-major in, [N][C] out) and a general 2-D transpose between the two layouts.
// The MobileNet chain keeps every intermediate activation in this layout so that the group-sparse
// 1x1 kernel can fill its shared-memory tiles with plain row copies.
#include "common.h"
#include "pipeline.cuh"

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
// side; with H = S*Ho the input rows of output row f are S*f - 1 .. S*f + 1.  Rows that belong to a
// neighbouring image are masked by the row index inside the image.
//
// Vector kernel (W and Wo multiples of 4): a thread owns 4 consecutive outputs of one row and one
// channel.  Per input row it reads the aligned float4 under its strip and the float4s left and right
// of it (the neighbours' strips, so those reads hit L1); consecutive lanes own consecutive strips,
// which makes every access a contiguous 512-byte warp transaction.
template <int S>
__global__ void __launch_bounds__(256)
dwconv3x3_cm_vec_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                        float* __restrict__ y, int ldy, long long NHo, int H, int W, int Ho, int Wo, int relu) {
    const int c = blockIdx.y, C = gridDim.y;
    const int spr = Wo >> 2;                                       // strips per output row
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= NHo * spr) return;
    const int strip = (int)(t % spr);
    const long long f = t / spr;
    const int oy = (int)(f % Ho);
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);      // weights are [3][3][C]
    const float bias = b ? __ldg(b + c) : 0.0f;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    float acc[4] = {bias, bias, bias, bias};
    const float* xc = x + (size_t)c * ldx;
    const int ix0 = strip * 4 * S;                                 // first input column under the strip
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;
        const float* row = xc + (f * S + kh - 1) * W;              // input row g = S*f + kh - 1
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 L = ix0 >= 4 ? __ldg(reinterpret_cast<const float4*>(row + ix0 - 4)) : z;
        const float4 A = __ldg(reinterpret_cast<const float4*>(row + ix0));
        const float k0 = wk[kh * 3], k1 = wk[kh * 3 + 1], k2 = wk[kh * 3 + 2];
        if constexpr (S == 1) {
            const float4 R = ix0 + 4 < W ? __ldg(reinterpret_cast<const float4*>(row + ix0 + 4)) : z;
            const float in[6] = {L.w, A.x, A.y, A.z, A.w, R.x};
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] = fmaf(in[i + 2], k2, fmaf(in[i + 1], k1, fmaf(in[i], k0, acc[i])));
        } else {
            const float4 B = __ldg(reinterpret_cast<const float4*>(row + ix0 + 4));   // ix0 + 7 < W always
            const float in[9] = {L.w, A.x, A.y, A.z, A.w, B.x, B.y, B.z, B.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
                acc[i] = fmaf(in[2 * i + 2], k2, fmaf(in[2 * i + 1], k1, fmaf(in[2 * i], k0, acc[i])));
        }
    }
    if (relu) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaxf(acc[i], 0.0f);
    }
    *reinterpret_cast<float4*>(y + (size_t)c * ldy + f * Wo + strip * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
}

// Row-block kernel (stride 1, W a multiple of 4, H a multiple of RR): a thread owns a strip of 4 columns in RR
// consecutive output rows of one channel and walks the RR + 2 input rows once, so an input value is loaded
// once per thread and the index arithmetic is shared by 4*RR outputs (the single-row kernel above is bound
// by instruction issue).  The values left and right of the strip come from the neighbouring lanes by
// shuffle; only the first and last lane of a warp fetch theirs from memory.  No thread leaves before the
// shuffles: threads past the end work on a clamped position and store nothing.
template <int RR>
__global__ void __launch_bounds__(128)
dwconv3x3_cm_rows_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                         float* __restrict__ y, int ldy, int items, int H, int W, int relu) {
    const int c = blockIdx.y, C = gridDim.y;
    const int spr = W >> 2;                                        // strips per row
    const int t0 = blockIdx.x * blockDim.x + threadIdx.x, lane = threadIdx.x & 31;
    const bool live = t0 < items;
    const int t = live ? t0 : items - 1;
    const int strip = t % spr, f0 = (t / spr) * RR;                // first output row (batch-wide row number)
    const int oy0 = f0 % H;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);
    const float bias = b ? __ldg(b + c) : 0.0f;
    float acc[RR][4];
#pragma unroll
    for (int o = 0; o < RR; ++o)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[o][i] = bias;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const float* xc = x + (size_t)c * ldx + (size_t)f0 * W + strip * 4;
    const bool first = strip == 0, last = strip == spr - 1;
    // all loads first (they are independent), so that a thread has RR + 2 rows in flight
    float4 A[RR + 2];
    float Le[RR + 2], Re[RR + 2];
#pragma unroll
    for (int j = 0; j < RR + 2; ++j) {                             // input row f0 - 1 + j
        const int iy = oy0 - 1 + j;
        const bool rowok = iy >= 0 && iy < H;                      // else a row of the padding (or of the next image)
        const float* row = xc + (j - 1) * W;
        A[j] = rowok ? __ldg(reinterpret_cast<const float4*>(row)) : make_float4(0.f, 0.f, 0.f, 0.f);
        Le[j] = (lane == 0 && !first && rowok) ? __ldg(row - 1) : 0.0f;
        Re[j] = (lane == 31 && !last && rowok) ? __ldg(row + 4) : 0.0f;
    }
#pragma unroll
    for (int j = 0; j < RR + 2; ++j) {
        float Lw = __shfl_up_sync(0xffffffffu, A[j].w, 1), Rx = __shfl_down_sync(0xffffffffu, A[j].x, 1);
        if (lane == 0) Lw = Le[j];
        if (lane == 31) Rx = Re[j];
        if (first) Lw = 0.0f;
        if (last) Rx = 0.0f;
        const float in[6] = {Lw, A[j].x, A[j].y, A[j].z, A[j].w, Rx};
#pragma unroll
        for (int kh = 0; kh < 3; ++kh) {
            const int o = j - kh;                                  // output row fed through tap row kh
            if (o >= 0 && o < RR) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    acc[o][i] = fmaf(in[i + 2], wk[kh * 3 + 2], fmaf(in[i + 1], wk[kh * 3 + 1], fmaf(in[i], wk[kh * 3], acc[o][i])));
            }
        }
    }
    if (!live) return;
    float* yc = y + (size_t)c * ldy + (size_t)f0 * W + strip * 4;
#pragma unroll
    for (int o = 0; o < RR; ++o) {
        float4 v = make_float4(acc[o][0], acc[o][1], acc[o][2], acc[o][3]);
        if (relu) v = make_float4(fmaxf(v.x, 0.f), fmaxf(v.y, 0.f), fmaxf(v.z, 0.f), fmaxf(v.w, 0.f));
        *reinterpret_cast<float4*>(yc + o * W) = v;
    }
}

// The same for stride 2 (W a multiple of 8, Ho a multiple of RR): 4 output columns x RR output rows per thread,
// 2*RR + 1 input rows of 8 columns each plus the column left of them, which is the left neighbour's last.
template <int RR>
__global__ void __launch_bounds__(128)
dwconv3x3_cm_rows_s2_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                            float* __restrict__ y, int ldy, int items, int Ho, int W, int relu) {
    const int c = blockIdx.y, C = gridDim.y;
    const int Wo = W >> 1, spr = Wo >> 2;
    const int t0 = blockIdx.x * blockDim.x + threadIdx.x, lane = threadIdx.x & 31;
    const bool live = t0 < items;
    const int t = live ? t0 : items - 1;
    const int strip = t % spr, f0 = (t / spr) * RR;                // first output row (batch-wide row number)
    const int oy0 = f0 % Ho;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);
    const float bias = b ? __ldg(b + c) : 0.0f;
    float acc[RR][4];
#pragma unroll
    for (int o = 0; o < RR; ++o)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[o][i] = bias;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const float* xc = x + (size_t)c * ldx + (size_t)(2 * f0) * W + strip * 8;   // input row 2*f0, first column of the strip
    const bool first = strip == 0;
    float4 A[2 * RR + 1], B[2 * RR + 1];                           // all loads first: 2*RR + 1 rows in flight
    float Le[2 * RR + 1];
#pragma unroll
    for (int j = 0; j < 2 * RR + 1; ++j) {                         // input row 2*f0 - 1 + j
        const bool rowok = j > 0 || oy0 > 0;                       // only the row above an image is padding
        const float* row = xc + (j - 1) * W;
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        A[j] = rowok ? __ldg(reinterpret_cast<const float4*>(row)) : z;
        B[j] = rowok ? __ldg(reinterpret_cast<const float4*>(row + 4)) : z;
        Le[j] = (lane == 0 && !first && rowok) ? __ldg(row - 1) : 0.0f;
    }
#pragma unroll
    for (int j = 0; j < 2 * RR + 1; ++j) {
        float Lw = __shfl_up_sync(0xffffffffu, B[j].w, 1);
        if (lane == 0) Lw = Le[j];
        if (first) Lw = 0.0f;
        const float in[9] = {Lw, A[j].x, A[j].y, A[j].z, A[j].w, B[j].x, B[j].y, B[j].z, B[j].w};
#pragma unroll
        for (int kh = 0; kh < 3; ++kh) {
            if ((j - kh) % 2 != 0) continue;
            const int o = (j - kh) / 2;                            // output row fed through tap row kh
            if (j - kh >= 0 && o < RR) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    acc[o][i] = fmaf(in[2 * i + 2], wk[kh * 3 + 2],
                                     fmaf(in[2 * i + 1], wk[kh * 3 + 1], fmaf(in[2 * i], wk[kh * 3], acc[o][i])));
            }
        }
    }
    if (!live) return;
    float* yc = y + (size_t)c * ldy + (size_t)f0 * Wo + strip * 4;
#pragma unroll
    for (int o = 0; o < RR; ++o) {
        float4 v = make_float4(acc[o][0], acc[o][1], acc[o][2], acc[o][3]);
        if (relu) v = make_float4(fmaxf(v.x, 0.f), fmaxf(v.y, 0.f), fmaxf(v.z, 0.f), fmaxf(v.w, 0.f));
        *reinterpret_cast<float4*>(yc + o * Wo) = v;
    }
}

// Kernel for the other widths (the 14- and 7-wide maps of the network).  A thread owns one output
// position (oy, ox) of one channel in up to NI consecutive images: the padding masks are computed
// once and reused for every image.  Consecutive lanes own consecutive positions of the plane, so each
// of the 9 taps is one shifted, contiguous window.  WT > 0 fixes the input width at compile time, which
// turns the 9 tap offsets into immediates of the load instructions (the kernel is bound by
// instruction issue, not by memory).
template <int S, int NI, int WT>
__global__ void __launch_bounds__(256)
dwconv3x3_cm_px_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                       float* __restrict__ y, int ldy, int N, int H, int Wrt, int C, int QB, int relu) {
    const int W = WT ? WT : Wrt;
    const int Ho = H / S, Wo = W / S;
    const int HoWo = Ho * Wo, HW = H * W;
    // small planes: a CTA takes CPB channels (CPB * HoWo <= blockDim.x), so its lanes are not left idle
    const int CPB = HoWo < (int)blockDim.x ? (int)blockDim.x / HoWo : 1;
    const int cl = CPB > 1 ? (int)threadIdx.x / HoWo : 0;
    const int c = blockIdx.y * CPB + cl;
    const int q = CPB > 1 ? (int)threadIdx.x - cl * HoWo : (blockIdx.x % QB) * (int)blockDim.x + (int)threadIdx.x;
    const int n0 = (blockIdx.x / QB) * NI;                           // first image of this thread
    if (q >= HoWo || cl >= CPB || c >= C) return;
    const int oy = q / Wo, ox = q - oy * Wo;
    float wk[9];
    bool ok[9];
#pragma unroll
    for (int kh = 0; kh < 3; ++kh)
#pragma unroll
        for (int kw = 0; kw < 3; ++kw) {
            const int iy = oy * S + kh - 1, ix = ox * S + kw - 1;
            ok[kh * 3 + kw] = iy >= 0 && iy < H && ix >= 0 && ix < W;
            wk[kh * 3 + kw] = __ldg(w + (kh * 3 + kw) * C + c);
        }
    const float bias = b ? __ldg(b + c) : 0.0f;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const float* pc = x + (size_t)c * ldx + (size_t)n0 * HW + oy * S * W + ox * S;   // centre tap, first image
    float* yc = y + (size_t)c * ldy + (size_t)n0 * HoWo + q;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        if (n0 + i >= N) break;
        float acc = bias;
#pragma unroll
        for (int kh = 0; kh < 3; ++kh)
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const float v = ok[kh * 3 + kw] ? __ldg(pc + (kh - 1) * W + (kw - 1)) : 0.0f;
                acc = fmaf(v, wk[kh * 3 + kw], acc);
            }
        *yc = relu ? fmaxf(acc, 0.0f) : acc;
        pc += HW;
        yc += HoWo;
    }
}

// Column-strip kernel for the stride-1 14- and 7-wide maps (H a multiple of 7): a thread owns 7 consecutive
// output rows of one column of one channel in up to NI consecutive images and slides a 9 x 3 register
// window down the column, so an input value is loaded once per thread instead of once per tap.  Consecutive
// lanes own consecutive columns, so every load and store of a warp covers contiguous runs of a row.
template <int NI, int WT>
__global__ void __launch_bounds__(128)
dwconv3x3_cm_col7_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                         float* __restrict__ y, int ldy, int N, int H, int C, int relu) {
    constexpr int W = WT;
    const int items = (H / 7) * W;                                   // (vertical strip, column) items of a plane
    const int QB = (items + blockDim.x - 1) / blockDim.x;
    // small planes: a CTA takes CPB channels (CPB * items <= blockDim.x), so its lanes are not left idle
    const int CPB = items < (int)blockDim.x ? (int)blockDim.x / items : 1;
    const int cl = CPB > 1 ? (int)threadIdx.x / items : 0;
    const int c = blockIdx.y * CPB + cl;
    const int q = CPB > 1 ? (int)threadIdx.x - cl * items : (blockIdx.x % QB) * (int)blockDim.x + (int)threadIdx.x;
    const int n0 = (blockIdx.x / QB) * NI;
    if (q >= items || cl >= CPB || c >= C) return;
    const int vs = q / W, ox = q - vs * W, oy0 = vs * 7;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);
    const float bias = b ? __ldg(b + c) : 0.0f;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const bool lok = ox > 0, rok = ox + 1 < W, top = oy0 > 0, bot = oy0 + 7 < H;
    const float* pc = x + (size_t)c * ldx + (size_t)n0 * H * W + (oy0 - 1) * W + ox;   // window origin (centre column)
    float* yc = y + (size_t)c * ldy + (size_t)n0 * H * W + oy0 * W + ox;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        if (n0 + i >= N) break;
        float acc[7];
#pragma unroll
        for (int o = 0; o < 7; ++o) acc[o] = bias;
#pragma unroll
        for (int r = 0; r < 9; ++r) {                                // input rows oy0-1 .. oy0+7
            const bool rowok = (r > 0 || top) && (r < 8 || bot);
            const float l = (rowok && lok) ? __ldg(pc + r * W - 1) : 0.0f;
            const float m = rowok ? __ldg(pc + r * W) : 0.0f;
            const float rr = (rowok && rok) ? __ldg(pc + r * W + 1) : 0.0f;
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                const int o = r - kh;                                // output row fed by this input row through tap row kh
                if (o >= 0 && o < 7)
                    acc[o] = fmaf(rr, wk[kh * 3 + 2], fmaf(m, wk[kh * 3 + 1], fmaf(l, wk[kh * 3], acc[o])));
            }
        }
#pragma unroll
        for (int o = 0; o < 7; ++o) yc[o * W] = relu ? fmaxf(acc[o], 0.0f) : acc[o];
        pc += H * W;
        yc += H * W;
    }
}

// 14 x 14 maps, stride 1: seven consecutive lanes own the seven column pairs of a row strip (7 output rows of one
// channel), so a lane needs one 8-byte load per input row and takes the columns left and right of its pair from
// its neighbours by shuffle: 9 load requests for 14 outputs.  (With one scalar load per tap the kernel above
// was limited by the number of load requests in flight, not by bytes.)  A warp holds 4 such strips in 28 lanes;
// lanes 28-31 only take part in the shuffles.  A CTA of 4 warps covers 8 channels x 2 strips.
template <int NI>
__global__ void __launch_bounds__(128)
dwconv3x3_cm_w14_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                        float* __restrict__ y, int ldy, int N, int C, int relu) {
    constexpr int W = 14, H = 14;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane / 7, j = lane - grp * 7;                  // strip within the warp, column pair
    const int gidx = warp * 4 + (grp & 3);
    const int cl = gidx >> 1, vs = gidx & 1;
    const int c0 = blockIdx.y * 8 + cl;
    const bool live = grp < 4 && c0 < C;
    const int c = c0 < C ? c0 : C - 1;
    const int oy0 = vs * 7, n0 = blockIdx.x * NI;
    float wk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);
    const float bias = b ? __ldg(b + c) : 0.0f;
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const float* pc = x + (size_t)c * ldx + (size_t)n0 * H * W + (oy0 - 1) * W + 2 * j;   // input row oy0 - 1, own pair
    float* yc = y + (size_t)c * ldy + (size_t)n0 * H * W + oy0 * W + 2 * j;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        if (n0 + i >= N) break;                                    // uniform over the CTA
        float2 v[9];
#pragma unroll
        for (int r = 0; r < 9; ++r) {                              // input rows oy0-1 .. oy0+7; row -1 and row 14 are padding
            const bool rowok = (r > 0 || vs == 1) && (r < 8 || vs == 0);
            v[r] = rowok ? __ldg(reinterpret_cast<const float2*>(pc + r * W)) : make_float2(0.f, 0.f);
        }
        float acc[7][2];
#pragma unroll
        for (int o = 0; o < 7; ++o) acc[o][0] = acc[o][1] = bias;
#pragma unroll
        for (int r = 0; r < 9; ++r) {
            float L = __shfl_up_sync(0xffffffffu, v[r].y, 1), R = __shfl_down_sync(0xffffffffu, v[r].x, 1);
            if (j == 0) L = 0.0f;
            if (j == 6) R = 0.0f;
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                const int o = r - kh;                              // output row fed through tap row kh
                if (o >= 0 && o < 7) {
                    acc[o][0] = fmaf(v[r].y, wk[kh * 3 + 2], fmaf(v[r].x, wk[kh * 3 + 1], fmaf(L, wk[kh * 3], acc[o][0])));
                    acc[o][1] = fmaf(R, wk[kh * 3 + 2], fmaf(v[r].y, wk[kh * 3 + 1], fmaf(v[r].x, wk[kh * 3], acc[o][1])));
                }
            }
        }
        if (live) {
#pragma unroll
            for (int o = 0; o < 7; ++o) {
                float2 out = make_float2(acc[o][0], acc[o][1]);
                if (relu) out = make_float2(fmaxf(out.x, 0.f), fmaxf(out.y, 0.f));
                *reinterpret_cast<float2*>(yc + o * W) = out;
            }
        }
        pc += H * W;
        yc += H * W;
    }
}

// 7 x 7 maps, stride 1 (the network's last depthwise layer): the planes of one channel are contiguous (49 floats per
// image), so a CTA copies the planes of up to 64 images of 2 channels into shared memory with aligned 16-byte loads,
// thread (channel, image) then holds its whole plane in registers (the 49 x 9 taps are unrolled with the padding
// resolved at compile time; plane t starts at float 49*t, an odd stride, so the lanes hit distinct banks), writes the
// 49 results back in place, and the CTA stores them with aligned 16-byte stores.  (One column strip per thread, as
// for the wider maps, left a warp's loads scattered over 4-5 planes: 15 us at batch 64 where this takes 5.)
__global__ void __launch_bounds__(128)
dwconv3x3_cm_7x7_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x, int ldx,
                        float* __restrict__ y, int ldy, int N, int C, int relu) {
    constexpr int HW = 49, NI = 64;
    __shared__ __align__(16) float sm[2][NI * HW];
    const int tid = threadIdx.x, cl = tid >> 6, img = tid & 63;
    const int n0 = blockIdx.x * NI, nimg = min(NI, N - n0), c0 = blockIdx.y * 2;
    const int c = c0 + cl;
    float wk[9];
    float bias = 0.0f;
    if (c < C) {
#pragma unroll
        for (int i = 0; i < 9; ++i) wk[i] = __ldg(w + i * C + c);
        bias = b ? __ldg(b + c) : 0.0f;
    }
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const int total = nimg * HW;                                    // floats per channel in this CTA
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if (c0 + k >= C) break;
        const float* src = x + (size_t)(c0 + k) * ldx + (size_t)n0 * HW;   // 16-byte aligned: ldx and 64 * 49 are multiples of 4
        for (int i = tid; i < (total + 3) / 4; i += 128) {
            if (4 * i + 3 < total) {
                *reinterpret_cast<float4*>(&sm[k][4 * i]) = __ldg(reinterpret_cast<const float4*>(src) + i);
            } else {
                for (int e = 4 * i; e < total; ++e) sm[k][e] = __ldg(src + e);
            }
        }
    }
    __syncthreads();
    float out[HW];
    const bool live = c < C && img < nimg;
    if (live) {
        float in[HW];
#pragma unroll
        for (int i = 0; i < HW; ++i) in[i] = sm[cl][img * HW + i];
#pragma unroll
        for (int oy = 0; oy < 7; ++oy)
#pragma unroll
            for (int ox = 0; ox < 7; ++ox) {
                float acc = bias;
#pragma unroll
                for (int kh = 0; kh < 3; ++kh)
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) {
                        const int iy = oy + kh - 1, ix = ox + kw - 1;
                        if (iy >= 0 && iy < 7 && ix >= 0 && ix < 7) acc = fmaf(in[iy * 7 + ix], wk[kh * 3 + kw], acc);
                    }
                out[oy * 7 + ox] = relu ? fmaxf(acc, 0.0f) : acc;
            }
    }
    __syncthreads();                                                // everybody has read its plane
    if (live) {
#pragma unroll
        for (int i = 0; i < HW; ++i) sm[cl][img * HW + i] = out[i];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if (c0 + k >= C) break;
        float* dst = y + (size_t)(c0 + k) * ldy + (size_t)n0 * HW;
        for (int i = tid; i < (total + 3) / 4; i += 128) {
            if (4 * i + 3 < total) {
                reinterpret_cast<float4*>(dst)[i] = *reinterpret_cast<const float4*>(&sm[k][4 * i]);
            } else {
                for (int e = 4 * i; e < total; ++e) dst[e] = sm[k][e];
            }
        }
    }
}

// ---- first layer: NHWC image with Cin <= 4 in, channel-major out --------------------------------
// Weights [Cout][3][3][Cin]; a CTA stages the 32 output channels of its channel group as [tap][Cin][32].
// Generic kernel (Cout % 32 == 0): one thread computes 2 consecutive output columns x 32 output
// channels, so every input value is loaded once per pixel pair (not once per channel group) and each
// broadcast float4 of weights feeds 4 packed FMAs (pairs of output channels, fma.rn.f32x2).  Consecutive lanes take consecutive column pairs; a
// channel's stores are 8-byte pieces that are contiguous across the warp.
template <int S>
__global__ void __launch_bounds__(128)
conv3x3_thin_cm32_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x,
                         float* __restrict__ y, int ldy, int N, int H, int W, int Cin, int Cout, int Ho, int Wo, int relu) {
    extern __shared__ __align__(16) float ws[];   // [9][Cin][32] of this CTA's channel group
    const int cg = blockIdx.y;
    for (int i = threadIdx.x; i < 9 * Cin * 32; i += blockDim.x) {
        const int o = i & 31, tc = i >> 5;
        ws[i] = w[(size_t)(cg * 32 + o) * 9 * Cin + tc];
    }
    __syncthreads();
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    constexpr int TW = 2, IW = S * (TW - 1) + 3;
    const int strips = (Wo + TW - 1) / TW;
    const long long total = (long long)N * Ho * strips;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int sx = (int)(t % strips);
    const long long f = t / strips;
    const int oy = (int)(f % Ho);
    const int n = (int)(f / Ho);
    const int ox0 = sx * TW, ix0 = ox0 * S - 1;

    f32x2 acc[TW][16];                                             // packed pairs of output channels
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float b0 = b ? __ldg(b + cg * 32 + 2 * j) : 0.f, b1 = b ? __ldg(b + cg * 32 + 2 * j + 1) : 0.f;
#pragma unroll
        for (int i = 0; i < TW; ++i) acc[i][j] = pack2(b0, b1);
    }
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * S + kh - 1;
        if (iy < 0 || iy >= H) continue;
        const float* row = x + ((size_t)n * H + iy) * W * Cin;
        for (int c = 0; c < Cin; ++c) {
            f32x2 in[IW];
#pragma unroll
            for (int j = 0; j < IW; ++j) {
                const int ix = ix0 + j;
                in[j] = dup2((ix >= 0 && ix < W) ? __ldg(row + (size_t)ix * Cin + c) : 0.f);
            }
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const ulonglong2* wp = reinterpret_cast<const ulonglong2*>(ws + ((kh * 3 + kw) * Cin + c) * 32);
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const ulonglong2 wv = wp[v];                   // channels (4v, 4v+1) and (4v+2, 4v+3)
#pragma unroll
                    for (int i = 0; i < TW; ++i) {
                        fma2(acc[i][2 * v], in[i * S + kw], wv.x);
                        fma2(acc[i][2 * v + 1], in[i * S + kw], wv.y);
                    }
                }
            }
        }
    }
    const long long p0 = f * Wo + ox0;
    const bool vec = (ox0 + 1 < Wo) && ((p0 & 1) == 0);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float v0[2], v1[2];
        unpack2(acc[0][j], v0[0], v0[1]);
        unpack2(acc[1][j], v1[0], v1[1]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float a0 = v0[e], a1 = v1[e];
            if (relu) { a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f); }
            float* yp = y + (size_t)(cg * 32 + 2 * j + e) * ldy + p0;
            if (vec) {
                *reinterpret_cast<float2*>(yp) = make_float2(a0, a1);
            } else {
                yp[0] = a0;
                if (ox0 + 1 < Wo) yp[1] = a1;
            }
        }
    }
}

// The network's first layer proper (stride 2, 3 input channels, W a multiple of 4): the 5 input columns x 3
// channels a thread needs from one image row are 15 consecutive floats that start one float after a 16-byte
// boundary, so four aligned 16-byte loads per row fetch them, and all twelve are issued before the first FMA
// (the generic kernel above issues 45 scalar loads in nine dependent batches).  Otherwise as above: 2 output
// columns x 32 output channels per thread, packed FMAs over channel pairs, weights broadcast from shared memory.
__global__ void __launch_bounds__(128)
conv3x3_first_s2c3_kernel(const float* __restrict__ w, const float* __restrict__ b, const float* __restrict__ x,
                          float* __restrict__ y, int ldy, int N, int H, int W, int Cout, int Ho, int Wo, int relu) {
    constexpr int Cin = 3;
    extern __shared__ __align__(16) float ws[];   // [9][3][32] of this CTA's channel group
    const int cg = blockIdx.y;
    for (int i = threadIdx.x; i < 9 * Cin * 32; i += blockDim.x) {
        const int o = i & 31, tc = i >> 5;
        ws[i] = w[(size_t)(cg * 32 + o) * 9 * Cin + tc];
    }
    __syncthreads();
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const int strips = Wo >> 1;
    const long long total = (long long)N * Ho * strips;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int sx = (int)(t % strips);
    const long long f = t / strips;
    const int oy = (int)(f % Ho);
    const int n = (int)(f / Ho);
    float v[3][16];                                                // per row: floats 12*sx - 4 .. 12*sx + 11
#pragma unroll
    for (int kh = 0; kh < 3; ++kh) {
        const int iy = oy * 2 + kh - 1;
        const bool rowok = iy >= 0 && iy < H;
        const float4* row = reinterpret_cast<const float4*>(x + ((size_t)n * H + (rowok ? iy : 0)) * W * Cin) + 3 * sx;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const bool ok = rowok && (q > 0 || sx > 0);            // the piece left of the row holds only the padding column
            const float4 t4 = ok ? __ldg(row + q - 1) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[kh][4 * q] = t4.x; v[kh][4 * q + 1] = t4.y; v[kh][4 * q + 2] = t4.z; v[kh][4 * q + 3] = t4.w;
        }
    }
    f32x2 acc[2][16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float b0 = b ? __ldg(b + cg * 32 + 2 * j) : 0.f, b1 = b ? __ldg(b + cg * 32 + 2 * j + 1) : 0.f;
        acc[0][j] = acc[1][j] = pack2(b0, b1);
    }
#pragma unroll
    for (int kh = 0; kh < 3; ++kh)
#pragma unroll
        for (int c = 0; c < Cin; ++c) {
            f32x2 in[5];
#pragma unroll
            for (int j = 0; j < 5; ++j) in[j] = dup2(v[kh][1 + 3 * j + c]);   // column 4*sx - 1 + j, channel c
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const ulonglong2* wp = reinterpret_cast<const ulonglong2*>(ws + ((kh * 3 + kw) * Cin + c) * 32);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const ulonglong2 wv = wp[q];
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        fma2(acc[i][2 * q], in[i * 2 + kw], wv.x);
                        fma2(acc[i][2 * q + 1], in[i * 2 + kw], wv.y);
                    }
                }
            }
        }
    const long long p0 = f * Wo + 2 * sx;                          // even, so the pair of columns is one 8-byte store
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float v0[2], v1[2];
        unpack2(acc[0][j], v0[0], v0[1]);
        unpack2(acc[1][j], v1[0], v1[1]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float a0 = v0[e], a1 = v1[e];
            if (relu) { a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f); }
            *reinterpret_cast<float2*>(y + (size_t)(cg * 32 + 2 * j + e) * ldy + p0) = make_float2(a0, a1);
        }
    }
}

// ---- global average pool: channel-major in ([C][ld], pixel index n*HW + p), channel-major [C][ldy] out --
// Eight lanes per (channel, image): the HW values are contiguous; the lanes stride over them (all loads issued
// before the adds) and reduce by shuffle.  (A whole warp per pair left most lanes with two loads and five
// shuffle steps for 49 values.)
__global__ void __launch_bounds__(256)
avgpool_cm_kernel(const float* __restrict__ x, int ldx, float* __restrict__ y, int ldy, int N, int HW, int C) {
    grid_dependency_wait();      // the activations come from the previous kernel of the stream
    grid_dependency_release();
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int sub = threadIdx.x & 7;
    const long long pair0 = t >> 3, pairs = (long long)N * C;
    const bool live = pair0 < pairs;
    const long long pair = live ? pair0 : pairs - 1;               // every lane stays for the shuffles
    const int n = (int)(pair % N), c = (int)(pair / N);
    const float* p = x + (size_t)c * ldx + (size_t)n * HW;
    float s = 0.f;
    int i = sub;
    for (; i + 56 < HW; i += 64) {                                 // 8 loads in flight per lane
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldg(p + i + 8 * k);
#pragma unroll
        for (int k = 0; k < 8; ++k) s += v[k];
    }
    {
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = (i + 8 * k < HW) ? __ldg(p + i + 8 * k) : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) s += v[k];
    }
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (live && sub == 0) y[(size_t)c * ldy + n] = s * (1.0f / (float)HW);
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
    if (H != stride * Ho || W != stride * Wo)
        return fail(SBNN_ERR_UNSUPPORTED, "channel-major depthwise needs H and W divisible by the stride");
    if (C > 65535) return fail(SBNN_ERR_SHAPE, "too many channels");
    const long long NHo = (long long)N * Ho;
    if (W % 4 == 0 && Wo % 4 == 0 && ldx % 4 == 0 && ldy % 4 == 0) {
        const long long threads = NHo * (Wo / 4);
        dim3 grid((unsigned)((threads + 255) / 256), C);
        constexpr int RR = 4;
        const long long items = NHo / RR * (W / 4);
        if (stride == 1 && H % RR == 0 && items > 0 && items < 0x7fffffffLL / 2) {
            dim3 gr((unsigned)((items + 127) / 128), C);
            SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_rows_kernel<RR>, gr, 128, 0, st, w, b, x, ldx, y, ldy, (int)items, H, W, relu));
        } else if (stride == 2 && Ho % 2 == 0 && NHo / 2 * (Wo / 4) > 0 && NHo / 2 * (Wo / 4) < 0x7fffffffLL / 2) {
            const long long items2 = NHo / 2 * (Wo / 4);
            dim3 gr((unsigned)((items2 + 127) / 128), C);
            SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_rows_s2_kernel<2>, gr, 128, 0, st, w, b, x, ldx, y, ldy, (int)items2, Ho, W, relu));
        } else if (stride == 1) {
            SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_vec_kernel<1>, grid, 256, 0, st, w, b, x, ldx, y, ldy, NHo, H, W, Ho, Wo, relu));
        } else {
            SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_vec_kernel<2>, grid, 256, 0, st, w, b, x, ldx, y, ldy, NHo, H, W, Ho, Wo, relu));
        }
    } else {
        constexpr int NI = 4;
        const int QB = (Ho * Wo + 255) / 256;
        const int cpb = Ho * Wo < 256 ? 256 / (Ho * Wo) : 1;          // channels per CTA for small planes
        dim3 grid((unsigned)(QB * ((N + NI - 1) / NI)), (C + cpb - 1) / cpb);
#define SBNN_DW_PX(S_, WT_) \
    SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_px_kernel<S_, NI, WT_>, grid, 256, 0, st, w, b, x, ldx, y, ldy, N, H, W, C, QB, relu))
#define SBNN_DW_C7(WT_)                                                                                       \
    {                                                                                                         \
        const int items = (H / 7) * W, qb = (items + 127) / 128;                                              \
        const int cpb7 = items < 128 ? 128 / items : 1;                                                       \
        dim3 g7((unsigned)(qb * ((N + NI - 1) / NI)), (C + cpb7 - 1) / cpb7);                                 \
        SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_col7_kernel<NI, WT_>, g7, 128, 0, st, w, b, x, ldx, y, ldy, N, H, C, relu)); \
    }
        if (stride == 1) {
            if (W == 14 && H == 14 && ldx % 2 == 0 && ldy % 2 == 0) {
                constexpr int NI2 = 2;
                dim3 g14((unsigned)((N + NI2 - 1) / NI2), (C + 7) / 8);
                SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_w14_kernel<NI2>, g14, 128, 0, st, w, b, x, ldx, y, ldy, N, C, relu));
            } else if (W == 14 && H % 7 == 0) SBNN_DW_C7(14)
            else if (W == 7 && H == 7 && ldx % 4 == 0 && ldy % 4 == 0) {
                dim3 g77((unsigned)((N + 63) / 64), (unsigned)((C + 1) / 2));
                SBNN_CUDA_TRY(launch_kernel(dwconv3x3_cm_7x7_kernel, g77, 128, 0, st, w, b, x, ldx, y, ldy, N, C, relu));
            } else if (W == 7 && H % 7 == 0) SBNN_DW_C7(7)
            else SBNN_DW_PX(1, 0);
        } else {
            if (W == 28) SBNN_DW_PX(2, 28);      // stride 2: the per-position kernel measured faster
            else if (W == 14) SBNN_DW_PX(2, 14);
            else SBNN_DW_PX(2, 0);
        }
#undef SBNN_DW_C7
#undef SBNN_DW_PX
    }
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

sbnn_status launch_conv3x3_thin_cm(const float* w, const float* b, const float* x, float* y, int ldy, int N, int H, int W,
                                   int Cin, int Cout, int stride, int relu, cudaStream_t st) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (Cout % 32 == 0 && ldy % 2 == 0) {
        const long long total = (long long)N * Ho * ((Wo + 1) / 2);
        const long long blocks = (total + 127) / 128;
        if (blocks > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "tensor too large");
        dim3 grid((unsigned)blocks, Cout / 32);
        const size_t smem = sizeof(float) * 9 * Cin * 32;
        if (stride == 2 && Cin == 3 && W % 4 == 0 && H % 2 == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
            SBNN_CUDA_TRY(launch_kernel(conv3x3_first_s2c3_kernel, grid, 128, smem, st, w, b, x, y, ldy, N, H, W, Cout, Ho, Wo, relu));
        } else if (stride == 1) {
            SBNN_CUDA_TRY(launch_kernel(conv3x3_thin_cm32_kernel<1>, grid, 128, smem, st, w, b, x, y, ldy, N, H, W, Cin, Cout, Ho, Wo, relu));
        } else {
            SBNN_CUDA_TRY(launch_kernel(conv3x3_thin_cm32_kernel<2>, grid, 128, smem, st, w, b, x, y, ldy, N, H, W, Cin, Cout, Ho, Wo, relu));
        }
        return SBNN_OK;
    }
    return fail(SBNN_ERR_UNSUPPORTED, "channel-major first layer needs Cout %% 32 == 0 and an even leading dimension");
}

sbnn_status launch_avgpool_cm(const float* x, int ldx, float* y, int ldy, int N, int HW, int C, cudaStream_t st) {
    const long long threads = (long long)N * C * 8;
    SBNN_CUDA_TRY(launch_kernel(avgpool_cm_kernel, dim3((unsigned)((threads + 255) / 256)), 256, 0, st, x, ldx, y, ldy, N, HW, C));
    return SBNN_OK;
}

}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_dwconv3x3_cm(const float* w_dev, const float* b_dev, const float* xt_dev, int ldx, float* yt_dev,
                                         int ldy, int N, int H, int W, int C, int stride, int flags, void* cuda_stream) {
    clear_error();
    if (!w_dev || !xt_dev || !yt_dev) return fail(SBNN_ERR_NULL, "w_dev, xt_dev and yt_dev must not be NULL");
    if (N < 0 || H < 0 || W < 0 || C <= 0) return fail(SBNN_ERR_SHAPE, "bad shape N=%d H=%d W=%d C=%d", N, H, W, C);
    if (stride != 1 && stride != 2) return fail(SBNN_ERR_SHAPE, "stride %d: only 1 and 2", stride);
    if (flags & ~SBNN_RELU) return fail(SBNN_ERR_UNSUPPORTED, "unknown flag bits 0x%x", flags);
    if ((long long)N * H * W > 0x7fffffffLL / 2) return fail(SBNN_ERR_SHAPE, "N*H*W too large");
    const int Ho = stride ? (H - 1) / stride + 1 : 0, Wo = stride ? (W - 1) / stride + 1 : 0;
    if (ldx < N * H * W || ldy < N * Ho * Wo || ldx % 4 || ldy % 4)
        return fail(SBNN_ERR_SHAPE, "ldx=%d / ldy=%d must cover the pixels of a channel and be multiples of 4", ldx, ldy);
    if (!aligned16(xt_dev) || !aligned16(yt_dev)) return fail(SBNN_ERR_ALIGN, "xt_dev and yt_dev must be 16-byte aligned");
    if ((long long)N * H * W == 0) return SBNN_OK;
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    return launch_dwconv3x3_cm(w_dev, b_dev, xt_dev, ldx, yt_dev, ldy, N, H, W, C, stride, flags & SBNN_RELU,
                               static_cast<cudaStream_t>(cuda_stream));
}

