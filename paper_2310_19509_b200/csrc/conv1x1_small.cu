// Group-sparse 1x1 convolution for launches with few pixels (Algorithm 1 with the loop nest turned round).
//
// The pipelined kernel of conv1x1_cm.cu deals tiles of 256 pixels x 16-24 groups to the SMs; a layer with a
// few hundred pixels (the classifier, every layer of a batch-1 forward) gives it a handful of tiles, and each
// of them walks all of Cin alone.  Here the work is cut the other way: a CTA owns 32 pixels of ONE group, its
// 1-8 warps (more for longer lists) split the group's kept-unit list and add their partial sums through shared memory.
// Lanes are pixels, so an activation row X[c][m0 .. m0+31] is one coalesced 128-byte read straight from the
// channel-major tensor (it stays in L1/L2 for the other groups' CTAs), and the unit's index and its G weights
// are the same address for the whole warp.  No private weight layout: the canonical packed arrays are read.
#include "common.h"
#include "pipeline.cuh"

namespace sbnn {
namespace {


// Index and weights of unit `u` for lane-parallel fetching: lane l of a warp fetches unit u0 + l (two coalesced
// requests for 32 units), and the warp then hands them round by shuffle, so the only per-unit memory access
// left is the activation row itself and 32 of those are independent.
template <int G>
struct UnitRegs {
    int c;
    float w[G];
};

template <int G>
__device__ __forceinline__ void fetch_unit(const int32_t* __restrict__ idx, const float* __restrict__ val, int u, int uend,
                                           UnitRegs<G>& r) {
    const bool ok = u < uend;
    r.c = ok ? __ldg(idx + u) : 0;
    const float* p = val + (size_t)(ok ? u : 0) * G;
    if constexpr (G % 4 == 0) {
#pragma unroll
        for (int q = 0; q < G / 4; ++q) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(p) + q);
            r.w[4 * q] = t.x; r.w[4 * q + 1] = t.y; r.w[4 * q + 2] = t.z; r.w[4 * q + 3] = t.w;
        }
    } else if constexpr (G == 2) {
        const float2 t = __ldg(reinterpret_cast<const float2*>(p));
        r.w[0] = t.x; r.w[1] = t.y;
    } else {
        r.w[0] = __ldg(p);
    }
    if (!ok) {
#pragma unroll
        for (int q = 0; q < G; ++q) r.w[q] = 0.0f;                 // units past the end multiply pixel row 0 by zero
    }
}

// KSPLIT = warps per CTA; each takes that fraction of the group's kept units.  PX = pixels per lane (the CTA covers
// 32 * PX pixels): with two, a unit's index and weights, which reach the lanes by shuffle, serve twice the FMAs.
template <int G, int KSPLIT, bool OUT_CM, int PX>
__global__ void __launch_bounds__(32 * KSPLIT)
conv1x1_small_kernel(const float* __restrict__ X, int ldx, float* __restrict__ Y, int ldy, const int32_t* __restrict__ group_ptr,
                     const int32_t* __restrict__ idx, const float* __restrict__ val, const float* __restrict__ bias, int M,
                     int relu) {
    __shared__ float red[KSPLIT][G][32 * PX];
    const int lane = threadIdx.x & 31, kq = threadIdx.x >> 5;
    const int g = blockIdx.y;
    int m[PX];
    const float* xp[PX];
#pragma unroll
    for (int j = 0; j < PX; ++j) {
        m[j] = (blockIdx.x * PX + j) * 32 + lane;
        xp[j] = X + (m[j] < M ? m[j] : M - 1);                     // lanes past the end read a valid pixel, store nothing
    }
    const int beg = group_ptr[g], n = group_ptr[g + 1] - beg;
    const int per = (n + KSPLIT - 1) / KSPLIT;
    const int u0 = beg + min(n, kq * per), uend = beg + min(n, (kq + 1) * per);
    float acc[PX][G];
#pragma unroll
    for (int j = 0; j < PX; ++j)
#pragma unroll
        for (int r = 0; r < G; ++r) acc[j][r] = 0.0f;
    UnitRegs<G> cur, nxt;
    fetch_unit<G>(idx, val, u0 + lane, uend, cur);
    grid_dependency_wait();      // X comes from the previous kernel of the stream; the weights above do not
    grid_dependency_release();
    for (int ub = u0; ub < uend; ub += 32) {
        fetch_unit<G>(idx, val, ub + 32 + lane, uend, nxt);        // the next 32 units, while these are consumed
        const int cnt = min(32, uend - ub);                        // warp-uniform
#pragma unroll
        for (int h = 0; h < 2; ++h) {                              // 16 * PX activation loads in flight per lane
            if (h * 16 >= cnt) break;
            float xv[PX][16];
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const int c = __shfl_sync(0xffffffffu, cur.c, h * 16 + k);
#pragma unroll
                for (int j = 0; j < PX; ++j) xv[j][k] = (h * 16 + k < cnt) ? __ldg(xp[j] + (size_t)c * ldx) : 0.0f;
            }
#pragma unroll
            for (int k = 0; k < 16; ++k)
#pragma unroll
                for (int r = 0; r < G; ++r) {
                    const float wr = __shfl_sync(0xffffffffu, cur.w[r], h * 16 + k);
#pragma unroll
                    for (int j = 0; j < PX; ++j) acc[j][r] = fmaf(xv[j][k], wr, acc[j][r]);
                }
        }
        cur = nxt;
    }
#pragma unroll
    for (int j = 0; j < PX; ++j)
#pragma unroll
        for (int r = 0; r < G; ++r) red[kq][r][j * 32 + lane] = acc[j][r];
    __syncthreads();
    if (kq != 0) return;
#pragma unroll
    for (int j = 0; j < PX; ++j) {
        if (m[j] >= M) continue;
        float v[G];
#pragma unroll
        for (int r = 0; r < G; ++r) {
            float s = red[0][r][j * 32 + lane];
#pragma unroll
            for (int q = 1; q < KSPLIT; ++q) s += red[q][r][j * 32 + lane];
            s += __ldg(bias + g * G + r);
            v[r] = relu ? fmaxf(s, 0.0f) : s;
        }
        if constexpr (OUT_CM) {
#pragma unroll
            for (int r = 0; r < G; ++r) Y[(size_t)(g * G + r) * ldy + m[j]] = v[r];
        } else {
            float* yp = Y + (size_t)m[j] * ldy + g * G;
            if constexpr (G >= 4) {
#pragma unroll
                for (int q = 0; q < G / 4; ++q)
                    reinterpret_cast<float4*>(yp)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            } else if constexpr (G == 2) {
                *reinterpret_cast<float2*>(yp) = make_float2(v[0], v[1]);
            } else {
                yp[0] = v[0];
            }
        }
    }
}

template <int G, int KS, int PX>
sbnn_status launch_small_ks(const sbnn_packed* p, const float* x, int ldx, float* y, int ldy, int M, int relu, bool out_cm,
                            cudaStream_t st) {
    dim3 grid((unsigned)((M + 32 * PX - 1) / (32 * PX)), (unsigned)p->ngroups);
    if (out_cm)
        SBNN_CUDA_TRY(launch_kernel(conv1x1_small_kernel<G, KS, true, PX>, grid, 32 * KS, 0, st, x, ldx, y, ldy, p->d_group_ptr, p->d_idx, p->d_val, p->d_bias, M, relu));
    else
        SBNN_CUDA_TRY(launch_kernel(conv1x1_small_kernel<G, KS, false, PX>, grid, 32 * KS, 0, st, x, ldx, y, ldy, p->d_group_ptr, p->d_idx, p->d_val, p->d_bias, M, relu));
    return SBNN_OK;
}

template <int G>
sbnn_status launch_small(const sbnn_packed* p, const float* x, int ldx, float* y, int ldy, int M, int relu, bool out_cm,
                         cudaStream_t st) {
    // Long lists are split over more warps (shorter dependent chains); short ones are not worth the reduction.
    const long long avg = p->ngroups ? p->nnz / p->ngroups : 0;
    if (avg >= 256) {
        // long lists and more than one 32-pixel block: two pixels per lane halve the shuffles per FMA (classifier at
        // batch 64: 18.3 -> 14.9 us inside the step); groups of 16 channels would need 32 more accumulators and stay with one
        if (G <= 8 && M > 32) return launch_small_ks<G, 8, 2>(p, x, ldx, y, ldy, M, relu, out_cm, st);
        return launch_small_ks<G, 8, 1>(p, x, ldx, y, ldy, M, relu, out_cm, st);
    }
    if (avg >= 96) return launch_small_ks<G, 4, 1>(p, x, ldx, y, ldy, M, relu, out_cm, st);
    if (avg >= 40) return launch_small_ks<G, 2, 1>(p, x, ldx, y, ldy, M, relu, out_cm, st);
    return launch_small_ks<G, 1, 1>(p, x, ldx, y, ldy, M, relu, out_cm, st);
}

}  // namespace

sbnn_status conv1x1_small(const sbnn_packed* p, const float* x, int ldx, float* y, int ldy, int M, int relu, bool out_cm,
                          cudaStream_t st) {
    if (p->ngroups > 65535) return fail(SBNN_ERR_SHAPE, "too many groups for the few-pixel kernel");
    if (prepare_only()) return SBNN_OK;   // reads the canonical arrays: nothing to build
    switch (p->G) {
        case 1: return launch_small<1>(p, x, ldx, y, ldy, M, relu, out_cm, st);
        case 2: return launch_small<2>(p, x, ldx, y, ldy, M, relu, out_cm, st);
        case 4: return launch_small<4>(p, x, ldx, y, ldy, M, relu, out_cm, st);
        case 8: return launch_small<8>(p, x, ldx, y, ldy, M, relu, out_cm, st);
        default: return launch_small<16>(p, x, ldx, y, ldy, M, relu, out_cm, st);
    }
}

}  // namespace sbnn
