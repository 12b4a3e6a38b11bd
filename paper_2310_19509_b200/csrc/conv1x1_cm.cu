// Group-sparse 1x1 convolution on channel-major activations, fp32 (Algorithm 1 re-thought for sm_100a).
//
//   Y[m][g*G + r] = act( bias[g*G + r] + sum_j val[g][j][r] * X[idx[g][j]][m] ),   X given as [Cin][ldx]
//
// With the pixels of one input channel contiguous in global memory, the [channel][pixel] shared
// memory tile that the compute warps want is a plain 2-D box of X, so the staging is done by
// the copy engine and costs the SM no instructions:
//   * warp NW (the producer) issues, per channel step, one tiled tensor-map copy of the step's
//     KC x TM box (one copy per channel row was measured to cap staging at a fifth of this rate)
//     and one linear copy of the step's weight block; their bytes complete a "full" mbarrier of the stage;
//   * the NW compute warps wait on "full", run their kept units out of the stage, and each
//     releases it by arriving on the stage's "empty" mbarrier; STAGES stages are in flight, so warps
//     whose groups keep more units in a step are not waited for until STAGES steps later
//     (balanced masks give every group the same total), and no CTA-wide barrier sits in the loop;
//   * every wait has an iteration cap; a wait that expires records SBNN_ERR_TIMEOUT in a device
//     status word, raises the CTA's abort flag, and the CTA drains its copies and returns.
// Compute warps: a lane owns P consecutive-by-4 pixels (LDS.128 along the row) and G x GPW output
// channels, accumulators packed in pairs of pixels and updated with fma.rn.f32x2.
#include <string.h>

#include <limits.h>

#include <algorithm>
#include <initializer_list>

#include <cuda.h>   // CUtensorMap and the encode call's types only; the call itself is looked up at run time

#include "common.h"
#include "pipeline.cuh"

namespace sbnn {
namespace {

// Device status word: 0, or the sbnn_status of the first bounded wait that gave up.
__device__ int g_async_status;

template <int G_, int P_, int GPW_, int NW_, int KC_, int STAGES_>
struct K2 {
    static constexpr int G = G_, P = P_, GPW = GPW_, NW = NW_, KC = KC_, STAGES = STAGES_;
    static constexpr int TM = 32 * P, GT = NW * GPW, NT = (NW + 1) * 32;
    static constexpr int ROW_BYTES = TM * 4;
    static constexpr int XS_BYTES = KC * ROW_BYTES;
    // GPW == 2 selects the union scheme: a warp's two groups share the activation fetch of every
    // channel both keep; its lists are (both, only first, only second).
    static constexpr bool UNION = (GPW == 2);
    static constexpr int NL = UNION ? 3 : GPW;             // lists per warp and step
    static constexpr int HDR = (NW * NL * 2 + 3) / 4;      // 16-byte units
    static constexpr int QUAD = 1 + G;                     // 4 row offsets + 4*G weights
    static constexpr int QUAD2 = 1 + 2 * G;                // the same for a unit that feeds two groups
    static constexpr int NQ = KC / 4 + 1;                  // quads of a full list incl. its all-zero end quad
    // Largest weight block of a step.  Union lists partition the step's KC channels, and a unit kept by both
    // groups is the most expensive, so the worst case is all KC channels in the first list and the other two empty
    // (one all-zero end quad each).
    static constexpr int WS_U4 = UNION ? HDR + NW * (NQ * QUAD2 + 2 * QUAD) : HDR + GT * NQ * QUAD;
    static constexpr int WS_BYTES = WS_U4 * 16;
    static constexpr size_t SMEM = (size_t)STAGES * (XS_BYTES + WS_BYTES) + 2 * STAGES * 8 + 16;
    static_assert(P % 4 == 0 && KC % 4 == 0, "tile shape");
    static_assert(SMEM <= 227 * 1024, "shared memory");
};

template <int G>
__device__ __forceinline__ void unit_weights(const float* wq, int u, float (&w)[G]) {
    if constexpr (G >= 4) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            const float4 t = reinterpret_cast<const float4*>(wq)[u * (G / 4) + v];
            w[4 * v + 0] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
        }
    } else if constexpr (G == 2) {
        const float2 t = reinterpret_cast<const float2*>(wq)[u];
        w[0] = t.x; w[1] = t.y;
    } else {
        w[0] = wq[u];
    }
}

// Runs one list of kept units against the stage: per unit P activations (packed pixel pairs) and
// NG*G weights feed NG groups' accumulators.  Two operand sets alternate, so the loads of the next
// unit are in flight while the FMAs of the current one issue and no register copies are needed.
// (Storing every weight twice, to load it as a ready (w, w) pair, was measured slower: the kernel is
// bound by shared-memory bandwidth.)  A list is followed by zero padding up to and including one
// unit past its end, so the look-ahead never reads garbage.
template <int P, int G, int NG>
__device__ __forceinline__ void run_list(const uint4* r, int n, const unsigned char* xs, f32x2 (&acc0)[P / 2][G],
                                         f32x2 (&acc1)[P / 2][G]) {
    constexpr int QUAD = 1 + NG * G;
    ulonglong2 aA[P / 4], aB[P / 4];
    float wA[NG * G], wB[NG * G];
    auto load_unit = [&](const uint4* quad, unsigned off, int u, ulonglong2 (&a)[P / 4], float (&w)[NG * G]) {
        const unsigned char* ap = xs + off;
#pragma unroll
        for (int i = 0; i < P / 4; ++i) a[i] = *reinterpret_cast<const ulonglong2*>(ap + i * 512);
        unit_weights<NG * G>(reinterpret_cast<const float*>(quad + 1), u, w);
    };
    auto fma_unit = [&](const ulonglong2 (&a)[P / 4], const float (&w)[NG * G]) {
#pragma unroll
        for (int rr = 0; rr < NG * G; ++rr) {
            const f32x2 ww = dup2(w[rr]);
#pragma unroll
            for (int i = 0; i < P / 4; ++i) {
                if (rr < G) {
                    fma2(acc0[2 * i][rr], a[i].x, ww);
                    fma2(acc0[2 * i + 1][rr], a[i].y, ww);
                } else {
                    fma2(acc1[2 * i][rr - G], a[i].x, ww);
                    fma2(acc1[2 * i + 1][rr - G], a[i].y, ww);
                }
            }
        }
    };
    uint4 off = r[0];
    load_unit(r, off.x, 0, aA, wA);
    const int nfull = n >> 2, rem = n & 3;
    for (int it = 0; it < nfull; ++it) {
        const uint4 off_next = r[QUAD];
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        load_unit(r, off.z, 2, aA, wA); fma_unit(aB, wB);
        load_unit(r, off.w, 3, aB, wB); fma_unit(aA, wA);
        load_unit(r + QUAD, off_next.x, 0, aA, wA); fma_unit(aB, wB);
        off = off_next;
        r += QUAD;
    }
    if (rem == 1) {   // last, short quad (warp-uniform)
        fma_unit(aA, wA);
    } else if (rem == 2) {
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        fma_unit(aB, wB);
    } else if (rem == 3) {
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        load_unit(r, off.z, 2, aA, wA); fma_unit(aB, wB);
        fma_unit(aA, wA);
    }
}

// ---- second form of the list loop, for G >= 8 ---------------------------------------------------------------
// The same loop with every shared-memory load written as a volatile instruction on a 32-bit shared address, which
// pins the loads to program order (the order the look-ahead was written in).  Measured: the one-group-per-warp
// G = 8 kernels gain 2-3 % from the pinned order (config 5 at 50 %: 0.594 -> 0.609 of roofline), the union-list
// G = 4 kernels lose about as much, so each keeps its own form.
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ ulonglong2 lds128_pairs(uint32_t addr) {
    ulonglong2 v;
    asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// The G weights of unit u of a quad whose weights start at shared address wq.
template <int G>
__device__ __forceinline__ void unit_weights_v(uint32_t wq, int u, float (&w)[G]) {
    if constexpr (G >= 4) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            const uint4 t = lds128(wq + (u * (G / 4) + v) * 16);
            w[4 * v + 0] = __uint_as_float(t.x); w[4 * v + 1] = __uint_as_float(t.y);
            w[4 * v + 2] = __uint_as_float(t.z); w[4 * v + 3] = __uint_as_float(t.w);
        }
    } else if constexpr (G == 2) {
        const uint2 t = lds64(wq + u * 8);
        w[0] = __uint_as_float(t.x); w[1] = __uint_as_float(t.y);
    } else {
        w[0] = __uint_as_float(lds32(wq + u * 4));
    }
}

// run_list with shared addresses: r = the list's first quad, xs = the lane's first pixels in the stage.
template <int P, int G, int NG>
__device__ __forceinline__ void run_list_v(uint32_t r, int n, uint32_t xs, f32x2 (&acc0)[P / 2][G],
                                           f32x2 (&acc1)[P / 2][G]) {
    constexpr int QUAD = 1 + NG * G;
    ulonglong2 aA[P / 4], aB[P / 4];
    float wA[NG * G], wB[NG * G];
    auto load_unit = [&](uint32_t quad, unsigned off, int u, ulonglong2 (&a)[P / 4], float (&w)[NG * G]) {
#pragma unroll
        for (int i = 0; i < P / 4; ++i) a[i] = lds128_pairs(xs + off + i * 512);
        unit_weights_v<NG * G>(quad + 16, u, w);
    };
    auto fma_unit = [&](const ulonglong2 (&a)[P / 4], const float (&w)[NG * G]) {
#pragma unroll
        for (int rr = 0; rr < NG * G; ++rr) {
            const f32x2 ww = dup2(w[rr]);
#pragma unroll
            for (int i = 0; i < P / 4; ++i) {
                if (rr < G) {
                    fma2(acc0[2 * i][rr], a[i].x, ww);
                    fma2(acc0[2 * i + 1][rr], a[i].y, ww);
                } else {
                    fma2(acc1[2 * i][rr - G], a[i].x, ww);
                    fma2(acc1[2 * i + 1][rr - G], a[i].y, ww);
                }
            }
        }
    };
    uint4 off = lds128(r);
    load_unit(r, off.x, 0, aA, wA);
    const int nfull = n >> 2, rem = n & 3;
    for (int it = 0; it < nfull; ++it) {
        const uint4 off_next = lds128(r + QUAD * 16);
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        load_unit(r, off.z, 2, aA, wA); fma_unit(aB, wB);
        load_unit(r, off.w, 3, aB, wB); fma_unit(aA, wA);
        load_unit(r + QUAD * 16, off_next.x, 0, aA, wA); fma_unit(aB, wB);
        off = off_next;
        r += QUAD * 16;
    }
    if (rem == 1) {   // last, short quad (warp-uniform)
        fma_unit(aA, wA);
    } else if (rem == 2) {
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        fma_unit(aB, wB);
    } else if (rem == 3) {
        load_unit(r, off.y, 1, aB, wB); fma_unit(aA, wA);
        load_unit(r, off.z, 2, aA, wA); fma_unit(aB, wB);
        fma_unit(aA, wA);
    }
}

// The compute warps of the pipelined kernels: wait for a stage ("full": activations [KC][TM] at xs0, weight block at
// ws0), run the warp's lists out of it, release it ("empty"), and write the tile's outputs.  Shared by the plain
// kernel (stages filled by the copy engine) and the fused depthwise + pointwise kernel (activations written by the
// CTA's own depthwise warps).
template <class C, bool OUT_CM>
__device__ __forceinline__ void compute_warps(unsigned char* xs0, unsigned char* ws0, uint64_t* full, uint64_t* empty,
                                              volatile int* abort_flag, float* __restrict__ Y, int ldy,
                                              const float* __restrict__ bias, int M, int ngroups, int nchunks, int ntiles,
                                              int total_tiles, int relu, int* status) {
    constexpr int G = C::G, P = C::P, GPW = C::GPW, S = C::STAGES;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    grid_dependency_wait();       // Y may still be read by the previous kernel of the stream
    grid_dependency_release();
    const unsigned lane_off = lane * 16;
    int consumed = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
    const int tile = t % ntiles, m0 = (t / ntiles) * C::TM;
    f32x2 acc[GPW][P / 2][G];   // acc[q][p2][r]: pixels (2*p2, 2*p2+1) of the lane, channel r of group q
    // The bias is fetched now and added in the epilogue: nothing waits for this global load until then,
    // which matters for layers with few channel steps per tile.
    // (Shapes whose main loop already uses every register fetch it at the start of the epilogue instead.)
    constexpr bool BIAS_EARLY = G * GPW * P < 64 || G < 8;
    float bv[GPW][G];
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + warp * GPW + q;
#pragma unroll
        for (int r = 0; r < G; ++r) {
            if constexpr (BIAS_EARLY) bv[q][r] = (g < ngroups) ? __ldg(bias + g * G + r) : 0.0f;
#pragma unroll
            for (int p = 0; p < P / 2; ++p) acc[q][p][r] = pack2(0.0f, 0.0f);
        }
    }

    bool ok = true;
    for (int k = 0; k < nchunks; ++k, ++consumed) {
        const int s = consumed % S;
        ok = mbar_wait(full + s, (consumed / S) & 1, abort_flag, status, SBNN_ERR_TIMEOUT);
        if (!ok) break;
        if constexpr (G >= 8) {
            const uint32_t xs = smem_u32(xs0) + (uint32_t)s * C::XS_BYTES + lane_off;
            const uint32_t ws = smem_u32(ws0) + (uint32_t)s * C::WS_BYTES;
            const uint32_t hdr = ws + warp * C::NL * 8;             // (start in 16-byte units, kept units) per list
            static_assert(G < 8 || !C::UNION, "the G >= 8 instances have one list per group");
#pragma unroll
            for (int q = 0; q < GPW; ++q) {
                const uint2 hd = lds64(hdr + q * 8);
                run_list_v<P, G, 1>(ws + hd.x * 16, (int)hd.y, xs, acc[q], acc[q]);
            }
        } else {
            const unsigned char* xs = xs0 + (size_t)s * C::XS_BYTES + lane_off;
            const uint4* ws = reinterpret_cast<const uint4*>(ws0 + (size_t)s * C::WS_BYTES);
            const int2* hdr = reinterpret_cast<const int2*>(ws) + warp * C::NL;   // (start, kept units) per list
            if constexpr (C::UNION) {
                const int2 hb = hdr[0], h0 = hdr[1], h1 = hdr[2];
                run_list<P, G, 2>(ws + hb.x, hb.y, xs, acc[0], acc[1]);   // channels both groups keep
                run_list<P, G, 1>(ws + h0.x, h0.y, xs, acc[0], acc[0]);   // only the first group
                run_list<P, G, 1>(ws + h1.x, h1.y, xs, acc[1], acc[1]);   // only the second group
            } else {
#pragma unroll
                for (int q = 0; q < GPW; ++q) {
                    const int2 hd = hdr[q];
                    run_list<P, G, 1>(ws + hd.x, hd.y, xs, acc[q], acc[q]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + s);
    }
    if (!ok) return;

    // epilogue
    if constexpr (!BIAS_EARLY) {
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int g = tile * C::GT + warp * GPW + q;
#pragma unroll
            for (int r = 0; r < G; ++r) bv[q][r] = (g < ngroups) ? __ldg(bias + g * G + r) : 0.0f;
        }
    }
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + warp * GPW + q;
        if (g >= ngroups) continue;
#pragma unroll
        for (int i = 0; i < P / 4; ++i) {
            const int mb = m0 + i * 128 + lane * 4;
            float v[4][G];
#pragma unroll
            for (int rr = 0; rr < G; ++rr) {
                unpack2(acc[q][2 * i][rr], v[0][rr], v[1][rr]);
                unpack2(acc[q][2 * i + 1][rr], v[2][rr], v[3][rr]);
#pragma unroll
                for (int e = 0; e < 4; ++e) v[e][rr] += bv[q][rr];
            }
            if (relu) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int rr = 0; rr < G; ++rr) v[e][rr] = fmaxf(v[e][rr], 0.0f);
            }
            if constexpr (OUT_CM) {
#pragma unroll
                for (int rr = 0; rr < G; ++rr) {
                    float* yp = Y + (size_t)(g * G + rr) * ldy + mb;
                    if (mb + 3 < M) {
                        *reinterpret_cast<float4*>(yp) = make_float4(v[0][rr], v[1][rr], v[2][rr], v[3][rr]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (mb + e < M) yp[e] = v[e][rr];
                    }
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (mb + e >= M) continue;
                    float* yp = Y + (size_t)(mb + e) * ldy + g * G;
                    if constexpr (G >= 4) {
#pragma unroll
                        for (int vv = 0; vv < G / 4; ++vv)
                            reinterpret_cast<float4*>(yp)[vv] =
                                make_float4(v[e][4 * vv], v[e][4 * vv + 1], v[e][4 * vv + 2], v[e][4 * vv + 3]);
                    } else if constexpr (G == 2) {
                        *reinterpret_cast<float2*>(yp) = make_float2(v[e][0], v[e][1]);
                    } else {
                        yp[0] = v[e][0];
                    }
                }
            }
        }
    }
    }   // tiles
}

template <class C, bool OUT_CM>
__global__ void __launch_bounds__(C::NT, 1)
conv1x1_cm_kernel(const __grid_constant__ CUtensorMap xmap, float* __restrict__ Y, int ldy,
                  const float* __restrict__ bias, const uint4* __restrict__ rec,
                  const int32_t* __restrict__ blk_ptr, int M, int Cin, int Cout, int ngroups, int nchunks,
                  int ntiles, int total_tiles, int relu, int* status) {
    constexpr int G = C::G, P = C::P, GPW = C::GPW, NW = C::NW, KC = C::KC, S = C::STAGES;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* xs0 = smem;
    unsigned char* ws0 = smem + (size_t)S * C::XS_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(ws0 + (size_t)S * C::WS_BYTES);
    uint64_t* empty = full + S;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + S);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Persistent CTAs: CTA b works on tiles b, b + gridDim.x, ...  A tile index t = ptile * ntiles + gtile
    // keeps the group tiles of one pixel tile adjacent, so they run at about the same time and the pixel
    // tile's activations come from DRAM once and from L2 afterwards.  Stage and phase counters run on
    // across tiles: the producer is already filling stages for the next tile while the compute warps
    // finish the current one and write its outputs.

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, NW);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == NW) {
        // ---------------- producer warp ----------------
        int issued = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const int tile = t % ntiles, m0 = (t / ntiles) * C::TM;
            const int32_t* bp = blk_ptr + (size_t)tile * (nchunks + 1);
            for (int k = 0; k < nchunks; ++k, ++issued) {
                const int s = issued % S;
                if (issued >= S) ok = mbar_wait(empty + s, ((issued / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT);
                if (!ok) break;
                if (lane == 0) {
                    // a linear copy brings the step's weight block, one tiled copy the step's KC x TM box of X
                    // (pixels past M and channels past Cin arrive as zeros and count towards the bytes).  The
                    // weights do not depend on the previous kernel of the stream, the activations do: the very
                    // first box is requested only once that kernel has finished.
                    const int wbeg = bp[k], wn = bp[k + 1] - wbeg;
                    mbar_arrive_expect_tx(full + s, (uint32_t)C::XS_BYTES + (uint32_t)wn * 16u);
                    bulk_g2s(ws0 + (size_t)s * C::WS_BYTES, rec + wbeg, (uint32_t)wn * 16u, full + s);
                    if (issued == 0) grid_dependency_wait();
                    tensor_g2s_2d(xs0 + (size_t)s * C::XS_BYTES, &xmap, m0, k * KC, full + s);
                }
            }
        }
        if (!ok) {
            // gave up: let the copies already issued land before the CTA's shared memory is released
            for (int k = max(0, issued - S); k < issued; ++k) {
                bool landed = false;
                for (uint32_t i = 0; i < kWaitLimit && !landed; ++i) landed = mbar_try_wait(full + k % S, (k / S) & 1);
            }
        }
        return;
    }

    // ---------------- compute warps ----------------
    compute_warps<C, OUT_CM>(xs0, ws0, full, empty, abort_flag, Y, ldy, bias, M, ngroups, nchunks, ntiles, total_tiles, relu, status);
}

// ---- depthwise 3x3 (stride 1, pad 1) fused into the pointwise kernel -----------------------------------------
// Y = pw( act( dw(X) ) ) without the depthwise output ever going to global memory (Section 3.2 names Conv1x1 and
// DwConv3x3 as the two principal layers; one follows the other in every block of the network).  The CTA is the
// pipelined kernel above plus NDW depthwise warps between the copy engine and the compute warps:
//   * the producer warp copies, per channel step, the RAW input the step's 256 output pixels need: the pixels of a
//     channel are contiguous, so the 3x3 neighbourhood of the run [m0, m0 + TM) lies in the run [m0 - W - 4,
//     m0 + TM + W + 4) of the same plane, fetched as two boxes of KC x bw pixels (a box is at most 256 wide), zeros
//     outside the tensor;
//   * depthwise warp d computes channels d, d + NDW, ... of the step: a lane owns the same 2 x 4 pixels as a compute
//     lane (aligned 16-byte loads of the three rows, the pixels left and right of its four from the neighbouring
//     lanes by shuffle), masks the taps that fall outside the image (a run of four never straddles an image row,
//     because W is a multiple of 4), adds the bias, applies the ReLU and writes the [KC][TM] activation stage that the
//     compute warps read; the step's weight block still arrives by bulk copy on the same "full" barrier.
// Barriers: raw_full / raw_empty between the copy engine and the depthwise warps, x_full (depthwise warps + weight
// bytes) / x_empty between those and the compute warps; all waits bounded as above.
constexpr int NDW = 7;

template <class C>
__global__ void __launch_bounds__(C::NT + NDW * 32, 1)
dwpw_fused_kernel(const __grid_constant__ CUtensorMap rawmap, float* __restrict__ Y, int ldy, const float* __restrict__ bias,
                  const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr, const float* __restrict__ dw_w,
                  const float* __restrict__ dw_b, int M, int Cin, int ngroups, int nchunks, int ntiles, int total_tiles,
                  int H, int W, int bw, int relu_dw, int relu, int* status) {
    constexpr int NW = C::NW, KC = C::KC, S = C::STAGES, RS = 2;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* xs0 = smem;
    unsigned char* ws0 = smem + (size_t)S * C::XS_BYTES;
    unsigned char* raw0 = ws0 + (size_t)S * C::WS_BYTES;
    const uint32_t box_bytes = (uint32_t)KC * bw * 4u, raw_bytes = 2u * box_bytes;
    uint64_t* x_full = reinterpret_cast<uint64_t*>(raw0 + (size_t)RS * raw_bytes);
    uint64_t* x_empty = x_full + S;
    uint64_t* raw_full = x_empty + S;
    uint64_t* raw_empty = raw_full + RS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(raw_empty + RS);
    float* dwsm = reinterpret_cast<float*>(raw_empty + RS) + 4;      // depthwise weights [9][Cin], then the bias [Cin]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < 10 * Cin; i += blockDim.x) dwsm[i] = i < 9 * Cin ? __ldg(dw_w + i) : (dw_b ? __ldg(dw_b + i - 9 * Cin) : 0.0f);
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(x_full + s, 1 + NDW);
            mbar_init(x_empty + s, NW);
        }
        for (int r = 0; r < RS; ++r) {
            mbar_init(raw_full + r, 1);
            mbar_init(raw_empty + r, NDW);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == NW) {
        // ---------------- producer warp ----------------
        int n = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const int tile = t % ntiles, m0 = (t / ntiles) * C::TM;
            const int32_t* bp = blk_ptr + (size_t)tile * (nchunks + 1);
            for (int k = 0; k < nchunks; ++k, ++n) {
                const int r = n % RS, s = n % S;
                if (n >= RS) ok = mbar_wait(raw_empty + r, ((n / RS) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT);
                if (!ok) break;
                if (lane == 0) {
                    unsigned char* dst = raw0 + (size_t)r * raw_bytes;
                    mbar_arrive_expect_tx(raw_full + r, raw_bytes);
                    if (n == 0) grid_dependency_wait();          // X comes from the previous kernel of the stream
                    tensor_g2s_2d(dst, &rawmap, m0 - W - 4, k * KC, raw_full + r);
                    tensor_g2s_2d(dst + box_bytes, &rawmap, m0 - W - 4 + bw, k * KC, raw_full + r);
                }
                if (n >= S) ok = mbar_wait(x_empty + s, ((n / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT);
                if (!ok) { ++n; break; }                         // the raw copies of this step are in flight
                if (lane == 0) {
                    const int wbeg = bp[k], wn = bp[k + 1] - wbeg;
                    mbar_arrive_expect_tx(x_full + s, (uint32_t)wn * 16u);
                    bulk_g2s(ws0 + (size_t)s * C::WS_BYTES, rec + wbeg, (uint32_t)wn * 16u, x_full + s);
                }
            }
        }
        if (!ok) {   // gave up: let the raw copies already issued land before the CTA's shared memory is released
            for (int k = max(0, n - RS); k < n; ++k) {
                bool landed = false;
                for (uint32_t i = 0; i < kWaitLimit && !landed; ++i) landed = mbar_try_wait(raw_full + k % RS, (k / RS) & 1);
            }
        }
        return;
    }

    if (warp > NW) {
        // ---------------- depthwise warps ----------------
        const int d = warp - NW - 1;
        int n = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            const int m0 = (t / ntiles) * C::TM;
            // the lane's two runs of four pixels: position in the image decides which taps exist
            // offA[i][kh]: where the run's row kh starts inside a channel's raw data (element j of a channel row sits in
            // the first box for j < bw, in the second otherwise; bw is a multiple of 4, so a run never straddles them);
            // offL / offR: the pixel left and right of the run (only lanes 0 and 31 fetch those, the others shuffle)
            int offA[2][3], offL[2][3], offR[2][3];
            bool lz[2], rz[2], rowok[2][3];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int p0 = i * 128 + 4 * lane, m = m0 + p0;
                const int x = m % W, y = (m / W) % H;
                lz[i] = x == 0; rz[i] = x == W - 4;
                rowok[i][0] = y > 0; rowok[i][1] = true; rowok[i][2] = y < H - 1;
#pragma unroll
                for (int kh = 0; kh < 3; ++kh) {
                    const int jj = p0 + W + 4 + (kh - 1) * W;     // index of the run's first pixel inside the raw row
                    auto off = [&](int j) { return j < bw ? j : KC * bw + j - bw; };
                    offA[i][kh] = off(jj); offL[i][kh] = off(jj - 1); offR[i][kh] = off(jj + 4);
                }
            }
            for (int k = 0; k < nchunks; ++k, ++n) {
                const int r = n % RS, s = n % S;
                if (!mbar_wait(raw_full + r, (n / RS) & 1, abort_flag, status, SBNN_ERR_TIMEOUT)) return;
                if (n >= S && !mbar_wait(x_empty + s, ((n / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT)) return;
                const float* raw = reinterpret_cast<const float*>(raw0 + (size_t)r * raw_bytes);
                float* xst = reinterpret_cast<float*>(xs0 + (size_t)s * C::XS_BYTES);
                // this warp's channels of the step: d, d + NDW, ... below min(KC, Cin - k*KC); rows past Cin are referenced
                // by no list.  All loads of a channel are issued before its first FMA, two channels are in flight.
                const int nch = min(KC, Cin - k * KC);
                const int mine = nch > d ? (nch - d + NDW - 1) / NDW : 0;
#pragma unroll 2
                for (int u = 0; u < mine; ++u) {
                    const int cl = d + u * NDW, c = k * KC + cl;
                    const float* rc = raw + cl * bw;
                    float4 A[2][3];
                    float Le[2][3], Re[2][3];
#pragma unroll
                    for (int i = 0; i < 2; ++i)
#pragma unroll
                        for (int kh = 0; kh < 3; ++kh) {
                            const bool ok = rowok[i][kh];
                            A[i][kh] = ok ? *reinterpret_cast<const float4*>(rc + offA[i][kh]) : make_float4(0.f, 0.f, 0.f, 0.f);
                            Le[i][kh] = (lane == 0 && ok && !lz[i]) ? rc[offL[i][kh]] : 0.0f;
                            Re[i][kh] = (lane == 31 && ok && !rz[i]) ? rc[offR[i][kh]] : 0.0f;
                        }
                    float wk[9];
#pragma unroll
                    for (int q = 0; q < 9; ++q) wk[q] = dwsm[q * Cin + c];
                    const float b = dwsm[9 * Cin + c];
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        float acc[4] = {b, b, b, b};
#pragma unroll
                        for (int kh = 0; kh < 3; ++kh) {
                            float L = __shfl_up_sync(0xffffffffu, A[i][kh].w, 1), R = __shfl_down_sync(0xffffffffu, A[i][kh].x, 1);
                            if (lane == 0) L = Le[i][kh];
                            if (lane == 31) R = Re[i][kh];
                            if (lz[i]) L = 0.0f;                  // (a row that does not exist was loaded as zeros)
                            if (rz[i]) R = 0.0f;
                            const float in[6] = {L, A[i][kh].x, A[i][kh].y, A[i][kh].z, A[i][kh].w, R};
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                acc[e] = fmaf(in[e + 2], wk[kh * 3 + 2], fmaf(in[e + 1], wk[kh * 3 + 1], fmaf(in[e], wk[kh * 3], acc[e])));
                        }
                        float4 o = make_float4(acc[0], acc[1], acc[2], acc[3]);
                        if (relu_dw) o = make_float4(fmaxf(o.x, 0.f), fmaxf(o.y, 0.f), fmaxf(o.z, 0.f), fmaxf(o.w, 0.f));
                        *reinterpret_cast<float4*>(xst + cl * C::TM + i * 128 + 4 * lane) = o;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(x_full + s);                      // this warp's channels of the stage are written
                    mbar_arrive(raw_empty + r);                   // and it is done with the raw rows
                }
            }
        }
        return;
    }

    // ---------------- compute warps ----------------
    compute_warps<C, true>(xs0, ws0, x_full, x_empty, abort_flag, Y, ldy, bias, M, ngroups, nchunks, ntiles, total_tiles, relu, status);
}

// Diagnostic: one warp waits, with a short cap, on an mbarrier that nothing ever completes.  Exercises the
// path a stalled pipeline takes (status word set, kernel returns normally) without any fault.
__global__ void wait_timeout_selftest_kernel(int* status, uint32_t limit) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_flag, status, SBNN_ERR_TIMEOUT, limit);
}

// X [M][C] (row-major, C contiguous) -> Xt [C][ld]: 32 x 32 tiles through padded shared memory.
__global__ void __launch_bounds__(256)
to_channel_major_kernel(const float* __restrict__ x, float* __restrict__ xt, int M, int C, int ld) {
    __shared__ float t[32][33];
    const int m0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i, c = c0 + tx;
        if (m < M && c < C) t[ty + 8 * i][tx] = x[(size_t)m * C + c];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, m = m0 + tx;
        if (m < M && c < C) xt[(size_t)c * ld + m] = t[tx][ty + 8 * i];
    }
}

// ---- host side -------------------------------------------------------------------------------

// Record stream for one tile shape.  Block (tile t, step k) = header of (start, kept units) per list,
// then the lists.  A list is a run of quads (4 byte offsets of the units' shared-memory rows, then the
// weights of the 4 units); it always ends with zero padding (offset 0, weight 0) up to and including
// one unit past its end, because the kernel fetches the operands of the next unit before it knows the
// list is over.  Plain layout: one list per group.  Union layout (GPW == 2): per warp the channels kept
// by both of its groups (2*G weights per unit), then those kept only by the first, only by the second.
sbnn_status build_stream_cm(const sbnn_packed* p, const TileCfg& c, Stream1x1* out) {
    const int G = p->G, GT = c.GT(), KC = c.KC, TM = c.TM();
    const bool un = (c.GPW == 2);
    const int NL = un ? 3 : c.GPW;
    const int ntiles = (p->ngroups + GT - 1) / GT, nchunks = (p->Cin + KC - 1) / KC;
    const int HDR = (c.NW * NL * 2 + 3) / 4;
    std::vector<int32_t> blk((size_t)ntiles * (nchunks + 1));
    std::vector<uint32_t> rec;
    int max_blk = 0;
    // one kept unit of a list: position in the canonical arrays for each group it feeds (-1: none)
    struct Unit { int c; int64_t j0, j1; };
    std::vector<Unit> lists[3];
    try {
        rec.reserve(((size_t)p->nnz / 4 + (size_t)ntiles * nchunks * (2 * GT + HDR)) * (1 + G) * 4);
        auto emit = [&](size_t blk_beg, int slot, const std::vector<Unit>& L, int ng, int k) {
            const int QUAD = 1 + ng * G;
            const int n = (int)L.size(), nq = n / 4 + 1;
            rec[blk_beg * 4 + 2 * slot + 0] = (uint32_t)(rec.size() / 4 - blk_beg);
            rec[blk_beg * 4 + 2 * slot + 1] = (uint32_t)n;
            for (int qd = 0; qd < nq; ++qd) {
                const size_t base = rec.size();
                rec.resize(base + (size_t)QUAD * 4, 0u);
                for (int u = 0; u < 4; ++u) {
                    const int i = qd * 4 + u;
                    if (i >= n) break;
                    rec[base + u] = (uint32_t)(L[i].c - k * KC) * (uint32_t)(TM * 4);
                    memcpy(&rec[base + 4 + u * ng * G], &p->val[(size_t)L[i].j0 * G], sizeof(float) * G);
                    if (ng == 2) memcpy(&rec[base + 4 + u * ng * G + G], &p->val[(size_t)L[i].j1 * G], sizeof(float) * G);
                }
            }
        };
        auto range = [&](int g, int k, int64_t* lo, int64_t* hi) {
            *lo = *hi = 0;
            if (g >= p->ngroups) return;
            const int32_t* b = p->idx.data() + p->group_ptr[g];
            const int32_t* e = p->idx.data() + p->group_ptr[g + 1];
            *lo = std::lower_bound(b, e, k * KC) - p->idx.data();
            *hi = std::lower_bound(b, e, (k + 1) * KC) - p->idx.data();
        };
        for (int t = 0; t < ntiles; ++t) {
            for (int k = 0; k < nchunks; ++k) {
                const size_t blk_beg = rec.size() / 4;
                blk[(size_t)t * (nchunks + 1) + k] = (int32_t)blk_beg;
                rec.resize(rec.size() + (size_t)HDR * 4, 0u);
                if (!un) {
                    for (int s = 0; s < GT; ++s) {
                        int64_t lo, hi;
                        range(t * GT + s, k, &lo, &hi);
                        lists[0].clear();
                        for (int64_t j = lo; j < hi; ++j) lists[0].push_back({p->idx[j], j, -1});
                        emit(blk_beg, s, lists[0], 1, k);
                    }
                } else {
                    for (int w = 0; w < c.NW; ++w) {
                        int64_t lo0, hi0, lo1, hi1;
                        range(t * GT + 2 * w, k, &lo0, &hi0);
                        range(t * GT + 2 * w + 1, k, &lo1, &hi1);
                        for (auto& L : lists) L.clear();
                        int64_t i0 = lo0, i1 = lo1;   // merge the two ascending index lists
                        while (i0 < hi0 || i1 < hi1) {
                            const int c0 = i0 < hi0 ? p->idx[i0] : INT_MAX, c1 = i1 < hi1 ? p->idx[i1] : INT_MAX;
                            if (c0 == c1) { lists[0].push_back({c0, i0, i1}); ++i0; ++i1; }
                            else if (c0 < c1) { lists[1].push_back({c0, i0, -1}); ++i0; }
                            else { lists[2].push_back({c1, i1, -1}); ++i1; }
                        }
                        emit(blk_beg, 3 * w + 0, lists[0], 2, k);
                        emit(blk_beg, 3 * w + 1, lists[1], 1, k);
                        emit(blk_beg, 3 * w + 2, lists[2], 1, k);
                    }
                }
                max_blk = std::max(max_blk, (int)(rec.size() / 4 - blk_beg));
            }
            blk[(size_t)t * (nchunks + 1) + nchunks] = (int32_t)(rec.size() / 4);
        }
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the channel-major weight stream");
    }
    if (rec.size() / 4 > 0x7fffffffull) return fail(SBNN_ERR_UNSUPPORTED, "weight stream too large");
    Stream1x1 s;
    s.ntiles = ntiles; s.nchunks = nchunks; s.max_blk = max_blk;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s.rec), std::max<size_t>(rec.size() * 4, 16)));
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&s.blk_ptr), blk.size() * 4);
    if (e == cudaSuccess && !rec.empty()) e = cudaMemcpy(s.rec, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s.blk_ptr, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        cudaFree(s.blk_ptr);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the channel-major weight stream: %s", cudaGetErrorString(e));
    }
    *out = s;
    return SBNN_OK;
}

sbnn_status get_stream_cm(const sbnn_packed* p, const TileCfg& c, Stream1x1* out) {
    std::lock_guard<std::mutex> lk(p->mu);
    auto it = p->streams_cm.find(c);
    if (it != p->streams_cm.end()) {
        *out = it->second;
        return SBNN_OK;
    }
    sbnn_status st = build_stream_cm(p, c, out);
    if (st == SBNN_OK) p->streams_cm[c] = *out;
    return st;
}

// Address of the device status word on the current device.
sbnn_status status_word(int** out) {
    static std::mutex mu;
    static std::map<int, int*> addr;
    int dev = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    auto it = addr.find(dev);
    if (it == addr.end()) {
        int* p = nullptr;
        SBNN_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_async_status));
        it = addr.emplace(dev, p).first;
    }
    *out = it->second;
    return SBNN_OK;
}

// Number of SMs of the current device (one persistent CTA each).
int sm_count() {
    static std::mutex mu;
    static std::map<int, int> n;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lk(mu);
    auto it = n.find(dev);
    if (it == n.end()) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        it = n.emplace(dev, v).first;
    }
    return it->second;
}

// Tensor map of the channel-major activations X [Cin][ldx] (M valid pixels per row), copied in boxes of
// `box_rows` channels x `box_px` pixels.  The driver's encode routine is looked up once per process.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
sbnn_status get_encode(EncodeTiledFn* out) {
    static std::mutex mu;
    static EncodeTiledFn encode = nullptr;
    std::lock_guard<std::mutex> lk(mu);
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        SBNN_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) return fail(SBNN_ERR_CUDA, "driver has no cuTensorMapEncodeTiled");
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = encode;
    return SBNN_OK;
}

// fp32 (elem_bytes 4) or bf16 (2) tensor of `rank` dimensions (innermost first), tiled copies of `box` elements,
// zeros outside the tensor.
sbnn_status encode_generic(void* out, const void* base, int elem_bytes, int rank, const unsigned long long* dims,
                           const unsigned long long* strides_bytes, const unsigned* box, bool swizzle128 = false) {
    EncodeTiledFn encode = nullptr;
    sbnn_status r = get_encode(&encode);
    if (r != SBNN_OK) return r;
    if (!aligned16(base)) return fail(SBNN_ERR_ALIGN, "tensor base must be 16-byte aligned");
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; ++i) {
        d[i] = dims[i];
        b[i] = box[i];
        es[i] = 1;
        if (i + 1 < rank) {
            st[i] = strides_bytes[i];
            if (st[i] % 16) return fail(SBNN_ERR_ALIGN, "tensor stride %llu is not a multiple of 16 bytes", (unsigned long long)st[i]);
        }
    }
    const CUresult cr = encode(static_cast<CUtensorMap*>(out),
                               elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                               (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(SBNN_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)cr);
    return SBNN_OK;
}

sbnn_status encode_x_map(const float* x, int ldx, int M, int Cin, int box_px, int box_rows, CUtensorMap* out) {
    if (ldx % 4) return fail(SBNN_ERR_ALIGN, "channel-major activations need ld %% 4 == 0");
    const unsigned long long dims[2] = {(unsigned long long)M, (unsigned long long)Cin};
    const unsigned long long strides[1] = {(unsigned long long)ldx * sizeof(float)};
    const unsigned box[2] = {(unsigned)box_px, (unsigned)box_rows};
    return encode_generic(out, x, 4, 2, dims, strides, box);
}

template <class C>
sbnn_status launch_cm(const sbnn_packed* p, const Stream1x1& s, const float* x, int ldx, float* y, int ldy, int M,
                      int relu, bool out_cm, cudaStream_t st) {
    sbnn_status r = set_max_dyn_smem(reinterpret_cast<const void*>(&conv1x1_cm_kernel<C, false>), (int)C::SMEM);
    if (r == SBNN_OK) r = set_max_dyn_smem(reinterpret_cast<const void*>(&conv1x1_cm_kernel<C, true>), (int)C::SMEM);
    if (r != SBNN_OK) return r;
    if (s.max_blk > C::WS_U4) return fail(SBNN_ERR_UNSUPPORTED, "internal: weight block %d exceeds buffer %d", s.max_blk, C::WS_U4);
    int* status = nullptr;
    if ((r = status_word(&status)) != SBNN_OK) return r;
    if (prepare_only()) return SBNN_OK;
    const long long nblk = (long long)((M + C::TM - 1) / C::TM) * s.ntiles;
    if (nblk > 0x7fffffffLL) return fail(SBNN_ERR_SHAPE, "too many tiles");
    const int total_tiles = (int)nblk;
    dim3 grid((unsigned)std::min<long long>(nblk, sm_count()));
    CUtensorMap xmap;
    r = encode_x_map(x, ldx, M, p->Cin, C::TM, C::KC, &xmap);
    if (r != SBNN_OK) return r;
    if (out_cm)
        SBNN_CUDA_TRY(launch_kernel(conv1x1_cm_kernel<C, true>, grid, C::NT, C::SMEM, st, xmap, y, ldy, p->d_bias, s.rec, s.blk_ptr, M,
                                    p->Cin, p->Cout, p->ngroups, s.nchunks, s.ntiles, total_tiles, relu, status));
    else
        SBNN_CUDA_TRY(launch_kernel(conv1x1_cm_kernel<C, false>, grid, C::NT, C::SMEM, st, xmap, y, ldy, p->d_bias, s.rec, s.blk_ptr, M,
                                    p->Cin, p->Cout, p->ngroups, s.nchunks, s.ntiles, total_tiles, relu, status));
    return SBNN_OK;
}

// Fused depthwise + pointwise launch (G = 4 layers, union lists, 8 warps, 32-channel steps, two stages).
using FusedCfg = K2<4, 8, 2, 8, 32, 2>;

sbnn_status launch_dwpw(const sbnn_packed* p, const float* dw_w, const float* dw_b, const float* x, int ldx, float* y, int ldy,
                        int N, int H, int W, int relu_dw, int relu, cudaStream_t st, bool* done) {
    using C = FusedCfg;
    *done = false;
    const long long M = (long long)N * H * W;
    // the raw rows of a step: TM + 2W + 5 pixels, rounded up to two boxes of bw (a multiple of 4, at most 256)
    const int bw = ((C::TM + 2 * W + 5 + 1) / 2 + 3) / 4 * 4;
    const size_t smem = (size_t)C::STAGES * (C::XS_BYTES + C::WS_BYTES) + (size_t)2 * 2 * C::KC * bw * 4 + 128 + (size_t)10 * p->Cin * 4;
    if (p->G != 4 || W % 4 || bw > 256 || smem > 227 * 1024 || M > 0x7fffffffLL - 1024) return SBNN_OK;
    const TileCfg cfg{C::P, C::GPW, C::NW, C::KC};
    Stream1x1 s;
    sbnn_status r = get_stream_cm(p, cfg, &s);
    if (r != SBNN_OK) return r;
    if ((r = set_max_dyn_smem(reinterpret_cast<const void*>(&dwpw_fused_kernel<C>), 227 * 1024)) != SBNN_OK) return r;
    if (s.max_blk > C::WS_U4) return fail(SBNN_ERR_UNSUPPORTED, "internal: weight block %d exceeds buffer %d", s.max_blk, C::WS_U4);
    int* status = nullptr;
    if ((r = status_word(&status)) != SBNN_OK) return r;
    *done = true;
    if (prepare_only()) return SBNN_OK;
    const long long nblk = ((M + C::TM - 1) / C::TM) * s.ntiles;
    if (nblk > 0x7fffffffLL) return fail(SBNN_ERR_SHAPE, "too many tiles");
    CUtensorMap rawmap;
    if ((r = encode_x_map(x, ldx, (int)M, p->Cin, bw, C::KC, &rawmap)) != SBNN_OK) return r;
    dim3 grid((unsigned)std::min<long long>(nblk, sm_count()));
    SBNN_CUDA_TRY(launch_kernel(dwpw_fused_kernel<C>, grid, C::NT + NDW * 32, smem, st, rawmap, y, ldy, p->d_bias, s.rec, s.blk_ptr, dw_w,
                                dw_b, (int)M, p->Cin, p->ngroups, s.nchunks, s.ntiles, (int)nblk, H, W, bw, relu_dw, relu, status));
    return SBNN_OK;
}

// Instantiated shapes: (G, P, GPW, NW, KC, STAGES).
#define SBNN_K2_CONFIGS(X) \
    X(1, 8, 4, 8, 32, 4)   \
    X(2, 8, 2, 8, 32, 4)   \
    X(4, 8, 1, 16, 32, 4)  \
    X(4, 8, 2, 8, 32, 4)   \
    X(4, 8, 2, 11, 32, 3)  \
    X(4, 8, 2, 12, 32, 3)  \
    X(4, 8, 2, 8, 64, 2)   \
    X(4, 8, 2, 11, 64, 2)  \
    X(4, 8, 2, 12, 64, 2)  \
    X(4, 8, 1, 16, 64, 2)  \
    X(8, 8, 1, 8, 64, 2)   \
    X(8, 8, 1, 12, 64, 2)  \
    X(4, 4, 1, 8, 32, 4)   \
    X(8, 8, 1, 8, 32, 4)   \
    X(8, 8, 1, 12, 32, 3)  \
    X(8, 4, 1, 16, 32, 4)  \
    X(16, 4, 1, 8, 32, 4)

sbnn_status dispatch_cm(const sbnn_packed* p, const TileCfg& c, const float* x, int ldx, float* y, int ldy, int M,
                        int relu, bool out_cm, cudaStream_t st) {
    Stream1x1 s;
#define SBNN_TRY(g, pp, gpw, nw, kc, stg)                                                        \
    if (p->G == g && c.P == pp && c.GPW == gpw && c.NW == nw && c.KC == kc) {                    \
        sbnn_status r = get_stream_cm(p, c, &s);                                                 \
        if (r != SBNN_OK) return r;                                                              \
        return launch_cm<K2<g, pp, gpw, nw, kc, stg>>(p, s, x, ldx, y, ldy, M, relu, out_cm, st); \
    }
    SBNN_K2_CONFIGS(SBNN_TRY)
#undef SBNN_TRY
    return fail(SBNN_ERR_UNSUPPORTED, "no channel-major 1x1 kernel instance for G=%d P=%d GPW=%d NW=%d KC=%d", p->G,
                c.P, c.GPW, c.NW, c.KC);
}

// Tile shape for a layer run on M pixels.  M <= 0 stands for "many pixels" (the choice made before M is known).
TileCfg choose_cfg_cm(const sbnn_packed* p, long long M);

// The choice is made once per (layer, pixel count) and remembered: computing it walks the layer's tiles.
TileCfg default_cfg_cm(const sbnn_packed* p, long long M) {
    if (M <= 0) return choose_cfg_cm(p, M);
    std::lock_guard<std::mutex> lk(p->mu);
    auto it = p->cfg_cm.find(M);
    if (it != p->cfg_cm.end()) return it->second;
    if (p->cfg_cm.size() > 64) p->cfg_cm.clear();
    const TileCfg c = choose_cfg_cm(p, M);
    p->cfg_cm[M] = c;
    return c;
}

TileCfg choose_cfg_cm(const sbnn_packed* p, long long M) {
    // Whole tiles are dealt to the persistent CTAs (CTA b takes tiles b, b + SMs, ...), and inside a CTA warp w runs
    // on scheduler w % 4, so a tile lasts as long as the scheduler with the most busy warps, and the launch as long as
    // the CTA with the most work.  The cost of a tile shape is that maximum, computed exactly from the layer's group
    // count (warps of a ragged last group tile are idle).  Measured on the 1024 -> 1024 layer with 64-channel steps:
    // 8 warps (2 per scheduler) 1034 us, 12 warps (3 per scheduler) 1039 us, 11 warps 1109 us -- eleven warps cost as
    // much per tile as twelve; three warps on a scheduler hide about 2 % more latency than two.
    // What a third warp on a scheduler hides of the per-list latencies grows as the lists get shorter: config 5,
    // 12 against 8 warps (whole launch, so including the 4 % of the 12-warp CTA): 50 % kept units 1033 / 1025 us,
    // 30 % kept 670 / 684 us, 10 % kept 313 / 352 us.
    const double kept = (p->ngroups > 0 && p->Cin > 0) ? (double)p->nnz / ((double)p->ngroups * p->Cin) : 1.0;
    const double hide3 = kept >= 0.5 ? 0.02 : (kept >= 0.3 ? 0.02 + 0.2 * (0.5 - kept) : 0.06 + 0.35 * (0.3 - kept));
    auto launch_cost = [&](const TileCfg& c) {
        const long long ptiles = (M + c.TM() - 1) / c.TM(), gtiles = (p->ngroups + c.GT() - 1) / c.GT();
        const long long sms = std::max(1, sm_count()), total = ptiles * gtiles;
        auto tile_cost = [&](long long gtile) {
            int load[4] = {0, 0, 0, 0};
            for (int w = 0; w < c.NW; ++w)
                if ((gtile * c.NW + w) * c.GPW < p->ngroups) ++load[w & 3];
            const int m = std::max(std::max(load[0], load[1]), std::max(load[2], load[3]));
            // (with the producer a 12-warp CTA has 13 warps, which the register file serves like 16: 128 registers a
            // thread instead of the 154 the loop wants, measured 4-6 % slower per tile than the 11-warp CTA)
            return (m >= 3 ? (1.0 - hide3) * m : (double)m) * (c.NW == 12 ? 1.04 : 1.0);
        };
        double full_tile = 0.0;                      // cost of one pass over the group tiles of a pixel tile
        for (long long g = 0; g < gtiles; ++g) full_tile += tile_cost(g);
        if (total > 64 * sms) return (double)total / sms * full_tile / gtiles;   // many rounds: the average is exact enough
        double worst = 0.0;
        for (long long b = 0; b < std::min(sms, total); ++b) {
            double sum = 0.0;
            for (long long t = b; t < total; t += sms) sum += tile_cost(t % gtiles);
            worst = std::max(worst, sum);
        }
        return worst;
    };
    auto pick = [&](const TileCfg& base, std::initializer_list<TileCfg> others) {
        if (M <= 0) return base;
        TileCfg best = base;
        double best_cost = 0.99 * launch_cost(base);
        for (const TileCfg& c : others) {
            const double cost = launch_cost(c);
            if (cost < best_cost) {
                best = c;
                best_cost = cost;
            }
        }
        return best;
    };
    // Channels per pipeline step: 64 (two stages) wherever the layer has that many.  A warp's lists are per step, and
    // every list costs a pipeline fill and drain, so longer steps are cheaper (config 5, G = 4, 50 %: 0.63 -> 0.68 of
    // the roofline; 70 %: 0.55 -> 0.62); thin layers (Cin < 64) keep 32 so that no stage is half zeros.
    const int kc = p->Cin >= 64 ? 64 : 32;
    switch (p->G) {
        case 1: return {8, 4, 8, 32};
        case 2: return {8, 2, 8, 32};
        case 4:
            // Two groups per warp with union lists at every density: with 64-channel steps they also beat one group
            // per warp on twice the warps for sparse layers (config 5 at 70 / 90 %: 0.63 / 0.45 against 0.61 / 0.42).
            return pick({8, 2, 8, kc}, {{8, 2, 11, kc}, {8, 2, 12, kc}});
        case 8: return pick({8, 1, 8, kc}, {{8, 1, 12, kc}});
        default: return {4, 1, 8, 32};
    }
}

// True when the pipelined kernel would get fewer tiles than half the SMs: such launches go to the few-pixel kernel.
bool few_tiles(const sbnn_packed* p, long long M) {
    const TileCfg c = default_cfg_cm(p, 0);
    const long long tiles = ((M + c.TM() - 1) / c.TM()) * ((p->ngroups + c.GT() - 1) / c.GT());
    return 2 * tiles < sm_count();
}

// Per-device scratch for the channel-major copy of X made on behalf of NHWC callers.  Grows on demand with a
// synchronous cudaMalloc; the outgrown buffer is parked, not freed, until the process exits: launches already
// enqueued on it, and CUDA graphs a caller recorded over an entry point that uses it, keep reading valid memory.
// (sbnn_prepare sizes it ahead of time, after which compute calls of no larger shape never get here to grow it.)
struct Workspace {
    float* ptr = nullptr;
    size_t bytes = 0;
    std::vector<float*> parked;
};
sbnn_status workspace(size_t bytes, cudaStream_t st, float** out) {
    static std::mutex mu;
    static std::map<int, Workspace> ws;
    int dev = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    Workspace& w = ws[dev];
    if (w.bytes < bytes) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (!prepare_only() && cudaStreamIsCapturing(st, &cs) != cudaSuccess) cudaGetLastError();
        if (cs != cudaStreamCaptureStatusNone)
            return fail(SBNN_ERR_UNSUPPORTED, "the scratch buffer must grow to %zu bytes, which cannot happen while the stream is "
                        "being captured: call sbnn_prepare (or this entry point once) for this shape before capturing", bytes);
        float* fresh = nullptr;
        SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&fresh), bytes));
        if (w.ptr) w.parked.push_back(w.ptr);
        w.ptr = fresh;
        w.bytes = bytes;
    }
    *out = w.ptr;
    return SBNN_OK;
}

}  // namespace

sbnn_status scratch_workspace(size_t bytes, cudaStream_t st, float** out) { return workspace(bytes, st, out); }

sbnn_status async_status_word(int** out) { return status_word(out); }

sbnn_status dwconv3x3_conv1x1_fused_cm(const sbnn_packed* pw, const float* dw_w, const float* dw_b, const float* x, int ldx, float* y,
                                       int ldy, int N, int H, int W, int relu_dw, int relu, cudaStream_t st, bool* done) {
    return launch_dwpw(pw, dw_w, dw_b, x, ldx, y, ldy, N, H, W, relu_dw, relu, st, done);
}

sbnn_status encode_tiled_map(void* out, const void* base, int elem_bytes, int rank, const unsigned long long* dims,
                             const unsigned long long* strides_bytes, const unsigned* box, bool swizzle128) {
    if (swizzle128 && (size_t)box[0] * elem_bytes > 128) return fail(SBNN_ERR_SHAPE, "a swizzled box row is at most 128 bytes");
    return encode_generic(out, base, elem_bytes, rank, dims, strides_bytes, box, swizzle128);
}

sbnn_status prepare_default_cm(const sbnn_packed* p, long long M) {
    Stream1x1 s;
    return get_stream_cm(p, default_cfg_cm(p, M), &s);
}

sbnn_status prepare_all_cm(const sbnn_packed* p) {
    // every tile shape default_cfg_cm can return for this layer's G and density
    std::vector<TileCfg> all;
    switch (p->G) {
        case 1: all = {{8, 4, 8, 32}}; break;
        case 2: all = {{8, 2, 8, 32}}; break;
        case 4: all = {{8, 2, 8, 32}, {8, 2, 11, 32}, {8, 2, 12, 32}, {8, 2, 8, 64}, {8, 2, 11, 64}, {8, 2, 12, 64}}; break;
        case 8: all = {{8, 1, 8, 32}, {8, 1, 12, 32}, {8, 1, 8, 64}, {8, 1, 12, 64}}; break;
        default: all = {{4, 1, 8, 32}}; break;
    }
    PrepareScope scope;   // dispatch_cm then builds the stream and sets the kernel's attributes, and launches nothing
    for (const TileCfg& c : all) {
        sbnn_status r = dispatch_cm(p, c, nullptr, 0, nullptr, 0, 1, 0, false, nullptr);
        if (r != SBNN_OK) return r;
    }
    return SBNN_OK;
}

sbnn_status prepare_cm(const sbnn_packed* p, int P, int GPW, int NW, int KC) {
    Stream1x1 s;
    return get_stream_cm(p, TileCfg{P, GPW, NW, KC}, &s);
}

void free_streams_cm(sbnn_packed* p) {
    for (auto& kv : p->streams_cm) {
        cudaFree(kv.second.rec);
        cudaFree(kv.second.blk_ptr);
    }
    p->streams_cm.clear();
}

sbnn_status read_async_status(int* value) {
    int* w = nullptr;
    sbnn_status r = status_word(&w);
    if (r != SBNN_OK) return r;
    SBNN_CUDA_TRY(cudaMemcpy(value, w, sizeof(int), cudaMemcpyDeviceToHost));
    if (*value) SBNN_CUDA_TRY(cudaMemset(w, 0, sizeof(int)));
    return SBNN_OK;
}

sbnn_status conv1x1_via_cm(const sbnn_packed* w, const float* x, float* y, int M, int relu, cudaStream_t st, bool* done) {
    *done = false;
    // worth the extra transposition pass only where the layer is bound by arithmetic
    if (w->Cin < 128 || w->Cout < 64 || M < 2048) return SBNN_OK;
    const int ld = (M + 3) / 4 * 4;
    float* xt = nullptr;
    sbnn_status r = workspace((size_t)w->Cin * ld * sizeof(float), st, &xt);
    if (r != SBNN_OK) return r;
    if (!prepare_only()) {
        dim3 grid((M + 31) / 32, (w->Cin + 31) / 32);
        to_channel_major_kernel<<<grid, 256, 0, st>>>(x, xt, M, w->Cin, ld);
        SBNN_CUDA_TRY(cudaGetLastError());
    }
    r = dispatch_cm(w, default_cfg_cm(w, M), xt, ld, y, w->Cout, M, relu, false, st);
    if (r == SBNN_OK) *done = true;
    return r;
}

}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_selftest_wait_timeout(void* cuda_stream) {
    clear_error();
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    int* status = nullptr;
    if ((st = status_word(&status)) != SBNN_OK) return st;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status, 2000u);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_to_channel_major(const float* x_dev, float* xt_dev, int M, int C, int ld, void* cuda_stream) {
    clear_error();
    if (!x_dev || !xt_dev) return fail(SBNN_ERR_NULL, "x_dev and xt_dev must not be NULL");
    if (M < 0 || C <= 0 || ld < M || ld % 4) return fail(SBNN_ERR_SHAPE, "bad shape M=%d C=%d ld=%d (ld >= M, ld %% 4 == 0)", M, C, ld);
    if (M == 0) return SBNN_OK;
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    dim3 grid((M + 31) / 32, (C + 31) / 32);
    if (grid.y > 65535) return fail(SBNN_ERR_SHAPE, "C too large");
    to_channel_major_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(x_dev, xt_dev, M, C, ld);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_conv1x1_gs_cm(const sbnn_packed* w, const float* xt_dev, int ldx, float* y_dev, int ldy, int M,
                                          int flags, int P, int GPW, int NW, int KC, void* cuda_stream) {
    clear_error();
    if (!w || !xt_dev || !y_dev) return fail(SBNN_ERR_NULL, "packed weights, xt_dev and y_dev must not be NULL");
    if (w->KH != 1 || w->KW != 1) return fail(SBNN_ERR_SHAPE, "packed layer is %dx%d, expected 1x1", w->KH, w->KW);
    if (flags & ~(SBNN_RELU | SBNN_OUT_CM)) return fail(SBNN_ERR_UNSUPPORTED, "flag bits 0x%x not accepted here", flags);
    const bool out_cm = (flags & SBNN_OUT_CM) != 0;
    if (M < 0 || ldx < M || ldx % 4) return fail(SBNN_ERR_SHAPE, "ldx=%d must be >= M=%d and a multiple of 4", ldx, M);
    if (out_cm ? (ldy < M || ldy % 4) : (ldy < w->Cout || ldy % 4))
        return fail(SBNN_ERR_SHAPE, "ldy=%d does not fit the output layout", ldy);
    if (!aligned16(xt_dev) || !aligned16(y_dev)) return fail(SBNN_ERR_ALIGN, "xt_dev and y_dev must be 16-byte aligned");
    if (M == 0) return SBNN_OK;
    sbnn_status st = check_packed_device(w);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    if (!(P | GPW | NW | KC) && few_tiles(w, M))
        return conv1x1_small(w, xt_dev, ldx, y_dev, ldy, M, flags & SBNN_RELU, out_cm, static_cast<cudaStream_t>(cuda_stream));
    const TileCfg c = (P | GPW | NW | KC) ? TileCfg{P, GPW, NW, KC} : default_cfg_cm(w, M);
    return dispatch_cm(w, c, xt_dev, ldx, y_dev, ldy, M, flags & SBNN_RELU, out_cm, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" sbnn_status sbnn_dwconv3x3_conv1x1_gs_cm(const sbnn_packed* pw, const float* dw_w_dev, const float* dw_b_dev,
                                                    const float* xt_dev, int ldx, float* yt_dev, int ldy, int N, int H, int W,
                                                    int dw_flags, int pw_flags, void* cuda_stream) {
    clear_error();
    if (!pw || !dw_w_dev || !xt_dev || !yt_dev) return fail(SBNN_ERR_NULL, "pw, dw_w_dev, xt_dev and yt_dev must not be NULL");
    if (pw->KH != 1 || pw->KW != 1) return fail(SBNN_ERR_SHAPE, "packed layer is %dx%d, expected 1x1", pw->KH, pw->KW);
    if ((dw_flags & ~SBNN_RELU) || (pw_flags & ~SBNN_RELU)) return fail(SBNN_ERR_UNSUPPORTED, "only SBNN_RELU is accepted here");
    if (N < 0 || H < 0 || W < 0) return fail(SBNN_ERR_SHAPE, "negative shape %dx%dx%d", N, H, W);
    const long long M = (long long)N * H * W;
    if (M > 0x7fffffffLL / 2) return fail(SBNN_ERR_SHAPE, "N*H*W too large");
    if (ldx < M || ldy < M || ldx % 4 || ldy % 4) return fail(SBNN_ERR_SHAPE, "ldx=%d / ldy=%d must cover the %lld pixels and be multiples of 4", ldx, ldy, M);
    if (!aligned16(xt_dev) || !aligned16(yt_dev)) return fail(SBNN_ERR_ALIGN, "xt_dev and yt_dev must be 16-byte aligned");
    if (M == 0) return SBNN_OK;
    sbnn_status st = check_packed_device(pw);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    bool done = false;
    st = launch_dwpw(pw, dw_w_dev, dw_b_dev, xt_dev, ldx, yt_dev, ldy, N, H, W, dw_flags & SBNN_RELU, pw_flags & SBNN_RELU,
                     static_cast<cudaStream_t>(cuda_stream), &done);
    if (st != SBNN_OK) return st;
    if (!done) return fail(SBNN_ERR_UNSUPPORTED, "the fused kernel takes G = 4 layers and image widths that are multiples of 4 up to 124");
    return SBNN_OK;
}
