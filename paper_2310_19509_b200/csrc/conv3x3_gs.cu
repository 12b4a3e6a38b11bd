// Group-sparse 3x3 convolution, stride 1, pad 1, fp32: whole 3x3 kernels of one input channel are
// kept or removed jointly for a group of G output channels (connectivity group pruning, Section 3.2).
//
//   Y[n][y][x][g*G+r] = act( b + sum_j sum_{kh,kw} val[g][j][kh*3+kw][r] * X[n][y+kh-1][x+kw-1][idx[g][j]] )
//
// Work decomposition
//   * Image rows of the whole batch are numbered f = n*H + y.  A CTA owns R consecutive rows f and GT
//     consecutive groups, and walks the input channels in steps of KC.
//   * Per step the rows f0-1 .. f0+R of KC channels are staged in shared memory as one plane per
//     channel ([row][column], column = x + 1, so that x = -1 and x = W are zero columns).  Row 0 of
//     every plane is an all-zero row: a lane whose image row is the first (last) of its image reads
//     that row instead of the row above (below), which gives the vertical padding without branches
//     and lets a CTA's rows span several images.
//   * A lane owns CW consecutive output columns of one row (CW = 7 or 8, chosen so that the lanes of
//     a row tile the width with least waste; ImageNet-style maps have W = 7 * 2^k), a warp owns 32/LPR
//     rows (LPR lanes per row), and keeps CW x G x GPW partial sums in registers.  Per kept unit and
//     kernel row a lane reads CW+2 activations and feeds 3*CW*G FMAs; the 9*G weights of the unit are
//     broadcast reads.  The plane pitch is picked on the host so that the 32 lanes of a warp hit 32
//     different banks.
#include <string.h>

#include <algorithm>

#include "common.h"
#include "pipeline.cuh"
#include "shares.h"

namespace sbnn {
namespace {

struct Geo3 {
    int N, H, W, Cin, Cout, ngroups;
    int LPR, RPW, R;        // lanes per row, rows per warp, rows per CTA
    int pitch, plane;       // floats
    int nchunks;
    int dpp_row, dpp_x;     // how (row, x) advance when a thread's staged pixel index grows by its stride
};

// RPL = output rows per lane (copy-engine kernel only): with two, a lane's CW x 2 outputs share the four input rows
// and the nine weight vectors of a kept kernel, so 36 activation loads and 9 weight loads feed 2 * 63 * G FMAs.
template <int G_, int CW_, int GPW_, int NPW_, int NGW_, int KC_, int RPL_ = 1>
struct K3 {
    static constexpr int G = G_, CW = CW_, GPW = GPW_, NPW = NPW_, NGW = NGW_, KC = KC_, RPL = RPL_;
    static constexpr int NW = NPW * NGW, NT = NW * 32, GT = NGW * GPW;
    static constexpr int UNIT = 1 + (9 * G + 3) / 4;   // record of one kept unit, 16-byte units
    static constexpr int HDR = (GT * 2 + 3) / 4;
    static constexpr int WS_U4 = HDR + GT * KC * UNIT;
    // Pattern layers use a list of kept taps instead (quads of 4 taps: 4 offsets, then 4 x G weights), see build_stream3_taps.
    static constexpr int TQUAD = 1 + G;
    static constexpr int WS_U4_TAPS = HDR + GT * ((KC * 9 + 3) / 4 + 1) * TQUAD;
    static_assert(KC % 4 == 0, "KC");
};

template <class C>
__global__ void __launch_bounds__(C::NT, 1)
conv3x3_gs_kernel(const float* __restrict__ X, float* __restrict__ Y, const float* __restrict__ bias,
                  const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr, Geo3 geo, int relu) {
    constexpr int G = C::G, CW = C::CW, GPW = C::GPW, KC = C::KC;
    extern __shared__ __align__(16) unsigned char smem[];
    float* xs = reinterpret_cast<float*>(smem);                                  // [KC][plane]
    uint4* ws = reinterpret_cast<uint4*>(smem + (size_t)KC * geo.plane * 4);     // weight block

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pw = warp % C::NPW, gw = warp / C::NPW;
    const int f0 = blockIdx.x * geo.R;
    const int tile = blockIdx.y;
    const int NH = geo.N * geo.H, W = geo.W, Cin = geo.Cin;
    const int32_t* bp = blk_ptr + (size_t)tile * (geo.nchunks + 1);

    // zero the planes once: zero rows, zero columns and rows outside the batch stay zero for good
    for (int i = tid; i < KC * geo.plane; i += C::NT) xs[i] = 0.0f;

    // this lane's pixels
    const int lrow = pw * geo.RPW + lane / geo.LPR;   // row inside the CTA tile
    const int lx = (lane % geo.LPR) * CW;             // first output column
    const int f = f0 + lrow;
    const int y = f % geo.H;
    // plane row r holds image row f0 - 2 + r  (r = 0 is the zero row)
    int rowoff[3];
    rowoff[0] = (y > 0) ? (lrow + 1) * geo.pitch : 0;
    rowoff[1] = (lrow + 2) * geo.pitch;
    rowoff[2] = (y < geo.H - 1) ? (lrow + 3) * geo.pitch : 0;
#pragma unroll
    for (int k = 0; k < 3; ++k) rowoff[k] += lx;

    float acc[GPW][CW][G];
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + gw * GPW + q;
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float b = (g < geo.ngroups) ? bias[g * G + r] : 0.0f;
#pragma unroll
            for (int p = 0; p < CW; ++p) acc[q][p][r] = b;
        }
    }

    // staging: a thread owns channel quad (tid % (KC/4)) of pixels tid/(KC/4) + j*stride
    constexpr int QPP = KC / 4;                 // float4 loads per pixel and step
    constexpr int PSTRIDE = C::NT / QPP;        // pixel stride between a thread's loads
    static_assert(C::NT % QPP == 0, "staging split");
    const int cq = tid % QPP;
    const int npix = (geo.R + 2) * W;           // pixels of rows f0-1 .. f0+R
    const long long pix0 = (long long)(f0 - 1) * W;   // global pixel index of the first staged pixel

    for (int k = 0; k < geo.nchunks; ++k) {
        __syncthreads();   // previous step's reads are done (and the zero fill, first time)
        {
            const int beg = bp[k], n = bp[k + 1] - beg;
            for (int i = tid; i < n; i += C::NT) ws[i] = rec[beg + i];
            const int c = k * KC + cq * 4;
            int pp = tid / QPP;
            int prow = pp / W, px = pp - prow * W;
            for (; pp < npix; pp += PSTRIDE) {
                const long long gp = pix0 + pp;
                if (c < Cin && gp >= 0 && gp < (long long)NH * W) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(X + (size_t)gp * Cin + c));
                    float* d = xs + (size_t)(cq * 4) * geo.plane + (prow + 1) * geo.pitch + px + 1;
                    d[0] = v.x;
                    d[geo.plane] = v.y;
                    d[2 * geo.plane] = v.z;
                    d[3 * geo.plane] = v.w;
                }
                prow += geo.dpp_row;
                px += geo.dpp_x;
                if (px >= W) { px -= W; ++prow; }
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int2 hd = reinterpret_cast<const int2*>(ws)[gw * GPW + q];   // (start, units)
            const uint4* r = ws + hd.x;
            for (int it = 0; it < hd.y; ++it, r += C::UNIT) {
                const float* plane = xs + r[0].x;                 // plane offset in floats
                const float* wq = reinterpret_cast<const float*>(r + 1);   // [9][G]
#pragma unroll
                for (int kh = 0; kh < 3; ++kh) {
                    const float* arow = plane + rowoff[kh];
                    float a[CW + 2];
#pragma unroll
                    for (int i = 0; i < CW + 2; ++i) a[i] = arow[i];
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) {
                        float w[G];
                        if constexpr (G % 4 == 0) {
#pragma unroll
                            for (int v = 0; v < G / 4; ++v) {
                                const float4 t = reinterpret_cast<const float4*>(wq + (kh * 3 + kw) * G)[v];
                                w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
                            }
                        } else {
#pragma unroll
                            for (int rr = 0; rr < G; ++rr) w[rr] = wq[(kh * 3 + kw) * G + rr];
                        }
#pragma unroll
                        for (int p = 0; p < CW; ++p)
#pragma unroll
                            for (int rr = 0; rr < G; ++rr) acc[q][p][rr] = fmaf(a[p + kw], w[rr], acc[q][p][rr]);
                    }
                }
            }
        }
    }

    if (f >= NH || lrow >= geo.R) return;
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + gw * GPW + q;
        if (g >= geo.ngroups) continue;
#pragma unroll
        for (int p = 0; p < CW; ++p) {
            const int x = lx + p;
            if (x >= W) continue;
            float* yp = Y + ((size_t)f * W + x) * geo.Cout + g * G;
            float v[G];
#pragma unroll
            for (int rr = 0; rr < G; ++rr) v[rr] = relu ? fmaxf(acc[q][p][rr], 0.0f) : acc[q][p][rr];
            if constexpr (G >= 4) {
#pragma unroll
                for (int vv = 0; vv < G / 4; ++vv)
                    reinterpret_cast<float4*>(yp)[vv] = make_float4(v[4 * vv], v[4 * vv + 1], v[4 * vv + 2], v[4 * vv + 3]);
            } else if constexpr (G == 2) {
                *reinterpret_cast<float2*>(yp) = make_float2(v[0], v[1]);
            } else {
                yp[0] = v[0];
            }
        }
    }
}


// ---- channel-major variant --------------------------------------------------------------------
// Same decomposition, but X is given as planes ([Cin][ldx], pixel index f*W + x) with W a multiple of 4.
// A plane row is then W/4 aligned 16-byte pieces, which cp.async copies straight into the shared
// memory plane (column = x + 4, so pieces stay 16-byte aligned; column 3 is the zero column for x = -1):
// no registers, no transposing stores, and the copies of step k+1 run while step k is computed
// (two buffers).  Accumulators are packed pairs of output channels updated with fma.rn.f32x2.
__device__ __forceinline__ void cp_async16_3(void* smem, const void* gmem) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}

template <class C>
__global__ void __launch_bounds__(C::NT, 1)
conv3x3_gs_cm_kernel(const float* __restrict__ X, int ldx, float* __restrict__ Y, const float* __restrict__ bias,
                     const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr, Geo3 geo, int relu) {
    constexpr int G = C::G, CW = C::CW, GPW = C::GPW, KC = C::KC;
    constexpr int GP = (G + 1) / 2;                 // packed channel pairs per group
    constexpr int NIT = 2;                          // staged (row, piece) positions per thread (checked on the host)
    extern __shared__ __align__(16) unsigned char smem[];
    const int xs_floats = KC * geo.plane;
    float* xs0 = reinterpret_cast<float*>(smem);                                          // two plane sets
    uint4* ws0 = reinterpret_cast<uint4*>(smem + (size_t)2 * xs_floats * 4);              // two weight blocks

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pw = warp % C::NPW, gw = warp / C::NPW;
    const int f0 = blockIdx.x * geo.R;
    const int tile = blockIdx.y;
    const int NH = geo.N * geo.H, W = geo.W;
    const int32_t* bp = blk_ptr + (size_t)tile * (geo.nchunks + 1);

    for (int i = tid; i < 2 * xs_floats; i += C::NT) xs0[i] = 0.0f;   // zero rows / columns stay zero for good

    // staging: a thread owns up to NIT (staged row, 16-byte piece) positions and copies them for every
    // channel of the step (source and destination advance by one plane per channel)
    const int QW = W >> 2, rows = geo.R + 2, pieces = rows * QW;
    int src_off[NIT], dst_off[NIT];
#pragma unroll
    for (int j = 0; j < NIT; ++j) {
        const int i = tid + j * C::NT;
        src_off[j] = -1;
        dst_off[j] = 0;
        if (i < pieces) {
            const int q = i % QW, row = i / QW;
            const long long f = (long long)f0 - 1 + row;
            if (f >= 0 && f < NH) {
                src_off[j] = (int)f * W + 4 * q;
                dst_off[j] = (row + 1) * geo.pitch + 4 + 4 * q;
            }
        }
    }
    auto issue = [&](int k, int buf) {
        const float* xk = X + (size_t)k * KC * ldx;
        float* xd = xs0 + buf * xs_floats;
        const int nc = min(KC, geo.Cin - k * KC);                                // channels of this step
#pragma unroll
        for (int j = 0; j < NIT; ++j)
            if (src_off[j] >= 0)
                for (int c = 0; c < nc; ++c) cp_async16_3(xd + c * geo.plane + dst_off[j], xk + (size_t)c * ldx + src_off[j]);
        uint4* wd = ws0 + buf * C::WS_U4;
        const int beg = bp[k], n = bp[k + 1] - beg;
        for (int i = tid; i < n; i += C::NT) cp_async16_3(wd + i, rec + beg + i);
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };

    const int lrow = pw * geo.RPW + lane / geo.LPR;
    const int lx = (lane % geo.LPR) * CW;
    const int f = f0 + lrow;
    const int y = f % geo.H;
    int rowoff[3];
    rowoff[0] = (y > 0) ? (lrow + 1) * geo.pitch : 0;
    rowoff[1] = (lrow + 2) * geo.pitch;
    rowoff[2] = (y < geo.H - 1) ? (lrow + 3) * geo.pitch : 0;
#pragma unroll
    for (int k = 0; k < 3; ++k) rowoff[k] += lx + 3;   // column of x = lx - 1

    f32x2 acc[GPW][CW][GP];
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + gw * GPW + q;
#pragma unroll
        for (int r = 0; r < GP; ++r) {
            const float b0 = (g < geo.ngroups) ? bias[g * G + 2 * r] : 0.0f;
            const float b1 = (g < geo.ngroups && 2 * r + 1 < G) ? bias[g * G + 2 * r + 1] : 0.0f;
#pragma unroll
            for (int p = 0; p < CW; ++p) acc[q][p][r] = pack2(b0, b1);
        }
    }

    __syncthreads();            // zero fill done before the first copies land
    issue(0, 0);
    for (int k = 0; k < geo.nchunks; ++k) {
        const int cur = k & 1;
        if (k + 1 < geo.nchunks) {
            issue(k + 1, cur ^ 1);
            asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        }
        __syncthreads();
        const float* xs = xs0 + cur * xs_floats;
        const uint4* ws = ws0 + cur * C::WS_U4;
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int2 hd = reinterpret_cast<const int2*>(ws)[gw * GPW + q];
            const uint4* r = ws + hd.x;
            for (int it = 0; it < hd.y; ++it, r += C::UNIT) {
                const float* plane = xs + r[0].x;
                const float* wq = reinterpret_cast<const float*>(r + 1);   // [9][G]
#pragma unroll
                for (int kh = 0; kh < 3; ++kh) {
                    const float* arow = plane + rowoff[kh];
                    f32x2 a[CW + 2];
#pragma unroll
                    for (int i = 0; i < CW + 2; ++i) a[i] = dup2(arow[i]);
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) {
                        f32x2 w[GP];
                        if constexpr (G % 4 == 0) {
#pragma unroll
                            for (int v = 0; v < G / 4; ++v) {
                                const ulonglong2 t = reinterpret_cast<const ulonglong2*>(wq + (kh * 3 + kw) * G)[v];
                                w[2 * v] = t.x;
                                w[2 * v + 1] = t.y;
                            }
                        } else if constexpr (G == 2) {
                            w[0] = *reinterpret_cast<const unsigned long long*>(wq + (kh * 3 + kw) * 2);
                        } else {
                            w[0] = pack2(wq[kh * 3 + kw], 0.0f);
                        }
#pragma unroll
                        for (int p = 0; p < CW; ++p)
#pragma unroll
                            for (int rr = 0; rr < GP; ++rr) fma2(acc[q][p][rr], a[p + kw], w[rr]);
                    }
                }
            }
        }
        __syncthreads();        // everyone is done with this buffer before the copies of step k+2 are issued
    }

    if (f >= NH) return;
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + gw * GPW + q;
        if (g >= geo.ngroups) continue;
#pragma unroll
        for (int p = 0; p < CW; ++p) {
            const int x = lx + p;
            if (x >= W) continue;
            float* yp = Y + ((size_t)f * W + x) * geo.Cout + g * G;
            float v[2 * GP];
#pragma unroll
            for (int rr = 0; rr < GP; ++rr) unpack2(acc[q][p][rr], v[2 * rr], v[2 * rr + 1]);
            if (relu) {
#pragma unroll
                for (int rr = 0; rr < 2 * GP; ++rr) v[rr] = fmaxf(v[rr], 0.0f);
            }
            if constexpr (G >= 4) {
#pragma unroll
                for (int vv = 0; vv < G / 4; ++vv)
                    reinterpret_cast<float4*>(yp)[vv] = make_float4(v[4 * vv], v[4 * vv + 1], v[4 * vv + 2], v[4 * vv + 3]);
            } else if constexpr (G == 2) {
                *reinterpret_cast<float2*>(yp) = make_float2(v[0], v[1]);
            } else {
                yp[0] = v[0];
            }
        }
    }
}

// ---- channel-major variant with a copy-engine pipeline ------------------------------------------------
// Same decomposition and inner loop as conv3x3_gs_cm_kernel, but the staging is taken off the compute warps: the
// planes of X are a 3-D tensor [Cin][N*H][W], and one tiled copy per channel step brings the box
// (pitch columns from x = -4, R + 2 rows from f0 - 1, KC channels) into a stage; columns and rows outside the
// tensor arrive as zeros, which is exactly the horizontal padding.  A producer warp issues that copy and the
// linear copy of the step's weight block onto the stage's "full" mbarrier; the compute warps release a stage
// through its "empty" mbarrier, so a warp whose groups keep more kernels in one step is not waited for at a
// CTA-wide barrier (ncu had 19 % of the stall cycles of the two-buffer version there).  Vertical padding between
// images: rows of a neighbouring image are replaced by a row of zeros kept beside the stages.  Waits are bounded.
struct Map3 { alignas(64) unsigned char bytes[128]; };

// The launch is a fixed number of persistent CTAs (one per SM), and the channel steps of all tiles, laid end to end,
// are dealt to them in equal shares of weight-stream volume, so a launch whose tile count is not a multiple of the SM
// count (config 4 of the paper's Table-3-style shapes: 256 equal tiles on 148 SMs) leaves no SM idle in a last round.
// A share is a list of segments; a tile that falls into several shares has nparts > 1: each part writes its partial
// sums to its slot, counts itself in on the tile's counter, and the part that arrives last adds the slots in part
// order (so the result does not depend on which part that was), adds the bias and stores the tile.  Nobody waits.
struct Seg3 {
    int bx, by;            // row tile, group tile
    int k0, k1;            // channel steps [k0, k1)
    int part, nparts;      // this segment's position among the tile's parts
    int slot, counter;     // first partial-sum slot and arrival counter of the tile (nparts > 1)
};

__device__ __forceinline__ void compute_warps_barrier(int nthreads) {
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

template <class C, bool PAT, bool OUT_CM = false>
__global__ void __launch_bounds__(C::NT + 32, 1)
conv3x3_gs_tma_kernel(const __grid_constant__ Map3 xmap, float* __restrict__ Y, const float* __restrict__ bias,
                      const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr, Geo3 geo, int relu, int S,
                      int stage_bytes, int* status, const int32_t* __restrict__ cta_ptr, const Seg3* __restrict__ segs,
                      f32x2* partial, int* counters, int ldy) {
    constexpr int G = C::G, CW = C::CW, GPW = C::GPW, KC = C::KC, NW = C::NW, RPL = C::RPL;
    constexpr int GP = (G + 1) / 2;
    static_assert(!PAT || RPL == 1, "the tap lists address one output row per lane");
    constexpr int ACC2 = GPW * RPL * CW * GP;                            // packed partial sums per thread
    extern __shared__ __align__(128) unsigned char smem[];
    const int xs_bytes = KC * geo.plane * 4;                       // one stage: KC planes, then the weight block
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)S * stage_bytes);
    uint64_t* empty = full + S;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + S);
    volatile int* last_flag = abort_flag + 1;
    float* zrow = reinterpret_cast<float*>(empty + S) + 4;         // geo.pitch zeros

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NH = geo.N * geo.H, W = geo.W;
    const int seg_beg = cta_ptr[blockIdx.x], seg_end = cta_ptr[blockIdx.x + 1];

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, NW);
        }
        *abort_flag = 0;
        *last_flag = 0;
        mbar_fence_init();
    }
    for (int i = tid; i < geo.pitch; i += blockDim.x) zrow[i] = 0.0f;
    __syncthreads();

    if (warp == NW) {
        // ---------------- producer warp ----------------
        bool ok = true;
        int it = 0;                                                // steps issued by this CTA so far (all segments)
        for (int si = seg_beg; si < seg_end && ok; ++si) {
            const Seg3 sg = segs[si];
            const int32_t* bp = blk_ptr + (size_t)sg.by * (geo.nchunks + 1);
            const int f0 = sg.bx * geo.R;
            for (int k = sg.k0; k < sg.k1; ++k, ++it) {
                const int s = it % S;
                if (it >= S) ok = mbar_wait(empty + s, ((it / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT);
                if (!ok) break;
                if (lane == 0) {
                    const int wbeg = bp[k], wn = bp[k + 1] - wbeg;
                    unsigned char* st = smem + (size_t)s * stage_bytes;
                    mbar_arrive_expect_tx(full + s, (uint32_t)xs_bytes + (uint32_t)wn * 16u);
                    tensor_g2s_3d(st, &xmap, -4, f0 - 1, k * KC, full + s);
                    bulk_g2s(st + xs_bytes, rec + wbeg, (uint32_t)wn * 16u, full + s);
                }
            }
        }
        if (!ok) {   // gave up: let the copies already issued land before the CTA's shared memory is released
            for (int j = max(0, it - S); j < it; ++j) {
                bool landed = false;
                for (uint32_t i = 0; i < kWaitLimit && !landed; ++i) landed = mbar_try_wait(full + j % S, (j / S) & 1);
            }
        }
        return;
    }

    // ---------------- compute warps ----------------
    const int pw = warp % C::NPW, gw = warp / C::NPW;
    const int lrow = (pw * geo.RPW + lane / geo.LPR) * RPL;      // first of the lane's RPL output rows
    const int lx = (lane % geo.LPR) * CW;
    // plane row j holds image row f0 - 1 + j; column c holds x = c - 4
    int rowoff[RPL + 2];
#pragma unroll
    for (int jr = 0; jr < RPL + 2; ++jr) rowoff[jr] = (lrow + jr) * geo.pitch + lx + 3;   // column of x = lx - 1
    const float* zr = zrow + lx + 3;
    const int lanebase = lrow * geo.pitch + lx + 3;                // tap (kh, kw) of a plane: + kh * pitch + kw, then CW inputs

    int it = 0;                                                    // steps consumed by this CTA so far (all segments)
    bool alive = true;                                             // false once a wait has given up; the barriers below are still joined
    for (int si = seg_beg; si < seg_end; ++si) {
        const Seg3 sg = segs[si];
        const bool split = sg.nparts > 1;
        const int tile = sg.by;
        const int f = sg.bx * geo.R + lrow;
        const int y = f % geo.H;
        // the lane's RPL rows lie in one image (H is a multiple of RPL), so only the rows above the first and below
        // the last can belong to a neighbouring image
        const bool ok_first = y > 0, ok_last = y + RPL - 1 < geo.H - 1;
        const unsigned rowmask = (ok_first ? 1u : 0u) | 2u | (ok_last ? 4u : 0u);
        (void)rowmask;

        f32x2 acc[GPW][RPL][CW][GP];
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int g = tile * C::GT + gw * GPW + q;
#pragma unroll
            for (int r = 0; r < GP; ++r) {
                // a tile in one piece starts from the bias; the parts of a split tile start from zero
                const float b0 = (!split && g < geo.ngroups) ? bias[g * G + 2 * r] : 0.0f;
                const float b1 = (!split && g < geo.ngroups && 2 * r + 1 < G) ? bias[g * G + 2 * r + 1] : 0.0f;
#pragma unroll
                for (int ro = 0; ro < RPL; ++ro)
#pragma unroll
                    for (int p = 0; p < CW; ++p) acc[q][ro][p][r] = pack2(b0, b1);
            }
        }

        if (alive) {
            for (int k = sg.k0; k < sg.k1; ++k, ++it) {
                const int s = it % S;
                if (!mbar_wait(full + s, (it / S) & 1, abort_flag, status, SBNN_ERR_TIMEOUT)) {
                    alive = false;
                    break;
                }
                const float* xs = reinterpret_cast<const float*>(smem + (size_t)s * stage_bytes);
                const uint4* ws = reinterpret_cast<const uint4*>(smem + (size_t)s * stage_bytes + xs_bytes);
#pragma unroll
                for (int q = 0; q < GPW; ++q) {
                    const int2 hd = reinterpret_cast<const int2*>(ws)[gw * GPW + q];
                    const uint4* r = ws + hd.x;
                    if constexpr (PAT) {
                        // Layers packed with kernel patterns (Section 3.3): the stream lists the kept taps of the group's kept
                        // kernels one by one, four to a record (offset of the tap's first input inside the stage with the kernel
                        // row in the top two bits, then the G weights of each), so pruned taps cost nothing and the loop has no
                        // data-dependent branch.  A list is padded to a whole record with taps of weight zero.
                        for (int j = 0; j < hd.y; ++j, r += C::TQUAD) {
                            const uint4 off4 = r[0];
                            const unsigned offs[4] = {off4.x, off4.y, off4.z, off4.w};
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const unsigned kh = offs[u] >> 30;
                                const float* arow = ((rowmask >> kh) & 1u) ? xs + (offs[u] & 0x3FFFFFFFu) + lanebase : zr;
                                f32x2 a[CW];
#pragma unroll
                                for (int i = 0; i < CW; ++i) a[i] = dup2(arow[i]);
                                const float* wq = reinterpret_cast<const float*>(r + 1) + u * G;
                                f32x2 w[GP];
                                if constexpr (G % 4 == 0) {
#pragma unroll
                                    for (int v = 0; v < G / 4; ++v) {
                                        const ulonglong2 t = reinterpret_cast<const ulonglong2*>(wq)[v];
                                        w[2 * v] = t.x;
                                        w[2 * v + 1] = t.y;
                                    }
                                } else if constexpr (G == 2) {
                                    w[0] = *reinterpret_cast<const unsigned long long*>(wq);
                                } else {
                                    w[0] = pack2(wq[0], 0.0f);
                                }
#pragma unroll
                                for (int p = 0; p < CW; ++p)
#pragma unroll
                                    for (int rr = 0; rr < GP; ++rr) fma2(acc[q][0][p][rr], a[p], w[rr]);
                            }
                        }
                    } else {
                    for (int j = 0; j < hd.y; ++j, r += C::UNIT) {
                        const float* plane = xs + r[0].x;
                        const float* wq = reinterpret_cast<const float*>(r + 1);   // [9][G]
                        f32x2 w[3][3][GP];                                          // tap row kh is fetched with input row kh
#pragma unroll
                        for (int jr = 0; jr < RPL + 2; ++jr) {
                            const bool ok = jr == 0 ? ok_first : (jr == RPL + 1 ? ok_last : true);
                            const float* arow = ok ? plane + rowoff[jr] : zr;
                            f32x2 a[CW + 2];
#pragma unroll
                            for (int i = 0; i < CW + 2; ++i) a[i] = dup2(arow[i]);
                            if (jr < 3) {
#pragma unroll
                                for (int kw = 0; kw < 3; ++kw) {
                                    if constexpr (G % 4 == 0) {
#pragma unroll
                                        for (int v = 0; v < G / 4; ++v) {
                                            const ulonglong2 t = reinterpret_cast<const ulonglong2*>(wq + (jr * 3 + kw) * G)[v];
                                            w[jr < 3 ? jr : 0][kw][2 * v] = t.x;
                                            w[jr < 3 ? jr : 0][kw][2 * v + 1] = t.y;
                                        }
                                    } else if constexpr (G == 2) {
                                        w[jr < 3 ? jr : 0][kw][0] = *reinterpret_cast<const unsigned long long*>(wq + (jr * 3 + kw) * 2);
                                    } else {
                                        w[jr < 3 ? jr : 0][kw][0] = pack2(wq[jr * 3 + kw], 0.0f);
                                    }
                                }
                            }
                            // input row jr is tap row kh = jr - ro of output row ro
#pragma unroll
                            for (int ro = 0; ro < RPL; ++ro) {
                                const int kh = jr - ro;
                                if (kh < 0 || kh > 2) continue;
#pragma unroll
                                for (int kw = 0; kw < 3; ++kw)
#pragma unroll
                                    for (int p = 0; p < CW; ++p)
#pragma unroll
                                        for (int rr = 0; rr < GP; ++rr) fma2(acc[q][ro][p][rr], a[p + kw], w[kh][kw][rr]);
                            }
                        }
                    }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + s);
            }
        }

        if (split) {
            // partial sums of this part -> its slot, [packed sum][thread]
            f32x2* mine = partial + (size_t)(sg.slot + sg.part) * (ACC2 * C::NT) + tid;
            if (alive) {
#pragma unroll
                for (int q = 0; q < GPW; ++q)
#pragma unroll
                    for (int ro = 0; ro < RPL; ++ro)
#pragma unroll
                        for (int p = 0; p < CW; ++p)
#pragma unroll
                            for (int rr = 0; rr < GP; ++rr)
                                mine[(size_t)(((q * RPL + ro) * CW + p) * GP + rr) * C::NT] = acc[q][ro][p][rr];
            }
            __threadfence();
            compute_warps_barrier(C::NT);
            if (tid == 0) *last_flag = (!*abort_flag && atomicAdd(counters + sg.counter, 1) == sg.nparts - 1) ? 1 : 0;
            compute_warps_barrier(C::NT);
            const bool last = *last_flag != 0;
            if (!last || !alive) continue;
            __threadfence();
            // Part 0 straight into the accumulators (all loads independent and in flight together), then the other
            // parts in part order, CW * GP loads at a time, and the bias last.  (One accumulator after the other, each
            // with its own loop over the parts, was a chain of ACC2 * nparts dependent L2 latencies.)
            const f32x2* src = partial + (size_t)sg.slot * (ACC2 * C::NT) + tid;
#pragma unroll
            for (int q = 0; q < GPW; ++q)
#pragma unroll
                for (int ro = 0; ro < RPL; ++ro)
#pragma unroll
                    for (int p = 0; p < CW; ++p)
#pragma unroll
                        for (int rr = 0; rr < GP; ++rr)
                            acc[q][ro][p][rr] = __ldcg(src + (size_t)(((q * RPL + ro) * CW + p) * GP + rr) * C::NT);
            for (int j = 1; j < sg.nparts; ++j) {
                src += (size_t)ACC2 * C::NT;
#pragma unroll
                for (int q = 0; q < GPW; ++q)
#pragma unroll
                    for (int ro = 0; ro < RPL; ++ro) {
                        f32x2 t[CW][GP];
#pragma unroll
                        for (int p = 0; p < CW; ++p)
#pragma unroll
                            for (int rr = 0; rr < GP; ++rr)
                                t[p][rr] = __ldcg(src + (size_t)(((q * RPL + ro) * CW + p) * GP + rr) * C::NT);
#pragma unroll
                        for (int p = 0; p < CW; ++p)
#pragma unroll
                            for (int rr = 0; rr < GP; ++rr) {
                                float s0, s1, t0, t1;
                                unpack2(acc[q][ro][p][rr], s0, s1);
                                unpack2(t[p][rr], t0, t1);
                                acc[q][ro][p][rr] = pack2(s0 + t0, s1 + t1);
                            }
                    }
            }
#pragma unroll
            for (int q = 0; q < GPW; ++q) {
                const int g = tile * C::GT + gw * GPW + q;
#pragma unroll
                for (int rr = 0; rr < GP; ++rr) {
                    const float b0 = (g < geo.ngroups) ? bias[g * G + 2 * rr] : 0.0f;
                    const float b1 = (g < geo.ngroups && 2 * rr + 1 < G) ? bias[g * G + 2 * rr + 1] : 0.0f;
#pragma unroll
                    for (int ro = 0; ro < RPL; ++ro)
#pragma unroll
                        for (int p = 0; p < CW; ++p) {
                            float s0, s1;
                            unpack2(acc[q][ro][p][rr], s0, s1);
                            acc[q][ro][p][rr] = pack2(s0 + b0, s1 + b1);
                        }
                }
            }
        } else if (!alive) {
            continue;
        }

#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int g = tile * C::GT + gw * GPW + q;
            if (g >= geo.ngroups) continue;
#pragma unroll
            for (int ro = 0; ro < RPL; ++ro)
#pragma unroll
            for (int p = 0; p < CW; ++p) {
                const int x = lx + p;
                if (x >= W || f + ro >= NH) continue;
                float v[2 * GP];
#pragma unroll
                for (int rr = 0; rr < GP; ++rr) unpack2(acc[q][ro][p][rr], v[2 * rr], v[2 * rr + 1]);
                if (relu) {
#pragma unroll
                    for (int rr = 0; rr < 2 * GP; ++rr) v[rr] = fmaxf(v[rr], 0.0f);
                }
                if constexpr (OUT_CM) {                             // [Cout][ldy]: a lane's CW columns are a contiguous run
#pragma unroll
                    for (int rr = 0; rr < G; ++rr) Y[(size_t)(g * G + rr) * ldy + (size_t)(f + ro) * W + x] = v[rr];
                    continue;
                }
                float* yp = Y + ((size_t)(f + ro) * W + x) * ldy + g * G;
                if constexpr (G >= 4) {
#pragma unroll
                    for (int vv = 0; vv < G / 4; ++vv)
                        reinterpret_cast<float4*>(yp)[vv] = make_float4(v[4 * vv], v[4 * vv + 1], v[4 * vv + 2], v[4 * vv + 3]);
                } else if constexpr (G == 2) {
                    *reinterpret_cast<float2*>(yp) = make_float2(v[0], v[1]);
                } else {
                    yp[0] = v[0];
                }
            }
        }
    }
}

// X [M][C] (pixel-major, M = rows * W) -> planes Xt [C][rows][Wp] with the image rows padded to Wp >= W floats (a
// multiple of 4, so that a row starts on a 16-byte boundary as the tiled copy requires): 32 x 32 tiles through
// padded shared memory.  The Wp - W floats behind a row are never read (the copy treats x >= W as outside the tensor).
__global__ void __launch_bounds__(256)
to_padded_planes_kernel(const float* __restrict__ x, float* __restrict__ xt, int M, int C, int W, int Wp, long long ld) {
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
        if (m < M && c < C) xt[(size_t)c * ld + (size_t)(m / W) * Wp + (m % W)] = t[tx][ty + 8 * i];
    }
}

// Planes Xt [C][ldx] (rows of W floats back to back) -> planes [C][rows][Wp] with rows padded to Wp floats.
__global__ void __launch_bounds__(256)
pad_plane_rows_kernel(const float* __restrict__ xt, long long ldx, float* __restrict__ xp, long long ldp, long long rows, int W,
                      int Wp) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // element of a plane
    const int c = blockIdx.y;
    if (i >= rows * W) return;
    xp[(size_t)c * ldp + (size_t)(i / W) * Wp + (i % W)] = xt[(size_t)c * ldx + i];
}

// ---- host side -------------------------------------------------------------------------------

// Number of SMs of the current device (one persistent CTA each).
int sm_count3() {
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

// True if a layer packed with kernel patterns should run the tap-list kernel: a listed tap costs about 60 us per "every
// kept kernel, one tap" on config 4's shape, the whole-kernel loop with two output rows per lane about 35 us per tap
// including the pruned ones (their stored weights are zeros), so lists pay below about five kept taps per kernel.
bool use_tap_lists(const sbnn_packed* p) {
    if (p->tap_mask.empty()) return false;
    std::lock_guard<std::mutex> lk(p->mu);
    if (p->kept_taps < 0) {
        long long n = 0;
        for (uint16_t m : p->tap_mask) n += __builtin_popcount(m);
        p->kept_taps = n;
    }
    return (double)p->kept_taps < 4.8 * (double)p->tap_mask.size();
}

int pow2_ceil(int v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Lanes per row for a column width; 0 if the image is too wide for one warp row.
int lanes_per_row(int W, int CW) {
    const int l = pow2_ceil((W + CW - 1) / CW);
    return l <= 32 ? l : 0;
}

// Smallest pitch >= LPR*CW+2 for which the first reads of the 32 lanes fall into 32 distinct banks.
int pick_pitch(int LPR, int CW) {
    const int lo = LPR * CW + 2;
    for (int p = lo; p < lo + 64; ++p) {
        unsigned used = 0;
        bool ok = true;
        for (int l = 0; l < 32 && ok; ++l) {
            const int b = ((l / LPR) * p + (l % LPR) * CW) & 31;
            ok = !((used >> b) & 1u);
            used |= 1u << b;
        }
        if (ok) return p;
    }
    return lo;
}

// Record stream: block (tile t, step k) = GT (start, units) pairs, then per group its units:
// one 16-byte word whose first lane is the plane offset in floats, then the 9*G weights.
sbnn_status build_stream3(const sbnn_packed* p, int GT, int KC, int plane, Stream3x3* out) {
    const int G = p->G;
    const int ntiles = (p->ngroups + GT - 1) / GT, nchunks = (p->Cin + KC - 1) / KC;
    const int HDR = (GT * 2 + 3) / 4, UNIT = 1 + (9 * G + 3) / 4;
    std::vector<int32_t> blk((size_t)ntiles * (nchunks + 1));
    std::vector<uint32_t> rec;
    int max_blk = 0;
    try {
        for (int t = 0; t < ntiles; ++t) {
            for (int k = 0; k < nchunks; ++k) {
                const size_t blk_beg = rec.size() / 4;
                blk[(size_t)t * (nchunks + 1) + k] = (int32_t)blk_beg;
                rec.resize(rec.size() + (size_t)HDR * 4, 0u);
                for (int s = 0; s < GT; ++s) {
                    const int g = t * GT + s;
                    int lo = 0, hi = 0;
                    if (g < p->ngroups) {
                        const int32_t* b = p->idx.data() + p->group_ptr[g];
                        const int32_t* e = p->idx.data() + p->group_ptr[g + 1];
                        lo = (int)(std::lower_bound(b, e, k * KC) - p->idx.data());
                        hi = (int)(std::lower_bound(b, e, (k + 1) * KC) - p->idx.data());
                    }
                    rec[blk_beg * 4 + 2 * s + 0] = (uint32_t)(rec.size() / 4 - blk_beg);
                    rec[blk_beg * 4 + 2 * s + 1] = (uint32_t)(hi - lo);
                    for (int j = lo; j < hi; ++j) {
                        const size_t base = rec.size();
                        rec.resize(base + (size_t)UNIT * 4, 0u);
                        rec[base] = (uint32_t)((p->idx[j] - k * KC) * plane);
                        memcpy(&rec[base + 4], &p->val[(size_t)j * 9 * G], sizeof(float) * 9 * G);
                    }
                }
                max_blk = std::max(max_blk, (int)(rec.size() / 4 - blk_beg));
            }
            blk[(size_t)t * (nchunks + 1) + nchunks] = (int32_t)(rec.size() / 4);
        }
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the 3x3 weight stream");
    }
    Stream3x3 s;
    s.ntiles = ntiles; s.nchunks = nchunks; s.max_blk = max_blk;
    s.blk_host = blk;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s.rec), std::max<size_t>(rec.size() * 4, 16)));
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&s.blk_ptr), blk.size() * 4);
    if (e == cudaSuccess && !rec.empty()) e = cudaMemcpy(s.rec, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s.blk_ptr, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        cudaFree(s.blk_ptr);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the 3x3 weight stream: %s", cudaGetErrorString(e));
    }
    *out = std::move(s);
    return SBNN_OK;
}

// Stream of a layer packed with kernel patterns, for the tiled-copy kernel: per (group tile, channel step) a header of
// (start, records) per group, then per group the kept taps of its kept kernels in records of four:
// [4 x offset][4 x G weights], offset = plane offset of the input channel + kh * pitch + kw (floats), kernel row kh in
// bits 30-31.  The last record of a list is padded with taps of offset 0 and weight 0.
sbnn_status build_stream3_taps(const sbnn_packed* p, int GT, int KC, int plane, int pitch, Stream3x3* out) {
    const int G = p->G;
    const int ntiles = (p->ngroups + GT - 1) / GT, nchunks = (p->Cin + KC - 1) / KC;
    const int HDR = (GT * 2 + 3) / 4, TQUAD = 1 + G;
    std::vector<int32_t> blk((size_t)ntiles * (nchunks + 1));
    std::vector<uint32_t> rec;
    int max_blk = 0;
    try {
        for (int t = 0; t < ntiles; ++t) {
            for (int k = 0; k < nchunks; ++k) {
                const size_t blk_beg = rec.size() / 4;
                blk[(size_t)t * (nchunks + 1) + k] = (int32_t)blk_beg;
                rec.resize(rec.size() + (size_t)HDR * 4, 0u);
                for (int s = 0; s < GT; ++s) {
                    const int g = t * GT + s;
                    int lo = 0, hi = 0;
                    if (g < p->ngroups) {
                        const int32_t* b = p->idx.data() + p->group_ptr[g];
                        const int32_t* e = p->idx.data() + p->group_ptr[g + 1];
                        lo = (int)(std::lower_bound(b, e, k * KC) - p->idx.data());
                        hi = (int)(std::lower_bound(b, e, (k + 1) * KC) - p->idx.data());
                    }
                    const size_t list_beg = rec.size();
                    int ntaps = 0;
                    for (int j = lo; j < hi; ++j)
                        for (int tap = 0; tap < 9; ++tap) {
                            if (!((p->tap_mask[j] >> tap) & 1u)) continue;
                            if (ntaps % 4 == 0) rec.resize(rec.size() + (size_t)TQUAD * 4, 0u);
                            const size_t base = list_beg + (size_t)(ntaps / 4) * TQUAD * 4;
                            const int kh = tap / 3, kw = tap % 3, u = ntaps % 4;
                            rec[base + u] = (uint32_t)((p->idx[j] - k * KC) * plane + kh * pitch + kw) | ((uint32_t)kh << 30);
                            memcpy(&rec[base + 4 + (size_t)u * G], &p->val[((size_t)j * 9 + tap) * G], sizeof(float) * G);
                            ++ntaps;
                        }
                    rec[blk_beg * 4 + 2 * s + 0] = (uint32_t)(list_beg / 4 - blk_beg);
                    rec[blk_beg * 4 + 2 * s + 1] = (uint32_t)((ntaps + 3) / 4);
                }
                max_blk = std::max(max_blk, (int)(rec.size() / 4 - blk_beg));
            }
            blk[(size_t)t * (nchunks + 1) + nchunks] = (int32_t)(rec.size() / 4);
        }
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the 3x3 tap stream");
    }
    Stream3x3 s;
    s.ntiles = ntiles; s.nchunks = nchunks; s.max_blk = max_blk;
    s.blk_host = blk;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s.rec), std::max<size_t>(rec.size() * 4, 16)));
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&s.blk_ptr), blk.size() * 4);
    if (e == cudaSuccess && !rec.empty()) e = cudaMemcpy(s.rec, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s.blk_ptr, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        cudaFree(s.blk_ptr);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the 3x3 tap stream: %s", cudaGetErrorString(e));
    }
    *out = std::move(s);
    return SBNN_OK;
}

// The launch's work plan (shares.h): the tile sequence is group tile (outermost), row tile; a step weighs its weight
// block (16-byte words: the kept kernels or taps it multiplies) plus a constant for what every step costs (barrier
// round trip, list headers).  `blk` is the stream's block table ([ntiles][nchunks + 1] offsets).  Host arithmetic only.
struct Plan3Host {
    std::vector<int32_t> cta_ptr;
    std::vector<Seg3> segs;
    int ncta = 0, nslots = 0, ncounters = 0;
};
void plan3_host(const int32_t* blk, int ntiles, int nchunks, int nrow, int ncta_max, Plan3Host* out) {
    constexpr long long kStepCost = 6;
    SharePlan sp;
    // the launch's tile sequence: group tile by = tile / nrow outermost, row tile bx = tile % nrow
    plan_shares((long long)ntiles * nrow, nchunks,
                [&](long long tile, int k) {
                    const int32_t* bp = blk + (size_t)(tile / nrow) * (nchunks + 1);
                    return (long long)(bp[k + 1] - bp[k]) + kStepCost;
                },
                ncta_max, &sp);
    out->cta_ptr = std::move(sp.cta_ptr);
    out->segs.resize(sp.segs.size());
    for (size_t i = 0; i < sp.segs.size(); ++i) {
        const ShareSeg& g = sp.segs[i];
        out->segs[i] = Seg3{g.tile % nrow, g.tile / nrow, g.k0, g.k1, g.part, g.nparts, g.slot, g.counter};
    }
    out->ncta = sp.ncta;
    out->nslots = sp.nslots;
    out->ncounters = sp.ncounters;
}

sbnn_status build_plan3(const Stream3x3& s, int nrow, int ncta_max, Plan3x3* out) {
    Plan3Host h;
    try {
        plan3_host(s.blk_host.data(), s.ntiles, s.nchunks, nrow, ncta_max, &h);
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory planning the 3x3 launch");
    }
    Plan3x3 pl;
    pl.ncta = h.ncta;
    pl.nslots = h.nslots;
    pl.ncounters = h.ncounters;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&pl.cta_ptr), h.cta_ptr.size() * 4));
    cudaError_t e = cudaMalloc(&pl.segs, std::max<size_t>(h.segs.size() * sizeof(Seg3), 32));
    if (e == cudaSuccess) e = cudaMemcpy(pl.cta_ptr, h.cta_ptr.data(), h.cta_ptr.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !h.segs.empty()) e = cudaMemcpy(pl.segs, h.segs.data(), h.segs.size() * sizeof(Seg3), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(pl.cta_ptr);
        cudaFree(pl.segs);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the 3x3 launch plan: %s", cudaGetErrorString(e));
    }
    *out = pl;
    return SBNN_OK;
}

template <class C>
sbnn_status launch3(const sbnn_packed* p, const float* x, float* y, int N, int H, int W, int relu, cudaStream_t st) {
    Geo3 g;
    g.N = N; g.H = H; g.W = W; g.Cin = p->Cin; g.Cout = p->Cout; g.ngroups = p->ngroups;
    g.LPR = lanes_per_row(W, C::CW);
    g.RPW = 32 / g.LPR;
    g.R = C::NPW * g.RPW;
    g.pitch = pick_pitch(g.LPR, C::CW);
    int plane = (g.R + 3) * g.pitch;
    plane = (plane + 7) / 8 * 8 + 4;   // multiple of 4 floats, and 4 (mod 8) to spread the staging stores over banks
    g.plane = plane;
    g.nchunks = (p->Cin + C::KC - 1) / C::KC;
    constexpr int PSTRIDE = C::NT / (C::KC / 4);
    g.dpp_row = PSTRIDE / W;
    g.dpp_x = PSTRIDE % W;
    const size_t smem = (size_t)C::KC * plane * 4 + (size_t)C::WS_U4 * 16;
    if (smem > 227 * 1024) return fail(SBNN_ERR_UNSUPPORTED, "3x3 tile for W=%d needs %zu bytes of shared memory", W, smem);

    // the stream's plane offsets depend on the plane size, hence on (W, tile shape)
    const Stream3x3* sp = nullptr;
    {
        std::lock_guard<std::mutex> lk(p->mu);
        const int key = (plane << 8) | (C::GT << 4) | (C::KC / 4);
        auto it = p->streams3x3.find(key);
        if (it == p->streams3x3.end()) {
            Stream3x3 built;
            sbnn_status r = build_stream3(p, C::GT, C::KC, plane, &built);
            if (r != SBNN_OK) return r;
            it = p->streams3x3.emplace(key, std::move(built)).first;
        }
        sp = &it->second;   // map nodes stay where they are until the layer is freed
    }
    const Stream3x3& s = *sp;
    if (s.max_blk > C::WS_U4) return fail(SBNN_ERR_UNSUPPORTED, "internal: 3x3 weight block %d exceeds buffer %d", s.max_blk, C::WS_U4);
    sbnn_status ra = set_max_dyn_smem(reinterpret_cast<const void*>(&conv3x3_gs_kernel<C>), (int)smem);
    if (ra != SBNN_OK) return ra;
    if (prepare_only()) return SBNN_OK;
    const long long NH = (long long)N * H;
    dim3 grid((unsigned)((NH + g.R - 1) / g.R), s.ntiles);
    conv3x3_gs_kernel<C><<<grid, C::NT, smem, st>>>(x, y, p->d_bias, s.rec, s.blk_ptr, g, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

// Pitch for the channel-major variant: a multiple of 4 (16-byte aligned row pieces), >= LPR*CW + 5, and such
// that the first reads of the 32 lanes fall into 32 distinct banks if possible.
int pick_pitch4(int LPR, int CW, int RPL = 1) {
    // Fewest lanes on the busiest bank; ties go to the smaller pitch.  (With few lanes per row a warp spans many rows,
    // whose offsets are multiples of the pitch: no multiple of 4 spreads them over 32 banks, but the choice still
    // matters: a pitch of 16 with two rows per lane puts all 32 lanes on one bank, 20 on four.)
    const int lo = (LPR * CW + 5 + 3) / 4 * 4;
    int best = lo, best_worst = 33;
    for (int p = lo; p < lo + 128; p += 4) {
        int count[32] = {0};
        int worst = 0;
        for (int l = 0; l < 32; ++l) worst = std::max(worst, ++count[((l / LPR) * RPL * p + (l % LPR) * CW) & 31]);
        if (worst < best_worst) {
            best_worst = worst;
            best = p;
        }
        if (worst == 1) break;
    }
    return best;
}

// Launches the channel-major variant; *done = false (and SBNN_OK) if the shape does not fit it.
template <class C>
sbnn_status launch3_cm(const sbnn_packed* p, const float* xt, int ldx, float* y, int N, int H, int W, int relu,
                       cudaStream_t st, bool* done) {
    *done = false;
    Geo3 g;
    g.N = N; g.H = H; g.W = W; g.Cin = p->Cin; g.Cout = p->Cout; g.ngroups = p->ngroups;
    g.LPR = lanes_per_row(W, C::CW);
    g.RPW = 32 / g.LPR;
    g.R = C::NPW * g.RPW;
    g.pitch = pick_pitch4(g.LPR, C::CW);
    const int plane = ((g.R + 3) * g.pitch + 7) / 8 * 8 + 4;   // multiple of 4 floats
    g.plane = plane;
    g.nchunks = (p->Cin + C::KC - 1) / C::KC;
    g.dpp_row = g.dpp_x = 0;
    const size_t smem = (size_t)2 * C::KC * plane * 4 + (size_t)2 * C::WS_U4 * 16;
    const long long pieces = (long long)(g.R + 2) * (W / 4);
    if (smem > 227 * 1024 || pieces > 2LL * C::NT || (long long)N * H * W * 1 > 0x7fffffffLL / 2) return SBNN_OK;
    const Stream3x3* sp = nullptr;
    {
        std::lock_guard<std::mutex> lk(p->mu);
        const int key = (plane << 8) | (C::GT << 4) | (C::KC / 4);
        auto it = p->streams3x3.find(key);
        if (it == p->streams3x3.end()) {
            Stream3x3 built;
            sbnn_status r = build_stream3(p, C::GT, C::KC, plane, &built);
            if (r != SBNN_OK) return r;
            it = p->streams3x3.emplace(key, std::move(built)).first;
        }
        sp = &it->second;   // map nodes stay where they are until the layer is freed
    }
    const Stream3x3& s = *sp;
    if (s.max_blk > C::WS_U4) return fail(SBNN_ERR_UNSUPPORTED, "internal: 3x3 weight block %d exceeds buffer %d", s.max_blk, C::WS_U4);
    sbnn_status ra = set_max_dyn_smem(reinterpret_cast<const void*>(&conv3x3_gs_cm_kernel<C>), (int)smem);
    if (ra != SBNN_OK) return ra;
    if (prepare_only()) {
        *done = true;
        return SBNN_OK;
    }
    const long long NH = (long long)N * H;
    dim3 grid((unsigned)((NH + g.R - 1) / g.R), s.ntiles);
    conv3x3_gs_cm_kernel<C><<<grid, C::NT, smem, st>>>(xt, ldx, y, p->d_bias, s.rec, s.blk_ptr, g, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    *done = true;
    return SBNN_OK;
}

// Launches the copy-engine variant; *done = false (and SBNN_OK) if the shape does not fit it.
template <class C>
sbnn_status launch3_tma(const sbnn_packed* p, const float* xt, long long ldx, int row_pitch, float* y, int ldy, bool out_cm, int N,
                        int H, int W, int relu, cudaStream_t st, unsigned char* extra, size_t extra_bytes, bool* done) {
    *done = false;
    Geo3 g;
    g.N = N; g.H = H; g.W = W; g.Cin = p->Cin; g.Cout = p->Cout; g.ngroups = p->ngroups;
    g.LPR = lanes_per_row(W, C::CW);
    g.RPW = 32 / g.LPR;
    g.R = C::NPW * g.RPW * C::RPL;
    g.pitch = pick_pitch4(g.LPR, C::CW, C::RPL);
    g.plane = (g.R + 2) * g.pitch;                                 // the copied box: no padding between planes
    if (H % C::RPL) return SBNN_OK;                                // a lane's rows must lie in one image
    g.nchunks = (p->Cin + C::KC - 1) / C::KC;
    g.dpp_row = g.dpp_x = 0;
    if (g.pitch > 256 || g.R + 2 > 256 || row_pitch % 4 || ldx % 4) return SBNN_OK;   // rows and planes start on 16-byte boundaries
    const bool pat = use_tap_lists(p);       // packed with kernel patterns: the kernel walks a list of kept taps
    if (pat && (long long)C::KC * g.plane + 2LL * g.pitch + 2 >= (1LL << 30)) return SBNN_OK;
    const int ws_u4 = pat ? C::WS_U4_TAPS : C::WS_U4;
    const int stage_bytes = (C::KC * g.plane * 4 + ws_u4 * 16 + 127) / 128 * 128;
    const size_t tail = (size_t)2 * 3 * 8 + 16 + (size_t)g.pitch * 4;
    int S = 3;
    while (S > 1 && (size_t)S * stage_bytes + tail > 227 * 1024) --S;   // (one stage: copy and arithmetic take turns; narrow maps with many rows per warp)
    const size_t smem = (size_t)S * stage_bytes + tail;
    if (smem > 227 * 1024) return SBNN_OK;
    const long long NH = (long long)N * H;
    const int nrow = (int)((NH + g.R - 1) / g.R);
    const Stream3x3* sp = nullptr;
    Plan3x3 plan;
    {
        std::lock_guard<std::mutex> lk(p->mu);
        const int key = (g.plane << 8) | (C::GT << 4) | (C::KC / 4) | (pat ? (1 << 30) : 0);
        auto it = p->streams3x3.find(key);
        if (it == p->streams3x3.end()) {
            Stream3x3 built;
            sbnn_status r = pat ? build_stream3_taps(p, C::GT, C::KC, g.plane, g.pitch, &built) : build_stream3(p, C::GT, C::KC, g.plane, &built);
            if (r != SBNN_OK) return r;
            it = p->streams3x3.emplace(key, std::move(built)).first;
        }
        sp = &it->second;   // map nodes stay where they are until the layer is freed
        const int ncta = sm_count3();
        const long long pkey = ((long long)key << 32) | ((long long)(nrow & 0xFFFFF) << 12) | (long long)(ncta & 0xFFF);
        auto ip = p->plans3x3.find(pkey);
        if (ip == p->plans3x3.end()) {
            Plan3x3 built;
            sbnn_status r = build_plan3(*sp, nrow, ncta, &built);
            if (r != SBNN_OK) return r;
            ip = p->plans3x3.emplace(pkey, built).first;
        }
        plan = ip->second;
    }
    const Stream3x3& s = *sp;
    if (s.max_blk > ws_u4) return fail(SBNN_ERR_UNSUPPORTED, "internal: 3x3 weight block %d exceeds buffer %d", s.max_blk, ws_u4);
    constexpr bool kTapLists = C::RPL == 1;                        // instances with several rows per lane have no tap-list form
    if (pat && !kTapLists) return SBNN_OK;
    using CP = K3<C::G, C::CW, C::GPW, C::NPW, C::NGW, C::KC, 1>;  // == C wherever the tap-list kernel is launched
    sbnn_status r = set_max_dyn_smem(pat ? reinterpret_cast<const void*>(&conv3x3_gs_tma_kernel<CP, true, false>)
                                         : reinterpret_cast<const void*>(&conv3x3_gs_tma_kernel<C, false, false>), (int)smem);
    if (r == SBNN_OK)
        r = set_max_dyn_smem(pat ? reinterpret_cast<const void*>(&conv3x3_gs_tma_kernel<CP, true, true>)
                                 : reinterpret_cast<const void*>(&conv3x3_gs_tma_kernel<C, false, true>), (int)smem);
    if (r != SBNN_OK) return r;
    int* status = nullptr;
    if ((r = async_status_word(&status)) != SBNN_OK) return r;
    if (prepare_only()) {
        *done = true;
        return SBNN_OK;
    }
    // partial sums of the split tiles and their arrival counters, behind the planes of X in the scratch buffer
    constexpr size_t slot_bytes = (size_t)C::GPW * C::RPL * C::CW * ((C::G + 1) / 2) * C::NT * sizeof(f32x2);
    const size_t counters_off = (plan.nslots * slot_bytes + 255) / 256 * 256;
    if (counters_off + (size_t)plan.ncounters * 4 > extra_bytes)
        return fail(SBNN_ERR_UNSUPPORTED, "internal: 3x3 launch plan needs %zu bytes of scratch, %zu reserved",
                    counters_off + (size_t)plan.ncounters * 4, extra_bytes);
    f32x2* partial = reinterpret_cast<f32x2*>(extra);
    int* counters = reinterpret_cast<int*>(extra + counters_off);
    if (plan.ncounters) SBNN_CUDA_TRY(cudaMemsetAsync(counters, 0, (size_t)plan.ncounters * 4, st));
    Map3 xmap;
    const unsigned long long dims[3] = {(unsigned long long)W, (unsigned long long)NH, (unsigned long long)p->Cin};
    const unsigned long long strides[2] = {(unsigned long long)row_pitch * 4, (unsigned long long)ldx * 4};
    const unsigned box[3] = {(unsigned)g.pitch, (unsigned)(g.R + 2), (unsigned)C::KC};
    if ((r = encode_tiled_map(&xmap, xt, 4, 3, dims, strides, box)) != SBNN_OK) return r;
    const Seg3* segs = static_cast<const Seg3*>(plan.segs);
#define SBNN_L3(KCFG, PATF, CMF)                                                                                              \
    conv3x3_gs_tma_kernel<KCFG, PATF, CMF><<<plan.ncta, C::NT + 32, smem, st>>>(xmap, y, p->d_bias, s.rec, s.blk_ptr, g, relu, S, \
                                                                               stage_bytes, status, plan.cta_ptr, segs, partial, \
                                                                               counters, ldy)
    if (pat) {
        if (out_cm) SBNN_L3(CP, true, true); else SBNN_L3(CP, true, false);
    } else {
        if (out_cm) SBNN_L3(C, false, true); else SBNN_L3(C, false, false);
    }
#undef SBNN_L3
    SBNN_CUDA_TRY(cudaGetLastError());
    *done = true;
    return SBNN_OK;
}

template <int CW>
sbnn_status dispatch3_tma(const sbnn_packed* p, const float* xt, long long ldx, int row_pitch, float* y, int ldy, bool out_cm, int N,
                          int H, int W, int relu, cudaStream_t st, unsigned char* extra, size_t extra_bytes, bool* done) {
    // two output rows per lane where the image height allows it (whole-kernel layers; the tap lists keep one)
    const bool two_rows = H % 2 == 0 && !use_tap_lists(p);
    switch (p->G) {
        case 1:
            if (two_rows) return launch3_tma<K3<1, CW, 2, 3, 4, 8, 2>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
            return launch3_tma<K3<1, CW, 4, 7, 2, 8>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
        case 2:
            if (two_rows) return launch3_tma<K3<2, CW, 2, 3, 4, 8, 2>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
            return launch3_tma<K3<2, CW, 4, 7, 2, 8>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
        case 4:
            if (two_rows) {
                // 2 row warps x 6 group warps with 16-channel steps is about 6 % faster per group than 3 x 4 with
                // 8-channel steps (half the steps, lists twice as long); it wins unless the last tile of six groups is
                // mostly empty.  Falls back to 3 x 4 when two stages of the larger tile do not fit.
                const int ng = p->ngroups;
                if ((ng + 5) / 6 * 6 * 0.94 < (ng + 3) / 4 * 4) {
                    sbnn_status r = launch3_tma<K3<4, CW, 1, 2, 6, 16, 2>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
                    if (r != SBNN_OK || *done) return r;
                }
                return launch3_tma<K3<4, CW, 1, 3, 4, 8, 2>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
            }
            {
                // one row per lane (tap lists, odd heights): one group per warp on 3 x 4 warps with 16-channel steps
                // (four-tap pattern layer of config 4's shape: 263 -> 220 us against two groups per warp on 7 x 2 warps)
                sbnn_status r = launch3_tma<K3<4, CW, 1, 3, 4, 16>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
                if (r != SBNN_OK || *done) return r;
            }
            return launch3_tma<K3<4, CW, 2, 7, 2, 8>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
        case 8: {
            // one row per lane (two would need 112 accumulators); 16-channel steps on 12 warps measured 8 % faster than
            // 8-channel steps on 14 (config 4's shape with G = 8: 339 -> 311 us), tiles of six groups where they fit
            sbnn_status r;
            if ((p->ngroups + 5) / 6 * 6 * 0.94 < (p->ngroups + 3) / 4 * 4)
                r = launch3_tma<K3<8, CW, 1, 2, 6, 16>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
            else
                r = launch3_tma<K3<8, CW, 1, 3, 4, 16>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
            if (r != SBNN_OK || *done) return r;
            return launch3_tma<K3<8, CW, 1, 7, 2, 8>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
        }
        default: return launch3_tma<K3<16, CW, 1, 7, 1, 8>>(p, xt, ldx, row_pitch, y, ldy, out_cm, N, H, W, relu, st, extra, extra_bytes, done);
    }
}

// Scratch the copy-engine kernel may need beyond the planes of X: every CTA border splits at most one tile, so there are
// at most 2 * CTAs partial-sum slots (NT threads x GPW * CW * G sums: at most 448 * 8 * CW floats in every instance
// above) and as many counters.
size_t tma_extra_bytes(int cw) {
    const size_t sms = (size_t)sm_count3();
    return 2 * sms * (size_t)448 * 8 * cw * sizeof(float) + 256 + 2 * sms * sizeof(int);
}

template <int CW>
sbnn_status dispatch3_cm(const sbnn_packed* p, const float* xt, int ldx, float* y, int N, int H, int W, int relu,
                         cudaStream_t st, bool* done) {
    switch (p->G) {
        case 1: return launch3_cm<K3<1, CW, 4, 7, 2, 8>>(p, xt, ldx, y, N, H, W, relu, st, done);
        case 2: return launch3_cm<K3<2, CW, 4, 7, 2, 8>>(p, xt, ldx, y, N, H, W, relu, st, done);
        case 4: return launch3_cm<K3<4, CW, 2, 7, 2, 8>>(p, xt, ldx, y, N, H, W, relu, st, done);
        case 8: return launch3_cm<K3<8, CW, 1, 7, 2, 8>>(p, xt, ldx, y, N, H, W, relu, st, done);
        default: return launch3_cm<K3<16, CW, 1, 7, 1, 8>>(p, xt, ldx, y, N, H, W, relu, st, done);
    }
}

// Column width per lane: the one that tiles the row with least waste (ties go to 8).
int choose_cw(int W) {
    const int l7 = lanes_per_row(W, 7), l8 = lanes_per_row(W, 8);
    if (!l7 && !l8) return 0;
    if (!l7) return 8;
    if (!l8) return 7;
    return (l7 * 7 < l8 * 8) ? 7 : 8;
}

template <int CW>
sbnn_status dispatch3(const sbnn_packed* p, const float* x, float* y, int N, int H, int W, int relu, cudaStream_t st) {
    switch (p->G) {
        case 1: return launch3<K3<1, CW, 4, 7, 2, 8>>(p, x, y, N, H, W, relu, st);
        case 2: return launch3<K3<2, CW, 4, 7, 2, 8>>(p, x, y, N, H, W, relu, st);
        case 4: return launch3<K3<4, CW, 2, 7, 2, 8>>(p, x, y, N, H, W, relu, st);
        case 8: return launch3<K3<8, CW, 1, 7, 2, 8>>(p, x, y, N, H, W, relu, st);
        default: return launch3<K3<16, CW, 1, 7, 1, 8>>(p, x, y, N, H, W, relu, st);
    }
}
}  // namespace

sbnn_status prepare_default_3x3(const sbnn_packed*) { return SBNN_OK; }  // the re-layout depends on the image width

void free_streams_3x3(sbnn_packed* p) {
    for (auto& kv : p->streams3x3) {
        cudaFree(kv.second.rec);
        cudaFree(kv.second.blk_ptr);
    }
    p->streams3x3.clear();
    for (auto& kv : p->plans3x3) {
        cudaFree(kv.second.cta_ptr);
        cudaFree(kv.second.segs);
    }
    p->plans3x3.clear();
}

}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_conv3x3_gs(const sbnn_packed* w, const float* x_dev, float* y_dev, int N, int H, int W,
                                       int flags, void* cuda_stream) {
    clear_error();
    if (!w || !x_dev || !y_dev) return fail(SBNN_ERR_NULL, "packed weights, x_dev and y_dev must not be NULL");
    if (w->KH != 3 || w->KW != 3) return fail(SBNN_ERR_SHAPE, "packed layer is %dx%d, expected 3x3", w->KH, w->KW);
    if (N < 0 || H < 0 || W < 0) return fail(SBNN_ERR_SHAPE, "negative activation shape %dx%dx%d", N, H, W);
    if ((int64_t)N * H * W > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "N*H*W exceeds 2^31-1");
    if (flags & ~SBNN_RELU) return fail(SBNN_ERR_UNSUPPORTED, "flag bits 0x%x not accepted by the 3x3 kernel", flags);
    if (!aligned16(x_dev) || !aligned16(y_dev)) return fail(SBNN_ERR_ALIGN, "x_dev and y_dev must be 16-byte aligned");
    if (w->Cin % 4) return fail(SBNN_ERR_UNSUPPORTED, "Cin=%d is not a multiple of 4", w->Cin);
    if ((int64_t)N * H * W == 0) return SBNN_OK;
    const int cw = choose_cw(W);
    if (!cw) return fail(SBNN_ERR_UNSUPPORTED, "W=%d: the 3x3 kernel handles rows of at most 256 pixels", W);
    sbnn_status st = check_packed_device(w);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    {
        // fast path: planes of the input in the per-device scratch buffer ([Cin][N*H][Wp], rows padded to a multiple of
        // 4 floats), then the copy-engine kernel
        const int M = N * H * W, Wp = (W + 3) / 4 * 4;
        const long long ld = (long long)N * H * Wp;
        float* xt = nullptr;
        const size_t xt_bytes = ((size_t)w->Cin * ld * sizeof(float) + 255) / 256 * 256, extra_bytes = tma_extra_bytes(cw);
        if ((st = scratch_workspace(xt_bytes + extra_bytes, s, &xt)) != SBNN_OK) return st;
        if (!prepare_only()) {
            if (Wp == W) {
                if ((st = launch_transpose(x_dev, w->Cin, xt, (int)ld, M, w->Cin, s)) != SBNN_OK) return st;
            } else {
                dim3 grid((M + 31) / 32, (w->Cin + 31) / 32);
                to_padded_planes_kernel<<<grid, 256, 0, s>>>(x_dev, xt, M, w->Cin, W, Wp, ld);
                SBNN_CUDA_TRY(cudaGetLastError());
            }
        }
        unsigned char* extra = reinterpret_cast<unsigned char*>(xt) + xt_bytes;
        bool done = false;
        st = cw == 7 ? dispatch3_tma<7>(w, xt, ld, Wp, y_dev, w->Cout, false, N, H, W, flags & SBNN_RELU, s, extra, extra_bytes, &done)
                     : dispatch3_tma<8>(w, xt, ld, Wp, y_dev, w->Cout, false, N, H, W, flags & SBNN_RELU, s, extra, extra_bytes, &done);
        if (st != SBNN_OK || done) return st;
        if (Wp == W && ld <= 0x7fffffffLL) {
            st = cw == 7 ? dispatch3_cm<7>(w, xt, (int)ld, y_dev, N, H, W, flags & SBNN_RELU, s, &done)
                         : dispatch3_cm<8>(w, xt, (int)ld, y_dev, N, H, W, flags & SBNN_RELU, s, &done);
            if (st != SBNN_OK || done) return st;
        }
    }
    return cw == 7 ? dispatch3<7>(w, x_dev, y_dev, N, H, W, flags & SBNN_RELU, s)
                   : dispatch3<8>(w, x_dev, y_dev, N, H, W, flags & SBNN_RELU, s);
}

extern "C" sbnn_status sbnn_debug_plan_conv3x3(const int32_t* block_ptr, int ntiles, int nchunks, int nrow, int ncta,
                                               int32_t* cta_ptr_out, int32_t* segs_out, int seg_capacity, int* nsegs,
                                               int* nslots, int* ncounters) {
    clear_error();
    if (!block_ptr || !cta_ptr_out || !segs_out || !nsegs) return fail(SBNN_ERR_NULL, "block_ptr, cta_ptr_out, segs_out and nsegs must not be NULL");
    if (ntiles < 1 || nchunks < 1 || nrow < 1 || ncta < 1 || seg_capacity < 0) return fail(SBNN_ERR_SHAPE, "ntiles, nchunks, nrow and ncta must be positive");
    for (int t = 0; t < ntiles; ++t)
        for (int k = 0; k < nchunks; ++k)
            if (block_ptr[(size_t)t * (nchunks + 1) + k + 1] < block_ptr[(size_t)t * (nchunks + 1) + k])
                return fail(SBNN_ERR_SHAPE, "block_ptr must not decrease inside a tile");
    Plan3Host h;
    try {
        plan3_host(block_ptr, ntiles, nchunks, nrow, ncta, &h);
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory planning the 3x3 launch");
    }
    *nsegs = (int)h.segs.size();
    if (nslots) *nslots = h.nslots;
    if (ncounters) *ncounters = h.ncounters;
    if ((int)h.segs.size() > seg_capacity) return fail(SBNN_ERR_SHAPE, "%zu segments do not fit seg_capacity=%d", h.segs.size(), seg_capacity);
    for (int c = 0; c <= h.ncta; ++c) cta_ptr_out[c] = h.cta_ptr[c];
    for (int c = h.ncta + 1; c <= ncta; ++c) cta_ptr_out[c] = h.cta_ptr[h.ncta];
    static_assert(sizeof(Seg3) == 8 * sizeof(int32_t), "Seg3 is eight ints");
    if (!h.segs.empty()) memcpy(segs_out, h.segs.data(), h.segs.size() * sizeof(Seg3));
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_conv3x3_gs_cm(const sbnn_packed* w, const float* xt_dev, int ldx, float* y_dev, int ldy, int N, int H,
                                          int W, int flags, void* cuda_stream) {
    clear_error();
    if (!w || !xt_dev || !y_dev) return fail(SBNN_ERR_NULL, "packed weights, xt_dev and y_dev must not be NULL");
    if (w->KH != 3 || w->KW != 3) return fail(SBNN_ERR_SHAPE, "packed layer is %dx%d, expected 3x3", w->KH, w->KW);
    if (N < 0 || H < 0 || W < 0) return fail(SBNN_ERR_SHAPE, "negative activation shape %dx%dx%d", N, H, W);
    if ((int64_t)N * H * W > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "N*H*W exceeds 2^31-1");
    if (flags & ~(SBNN_RELU | SBNN_OUT_CM)) return fail(SBNN_ERR_UNSUPPORTED, "flag bits 0x%x not accepted here", flags);
    const bool out_cm = (flags & SBNN_OUT_CM) != 0;
    const long long M = (long long)N * H * W;
    if (ldx < M || ldx % 4) return fail(SBNN_ERR_SHAPE, "ldx=%d must be >= N*H*W=%lld and a multiple of 4", ldx, M);
    if (out_cm ? (ldy < M) : (ldy < w->Cout || ldy % 4))
        return fail(SBNN_ERR_SHAPE, "ldy=%d does not fit the output layout", ldy);
    if (!aligned16(xt_dev) || !aligned16(y_dev)) return fail(SBNN_ERR_ALIGN, "xt_dev and y_dev must be 16-byte aligned");
    if (w->Cin % 4) return fail(SBNN_ERR_UNSUPPORTED, "Cin=%d is not a multiple of 4", w->Cin);
    if (M == 0) return SBNN_OK;
    const int cw = choose_cw(W);
    if (!cw) return fail(SBNN_ERR_UNSUPPORTED, "W=%d: the 3x3 kernel handles rows of at most 256 pixels", W);
    if (w->Cin > 65535) return fail(SBNN_ERR_SHAPE, "too many input channels");
    sbnn_status st = check_packed_device(w);
    if (st != SBNN_OK) return st;
    if ((st = check_device()) != SBNN_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // Widths that are not multiples of 4: the rows of the planes do not start on 16-byte boundaries, which the tiled
    // copy needs, so the planes are first copied into the scratch buffer with padded rows.
    const int Wp = (W + 3) / 4 * 4;
    const long long rows = (long long)N * H, ldp = rows * Wp;
    const size_t pad_bytes = Wp == W ? 0 : ((size_t)w->Cin * ldp * sizeof(float) + 255) / 256 * 256;
    float* scratch = nullptr;
    const size_t extra_bytes = tma_extra_bytes(cw);
    if ((st = scratch_workspace(pad_bytes + extra_bytes, s, &scratch)) != SBNN_OK) return st;
    const float* planes = xt_dev;
    long long ldplanes = ldx;
    if (Wp != W) {
        if (!prepare_only()) {
            dim3 grid((unsigned)((M + 255) / 256), (unsigned)w->Cin);
            pad_plane_rows_kernel<<<grid, 256, 0, s>>>(xt_dev, ldx, scratch, ldp, rows, W, Wp);
            SBNN_CUDA_TRY(cudaGetLastError());
        }
        planes = scratch;
        ldplanes = ldp;
    }
    bool done = false;
    unsigned char* extra = reinterpret_cast<unsigned char*>(scratch) + pad_bytes;
    st = cw == 7 ? dispatch3_tma<7>(w, planes, ldplanes, Wp, y_dev, ldy, out_cm, N, H, W, flags & SBNN_RELU, s, extra, extra_bytes, &done)
                 : dispatch3_tma<8>(w, planes, ldplanes, Wp, y_dev, ldy, out_cm, N, H, W, flags & SBNN_RELU, s, extra, extra_bytes, &done);
    if (st != SBNN_OK || done) return st;
    return fail(SBNN_ERR_UNSUPPORTED, "the pipelined 3x3 kernel does not take this shape (rows of %d pixels; it stages rows of at most 224)", W);
}
