// bf16 tensor-core mode of the group-sparse 1x1 convolution (flag SBNN_BF16_TC).
//
// Activations and kept weights are rounded to bf16 (round to nearest even), products are exact in
// fp32 and accumulate in fp32 inside the tensor core; bias and ReLU stay fp32.
//
// Per group the work is a dense contraction  Y_g[pixels x G] = Xg[pixels x K'] * Wg[K' x G]  whose A
// operand is a *gather* of K' channel rows.  The 5th-generation tensor-core path (tcgen05) reads its
// operands from shared memory in fixed canonical layouts, so a per-channel gather would first have
// to be copied into such a layout, which costs the shared-memory traffic the FFMA kernel already
// pays.  The warp-level path does not have that restriction: ldmatrix takes one address per 8x8
// sub-matrix row, and in the [channel][pixel] tile a sub-matrix row is 8 consecutive pixels of one
// (arbitrary) channel.  So one `ldmatrix.x4.trans` with gathered row addresses yields the 16x16 A
// fragment of an m16n8k16 MMA at 4 shared-memory wavefronts per 2048 MACs, against 9 per 1024 in
// the fp32 kernel.  The N = 8 columns of the MMA are the group's output channels (G = 8 fills them,
// G = 16 takes two MMAs per A fragment, smaller groups are merged into 8-column groups at pack time).
//
// CTA = 128 pixels x 8 warps; a warp owns GPW groups over all 128 pixels (8 row blocks of 16), i.e.
// 32 fp32 accumulators per N-tile.  A pre-pass converts X once to bf16 in channel-major order
// ([Cin][ld], pixels contiguous); a ninth warp then fills the [channel][pixel] tile of every channel
// step with one tiled tensor-map copy (plus a linear copy of the step's weight block) onto a "full"
// mbarrier, and the MMA warps hand a stage back through an "empty" mbarrier, so no CTA-wide barrier
// makes warps with fewer kept channels in a step wait for the others (two stages, bounded waits).  The
// weight stream holds, per 16 kept channels, 16 row offsets and the B fragments in register order.
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "common.h"
#include "pipeline.cuh"

namespace sbnn {
namespace {

constexpr int TM = 128;                    // pixels per CTA
constexpr int KC = 64;                     // channels per step
constexpr int ROWB = TM * 2 + 16;          // bytes per channel row (+16: spreads rows over bank groups)
constexpr int NWARP = 8;

struct StreamBf16 {
    uint4* rec = nullptr;
    int32_t* blk_ptr = nullptr;
    int ntiles = 0, nchunks = 0, max_blk = 0, GT = 0;
};

template <int NT8>   // N-tiles of 8 output channels per group (1 for G <= 8, 2 for G = 16)
struct KB {
    static constexpr int BLK = 4 + NT8 * 16;   // one 16-channel block: 16 offsets + B fragments, 16-byte units
};

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct MapB { alignas(64) unsigned char bytes[128]; };

constexpr int STAGE_X = KC * ROWB;         // bytes of activations per stage (a multiple of 128)

template <int G, int GPW>
__global__ void __launch_bounds__((NWARP + 1) * 32)
conv1x1_bf16_kernel(const __grid_constant__ MapB xmap, float* __restrict__ Y, const float* __restrict__ bias,
                    const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr, int M, int Cin, int Cout,
                    int ngroups, int nchunks, int ntiles, int ws_u4, int S, int stage_bytes, int relu, int* status) {
    constexpr int NT8 = (G + 7) / 8;
    constexpr int GT = NWARP * GPW;
    extern __shared__ __align__(128) unsigned char smem[];
    // S stages of [KC][ROWB] activations + the step's weight block, then the stages' "full" and "empty" mbarriers
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)S * stage_bytes);
    uint64_t* empty = full + S;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + S);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x % ntiles;
    const int m0 = (blockIdx.x / ntiles) * TM;
    const int32_t* bp = blk_ptr + (size_t)tile * (nchunks + 1);
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, NWARP);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == NWARP) {
        // producer warp: per channel step one tiled copy of the [KC][TM + 8] box of X (the 8 extra pixels are the row
        // padding that spreads the rows over the banks; channels past Cin and pixels past the tensor arrive as zeros)
        // and one linear copy of the step's weight block, both onto the stage's "full" barrier
        bool ok = true;
        int k = 0;
        for (; k < nchunks && ok; ++k) {
            const int s = k % S;
            if (k >= S) ok = mbar_wait(empty + s, ((k / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT);
            if (!ok) break;
            if (lane == 0) {
                const int beg = bp[k], n = bp[k + 1] - beg;
                unsigned char* st = smem + (size_t)s * stage_bytes;
                mbar_arrive_expect_tx(full + s, (uint32_t)STAGE_X + (uint32_t)n * 16u);
                tensor_g2s_2d(st, &xmap, m0, k * KC, full + s);
                bulk_g2s(st + STAGE_X, rec + beg, (uint32_t)n * 16u, full + s);
            }
        }
        if (!ok) {   // gave up: let the copies already issued land before the CTA's shared memory is released
            for (int j = max(0, k - S); j < k; ++j) {
                bool landed = false;
                for (uint32_t i = 0; i < kWaitLimit && !landed; ++i) landed = mbar_try_wait(full + j % S, (j / S) & 1);
            }
        }
        return;
    }

    const int gq = lane >> 2, tq = lane & 3;

    float acc[GPW][NT8][8][4];
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * GT + warp * GPW + q;
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            const int c0 = n * 8 + 2 * tq;
            const float b0 = (g < ngroups && c0 < G && g * G + c0 < Cout) ? bias[g * G + c0] : 0.f;
            const float b1 = (g < ngroups && c0 + 1 < G && g * G + c0 + 1 < Cout) ? bias[g * G + c0 + 1] : 0.f;
#pragma unroll
            for (int pb = 0; pb < 8; ++pb) {
                acc[q][n][pb][0] = b0; acc[q][n][pb][1] = b1; acc[q][n][pb][2] = b0; acc[q][n][pb][3] = b1;
            }
        }
    }
    // ldmatrix: lane l addresses row (l & 7) of sub-matrix (l >> 3): channels 8*(l>>4) + (l&7), pixels 8*((l>>3)&1)..
    const int off_idx = 8 * (lane >> 4) + (lane & 7);
    const uint32_t xs_base = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + ((lane >> 3) & 1) * 16;

    for (int k = 0; k < nchunks; ++k) {
        const int s = k % S;
        if (!mbar_wait(full + s, (k / S) & 1, abort_flag, status, SBNN_ERR_TIMEOUT)) return;
        const uint4* ws = reinterpret_cast<const uint4*>(smem + (size_t)s * stage_bytes + STAGE_X);
        const uint32_t xs_lane = xs_base + s * stage_bytes;
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int2 hd = reinterpret_cast<const int2*>(ws)[warp * GPW + q];   // (start, 16-channel blocks)
            const uint4* r = ws + hd.x;
            for (int it = 0; it < hd.y; ++it, r += KB<NT8>::BLK) {
                const uint32_t row = xs_lane + reinterpret_cast<const uint32_t*>(r)[off_idx];
                uint32_t b[NT8][2];
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    const uint2 t = reinterpret_cast<const uint2*>(r + 4 + n * 16)[lane];
                    b[n][0] = t.x; b[n][1] = t.y;
                }
#pragma unroll
                for (int pb = 0; pb < 8; ++pb) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, row + pb * 32);
#pragma unroll
                    for (int n = 0; n < NT8; ++n) mma_bf16(acc[q][n][pb], a, b[n][0], b[n][1]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + s);   // the warp is done with the stage
    }
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * GT + warp * GPW + q;
        if (g >= ngroups) continue;
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            const int c0 = n * 8 + 2 * tq;
            if (c0 >= G) continue;
#pragma unroll
            for (int pb = 0; pb < 8; ++pb)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int m = m0 + pb * 16 + gq + 8 * h;
                    if (m >= M) continue;
                    float v0 = acc[q][n][pb][2 * h], v1 = acc[q][n][pb][2 * h + 1];
                    if (relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
                    const int ch = g * G + c0;                      // merged groups may reach past Cout
                    if (ch >= Cout) continue;
                    float* yp = Y + (size_t)m * Cout + ch;
                    if (G >= 2 && ch + 1 < Cout && (Cout & 1) == 0) {
                        *reinterpret_cast<float2*>(yp) = make_float2(v0, v1);
                    } else {
                        yp[0] = v0;
                        if (G >= 2 && ch + 1 < Cout) yp[1] = v1;
                    }
                }
        }
    }
}

// X [M][C] fp32 (row-major) -> Xb [C][ldb] bf16, round to nearest even; 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256)
to_channel_major_bf16_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ xb, int M, int C, int ldb) {
    __shared__ float t[32][33];
    const int m0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i, c = c0 + tx;
        t[ty + 8 * i][tx] = (m < M && c < C) ? x[(size_t)m * C + c] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, m = m0 + tx;
        if (m < ldb && c < C) xb[(size_t)c * ldb + m] = __float2bfloat16_rn(t[tx][ty + 8 * i]);
    }
}

// ---- host side -------------------------------------------------------------------------------

// fp32 -> bf16 bits, round to nearest even (bf16 is the upper half of an IEEE-754 binary32).
uint16_t bf16_bits(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return (uint16_t)(u >> 16);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// Stream: block (tile t, step k) = GT (start, blocks) pairs, then per group its 16-channel blocks:
// 16 byte offsets of the channels' shared-memory rows, then per N-tile the B fragment of m16n8k16 in
// register order (lane l: {B[2t][g], B[2t+1][g]}, {B[2t+8][g], B[2t+9][g]}, g = l/4, t = l%4).
// The layer as the kernel sees it.  An MMA has 8 output columns, so groups of fewer than 8 channels are merged, 8 / G
// neighbours at a time, into one group of 8 whose kept set is the union of theirs and whose weights are zero where a
// member does not keep the channel: one activation fragment then serves all 8 columns instead of leaving most of
// them as padding (G = 4, dense: half the MMAs and fragment loads).
struct LayerView {
    int G = 0, ngroups = 0;
    std::vector<int32_t> group_ptr, idx;
    std::vector<float> val;
};

LayerView view_for_mma(const sbnn_packed* p) {
    LayerView v;
    if (p->G >= 8) {
        v.G = p->G; v.ngroups = p->ngroups; v.group_ptr = p->group_ptr; v.idx = p->idx; v.val = p->val;
        return v;
    }
    const int G = p->G, per = 8 / G;
    v.G = 8;
    v.ngroups = (p->ngroups + per - 1) / per;
    v.group_ptr.assign(v.ngroups + 1, 0);
    std::vector<int32_t> pos(per);
    for (int sg = 0; sg < v.ngroups; ++sg) {
        const int g0 = sg * per, g1 = std::min(p->ngroups, g0 + per);
        for (int g = g0; g < g1; ++g) pos[g - g0] = p->group_ptr[g];
        for (;;) {                                                   // merge the members' ascending lists
            int32_t c = INT32_MAX;
            for (int g = g0; g < g1; ++g)
                if (pos[g - g0] < p->group_ptr[g + 1]) c = std::min(c, p->idx[pos[g - g0]]);
            if (c == INT32_MAX) break;
            v.idx.push_back(c);
            const size_t base = v.val.size();
            v.val.resize(base + 8, 0.0f);
            for (int g = g0; g < g1; ++g)
                if (pos[g - g0] < p->group_ptr[g + 1] && p->idx[pos[g - g0]] == c) {
                    for (int r = 0; r < G; ++r) v.val[base + (size_t)(g - g0) * G + r] = p->val[(size_t)pos[g - g0] * G + r];
                    ++pos[g - g0];
                }
        }
        v.group_ptr[sg + 1] = (int32_t)v.idx.size();
    }
    return v;
}

sbnn_status build_stream_bf16(const sbnn_packed* pk, StreamBf16* out) {
    LayerView lv;
    try {
        lv = view_for_mma(pk);
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the bf16 weight stream");
    }
    struct { int G, ngroups, Cin; std::vector<int32_t>&group_ptr, &idx; std::vector<float>& val; }
        view{lv.G, lv.ngroups, pk->Cin, lv.group_ptr, lv.idx, lv.val};
    auto* p = &view;
    const int G = p->G, NT8 = (G + 7) / 8, GT = NWARP * (G <= 8 ? 2 : 1), BLK = 4 + NT8 * 16;
    const int ntiles = (p->ngroups + GT - 1) / GT, nchunks = (p->Cin + KC - 1) / KC;
    const int HDR = (GT * 2 + 3) / 4;
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
                    const int nb = (hi - lo + 15) / 16;
                    // Order of the kept channels inside the step: each ldmatrix sub-matrix reads 8 rows at
                    // once, and rows whose channel indices are equal mod 8 fall into the same banks (a row
                    // is 17 x 16 bytes).  So deal the channels out in rounds of 8 with distinct residues,
                    // taking from the fullest residue classes first.  (The sum does not depend on the order
                    // beyond rounding.)
                    std::vector<int> order;
                    {
                        std::vector<int> bucket[8];
                        for (int j = hi - 1; j >= lo; --j) bucket[p->idx[j] & 7].push_back(j);
                        int left = hi - lo;
                        while (left > 0) {
                            int cls[8] = {0, 1, 2, 3, 4, 5, 6, 7};
                            std::sort(cls, cls + 8, [&](int a, int b) { return bucket[a].size() > bucket[b].size(); });
                            for (int i = 0; i < 8 && left > 0; ++i) {
                                if (bucket[cls[i]].empty()) continue;
                                order.push_back(bucket[cls[i]].back());
                                bucket[cls[i]].pop_back();
                                --left;
                            }
                        }
                    }
                    rec[blk_beg * 4 + 2 * s + 0] = (uint32_t)(rec.size() / 4 - blk_beg);
                    rec[blk_beg * 4 + 2 * s + 1] = (uint32_t)nb;
                    for (int b16 = 0; b16 < nb; ++b16) {
                        const size_t base = rec.size();
                        rec.resize(base + (size_t)BLK * 4, 0u);   // padding: row 0, zero weights
                        auto unit = [&](int kk) -> int {
                            const size_t i = (size_t)b16 * 16 + kk;
                            return i < order.size() ? order[i] : -1;
                        };
                        auto wbits = [&](int kk, int col) -> uint32_t {
                            const int j = unit(kk);
                            if (j < 0 || col >= G) return 0u;
                            return bf16_bits(p->val[(size_t)j * G + col]);
                        };
                        for (int kk = 0; kk < 16; ++kk) {
                            const int j = unit(kk);
                            if (j >= 0) rec[base + kk] = (uint32_t)(p->idx[j] - k * KC) * (uint32_t)ROWB;
                        }
                        for (int n = 0; n < NT8; ++n)
                            for (int l = 0; l < 32; ++l) {
                                const int gq = l >> 2, tq = l & 3, col = n * 8 + gq;
                                rec[base + 16 + n * 64 + l * 2 + 0] = wbits(2 * tq, col) | (wbits(2 * tq + 1, col) << 16);
                                rec[base + 16 + n * 64 + l * 2 + 1] = wbits(2 * tq + 8, col) | (wbits(2 * tq + 9, col) << 16);
                            }
                    }
                }
                max_blk = std::max(max_blk, (int)(rec.size() / 4 - blk_beg));
            }
            blk[(size_t)t * (nchunks + 1) + nchunks] = (int32_t)(rec.size() / 4);
        }
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the bf16 weight stream");
    }
    StreamBf16 s;
    s.ntiles = ntiles; s.nchunks = nchunks; s.max_blk = max_blk; s.GT = GT;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s.rec), std::max<size_t>(rec.size() * 4, 16)));
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&s.blk_ptr), blk.size() * 4);
    if (e == cudaSuccess && !rec.empty()) e = cudaMemcpy(s.rec, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s.blk_ptr, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        cudaFree(s.blk_ptr);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the bf16 weight stream: %s", cudaGetErrorString(e));
    }
    *out = s;
    return SBNN_OK;
}

template <int G>
sbnn_status launch_bf16(const sbnn_packed* p, const StreamBf16& s, int ngroups, const float* x, float* y, int M, int relu,
                        cudaStream_t st) {
    constexpr int GPW = (G <= 8) ? 2 : 1;
    // bf16 channel-major copy of X in the per-device scratch buffer; rows padded to whole pixel tiles
    const int ldb = (M + TM - 1) / TM * TM;
    float* scratch = nullptr;
    sbnn_status r = scratch_workspace((size_t)p->Cin * ldb * sizeof(__nv_bfloat16), st, &scratch);
    if (r != SBNN_OK) return r;
    __nv_bfloat16* xb = reinterpret_cast<__nv_bfloat16*>(scratch);
    if (!prepare_only()) {
        dim3 tg((ldb + 31) / 32, (p->Cin + 31) / 32);
        to_channel_major_bf16_kernel<<<tg, 256, 0, st>>>(x, xb, M, p->Cin, ldb);
        SBNN_CUDA_TRY(cudaGetLastError());
    }

    const int stage_bytes = (STAGE_X + s.max_blk * 16 + 127) / 128 * 128;
    // Two stages: with about 38 KB per stage that leaves room for two or three CTAs per SM, which measured faster
    // than one CTA with four stages (config 5, G = 8, dense: 577 us against 722 us).
    const int S = 2;
    const size_t smem = (size_t)S * stage_bytes + 2 * S * 8 + 16;
    if (smem > 200 * 1024) return fail(SBNN_ERR_UNSUPPORTED, "internal: bf16 tile needs %zu bytes of shared memory", smem);
    if ((r = set_max_dyn_smem(reinterpret_cast<const void*>(&conv1x1_bf16_kernel<G, GPW>), (int)smem)) != SBNN_OK) return r;
    if (prepare_only()) return SBNN_OK;
    MapB xmap;
    const unsigned long long dims[2] = {(unsigned long long)ldb, (unsigned long long)p->Cin};
    const unsigned long long strides[1] = {(unsigned long long)ldb * sizeof(__nv_bfloat16)};
    const unsigned box[2] = {(unsigned)(ROWB / 2), (unsigned)KC};
    if ((r = encode_tiled_map(&xmap, xb, 2, 2, dims, strides, box)) != SBNN_OK) return r;
    int* status = nullptr;
    if ((r = async_status_word(&status)) != SBNN_OK) return r;
    const long long nblk = (long long)(ldb / TM) * s.ntiles;
    if (nblk > 0x7fffffffLL) return fail(SBNN_ERR_SHAPE, "too many tiles");
    conv1x1_bf16_kernel<G, GPW><<<(unsigned)nblk, (NWARP + 1) * 32, smem, st>>>(xmap, y, p->d_bias, s.rec, s.blk_ptr, M, p->Cin,
                                                                                p->Cout, ngroups, s.nchunks, s.ntiles, s.max_blk,
                                                                                S, stage_bytes, relu, status);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

}  // namespace

sbnn_status conv1x1_bf16(const sbnn_packed* p, const float* x, float* y, int M, int relu, cudaStream_t st) {
    StreamBf16* s = nullptr;
    {
        std::lock_guard<std::mutex> lk(p->mu);
        if (!p->bf16_stream) {   // first use of the mode on this layer: build the stream (allocates, copies)
            StreamBf16* n = new (std::nothrow) StreamBf16;
            if (!n) return fail(SBNN_ERR_ALLOC, "out of host memory");
            sbnn_status r = build_stream_bf16(p, n);
            if (r != SBNN_OK) {
                delete n;
                return r;
            }
            p->bf16_stream = n;
        }
        s = static_cast<StreamBf16*>(p->bf16_stream);
    }
    switch (p->G) {
        case 16: return launch_bf16<16>(p, *s, p->ngroups, x, y, M, relu, st);
        default: {   // G <= 8: groups merged into groups of 8 output channels (see view_for_mma)
            const int per = 8 / p->G;
            return launch_bf16<8>(p, *s, (p->ngroups + per - 1) / per, x, y, M, relu, st);
        }
    }
}

void free_stream_bf16(sbnn_packed* p) {
    if (!p->bf16_stream) return;
    StreamBf16* s = static_cast<StreamBf16*>(p->bf16_stream);
    cudaFree(s->rec);
    cudaFree(s->blk_ptr);
    delete s;
    p->bf16_stream = nullptr;
}

}  // namespace sbnn
