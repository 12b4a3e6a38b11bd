// Group-sparse 1x1 convolution, fp32 (Algorithm 1 re-thought for sm_100a).
//
//   Y[m][g*G + r] = act( bias[g*G + r] + sum_j val[g][j][r] * X[m][idx[g][j]] ),   m = pixel index in [0, N*H*W)
//
// Work decomposition
//   * A CTA owns TM = 32*P consecutive pixels and GT = NW*GPW consecutive groups and walks the
//     input channels in steps of KC.
//   * Each step the CTA's X tile [TM pixels][KC channels] is read from global memory with
//     128-byte coalesced float4 loads and written to shared memory TRANSPOSED ([channel][pixel]),
//     so that the pixels of one input channel are contiguous.  A lane then fetches the activations
//     of 4 of its pixels with one 128-bit shared load.  The 16-byte slots of a row are XOR-swizzled
//     with (channel/4)%8, which makes both the transposing stores and the row reads bank-conflict
//     free.
//   * A warp owns GPW groups for the whole channel loop and keeps their P x G partial sums per lane
//     in registers.  For every kept (group, channel) unit it issues P/4 128-bit activation loads and
//     one broadcast weight load, then P*G FMAs: one fetched activation feeds the G outputs of the
//     group, the same reuse the paper's NEON tile gets from one input vector (Section 3.3).
//   * Gather indices never reach the inner loop as indices: at pack time every kept unit is turned
//     into the byte offset of its shared-memory row with the swizzle term OR-ed in, so the address
//     of a lane's first float4 is (offset XOR lane*16).  Units are emitted four at a time
//     ("quads": 4 offsets, then 4*G weights); lists are padded with zero-weight units.
//   * Global loads of step k+1 are in flight (registers for X, cp.async for the weight block)
//     while step k is computed; two shared-memory buffers, one barrier per step.
#include <string.h>

#include <algorithm>

#include "common.h"

namespace sbnn {
namespace {

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }

// Packed pair of fp32 values in one 64-bit register; fma2 is two independent fp32 FMAs (round to
// nearest even each) issued as one instruction, which halves the issue slots the FMAs take.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(f32x2& d, f32x2 a, f32x2 b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

template <int G_, int P_, int GPW_, int NW_, int KC_>
struct K1 {
    static constexpr int G = G_, P = P_, GPW = GPW_, NW = NW_, KC = KC_;
    static constexpr int TM = 32 * P, GT = NW * GPW, NT = NW * 32;
    static constexpr int ROW_BYTES = TM * 4;
    static constexpr int XS_BYTES = KC * ROW_BYTES;
    static constexpr int HDR = (GT * 2 + 3) / 4;           // header size, 16-byte units
    static constexpr int QUAD = 1 + G;                     // 4 offsets + 4*G weights, 16-byte units
    static constexpr int WS_U4 = HDR + GT * (KC / 4) * QUAD;
    static constexpr int NLD = (TM / 4) * (KC / 32) / NW;  // float4 global loads per thread and step
    static constexpr size_t SMEM = 2 * (size_t)XS_BYTES + 2 * (size_t)WS_U4 * 16;
    static_assert(P % 4 == 0 && KC % 32 == 0, "tile shape");
    static_assert((TM / 4) * (KC / 32) % NW == 0, "load split");
    static_assert(ROW_BYTES % 512 == 0, "row base must leave bits 4..8 clear");
    static_assert(SMEM <= 227 * 1024, "shared memory");
};

template <int G>
__device__ __forceinline__ void load_unit_weights(const float* wq, int u, float (&w)[G]) {
    if constexpr (G >= 4) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            float4 t = reinterpret_cast<const float4*>(wq)[u * (G / 4) + v];
            w[4 * v + 0] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
        }
    } else if constexpr (G == 2) {
        float2 t = reinterpret_cast<const float2*>(wq)[u];
        w[0] = t.x; w[1] = t.y;
    } else {
        w[0] = wq[u];
    }
}

template <class C>
__global__ void __launch_bounds__(C::NT, 1)
conv1x1_gs_kernel(const float* __restrict__ X, float* __restrict__ Y, const float* __restrict__ bias,
                  const uint4* __restrict__ rec, const int32_t* __restrict__ blk_ptr,
                  int M, int Cin, int Cout, int ngroups, int nchunks, int ntiles, int relu) {
    constexpr int G = C::G, P = C::P, GPW = C::GPW, NW = C::NW, KC = C::KC, TM = C::TM;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* xs0 = smem;  // two X buffers, then two weight buffers
    uint4* ws0 = reinterpret_cast<uint4*>(smem + 2 * C::XS_BYTES);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // group tiles of one pixel tile are neighbours in launch order (they share the tile's activations in L2)
    const int tile = blockIdx.x % ntiles;
    const int m0 = (blockIdx.x / ntiles) * TM;
    const int32_t* bp = blk_ptr + (size_t)tile * (nchunks + 1);

    // acc[q][p2][r] holds pixels (2*p2, 2*p2+1) of the lane for output channel r of group q
    f32x2 acc[GPW][P / 2][G];
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + warp * GPW + q;
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float b = (g < ngroups) ? bias[g * G + r] : 0.0f;
#pragma unroll
            for (int p = 0; p < P / 2; ++p) acc[q][p][r] = pack2(b, b);
        }
    }

    float4 pre[C::NLD];
    auto issue_x_loads = [&](int k) {
#pragma unroll
        for (int t = 0; t < C::NLD; ++t) {
            const int wi = warp + t * NW;
            const int p = (wi / (KC / 32)) * 4 + (lane >> 3);
            const int cq = (wi % (KC / 32)) * 8 + (lane & 7);
            const int m = m0 + p, c = k * KC + cq * 4;
            pre[t] = (m < M && c < Cin) ? __ldg(reinterpret_cast<const float4*>(X + (size_t)m * Cin + c))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto store_x = [&](unsigned char* xs) {
#pragma unroll
        for (int t = 0; t < C::NLD; ++t) {
            const int wi = warp + t * NW;
            const int p = (wi / (KC / 32)) * 4 + (lane >> 3);
            const int cq = (wi % (KC / 32)) * 8 + (lane & 7);
            float* row = reinterpret_cast<float*>(xs + (size_t)(cq * 4) * C::ROW_BYTES) +
                         ((((p >> 2) ^ (cq & 7)) << 2) | (p & 3));
            row[0] = pre[t].x;
            row[TM] = pre[t].y;
            row[2 * TM] = pre[t].z;
            row[3 * TM] = pre[t].w;
        }
    };
    auto issue_w_loads = [&](int k, uint4* ws) {
        const int beg = bp[k], n = bp[k + 1] - beg;
        for (int i = tid; i < n; i += C::NT) cp_async16(ws + i, rec + beg + i);
        cp_async_commit();
    };

    issue_x_loads(0);
    issue_w_loads(0, ws0);
    store_x(xs0);
    cp_async_wait_all();
    __syncthreads();

    const unsigned lane_xor = lane * 16;
    for (int k = 0; k < nchunks; ++k) {
        const int cur = k & 1;
        const bool more = (k + 1 < nchunks);
        if (more) {
            issue_x_loads(k + 1);
            issue_w_loads(k + 1, ws0 + (cur ^ 1) * C::WS_U4);
        }
        const unsigned char* xs = xs0 + cur * C::XS_BYTES;
        const uint4* ws = ws0 + cur * C::WS_U4;
#pragma unroll
        for (int q = 0; q < GPW; ++q) {
            const int2 hd = reinterpret_cast<const int2*>(ws)[warp * GPW + q];  // (start, quads) of this group
            const uint4* r = ws + hd.x;
            for (int it = 0; it < hd.y; ++it, r += C::QUAD) {
                const uint4 off = r[0];
                const float* wq = reinterpret_cast<const float*>(r + 1);
                const unsigned offs[4] = {off.x, off.y, off.z, off.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const unsigned char* ap = xs + (offs[u] ^ lane_xor);
                    ulonglong2 a[P / 4];   // four consecutive pixels = two packed pairs
#pragma unroll
                    for (int i = 0; i < P / 4; ++i) a[i] = *reinterpret_cast<const ulonglong2*>(ap + i * 512);
                    float w[G];
                    load_unit_weights<G>(wq, u, w);
#pragma unroll
                    for (int rr = 0; rr < G; ++rr) {
                        const f32x2 ww = pack2(w[rr], w[rr]);
#pragma unroll
                        for (int i = 0; i < P / 4; ++i) {
                            fma2(acc[q][2 * i][rr], a[i].x, ww);
                            fma2(acc[q][2 * i + 1][rr], a[i].y, ww);
                        }
                    }
                }
            }
        }
        if (more) {
            store_x(xs0 + (cur ^ 1) * C::XS_BYTES);
            cp_async_wait_all();
        }
        __syncthreads();
    }

    // Epilogue: optional ReLU, then each lane writes the G outputs of its pixels.
#pragma unroll
    for (int q = 0; q < GPW; ++q) {
        const int g = tile * C::GT + warp * GPW + q;
        if (g >= ngroups) continue;
#pragma unroll
        for (int i = 0; i < P / 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int m = m0 + i * 128 + lane * 4 + e;
                if (m >= M) continue;
                float* yp = Y + (size_t)m * Cout + g * G;
                float v[G];
#pragma unroll
                for (int rr = 0; rr < G; ++rr) {
                    float lo, hi;
                    unpack2(acc[q][(i * 4 + e) / 2][rr], lo, hi);
                    const float t = (e & 1) ? hi : lo;
                    v[rr] = relu ? fmaxf(t, 0.0f) : t;
                }
                if constexpr (G >= 4) {
#pragma unroll
                    for (int vv = 0; vv < G / 4; ++vv)
                        reinterpret_cast<float4*>(yp)[vv] =
                            make_float4(v[4 * vv], v[4 * vv + 1], v[4 * vv + 2], v[4 * vv + 3]);
                } else if constexpr (G == 2) {
                    *reinterpret_cast<float2*>(yp) = make_float2(v[0], v[1]);
                } else {
                    yp[0] = v[0];
                }
            }
    }
}

// ---- host side -------------------------------------------------------------------------------

// Builds the record stream of one tile configuration from the canonical packed arrays.
// Block (tile t, step k) = header of GT (start, quads) pairs, then every group's quads.
sbnn_status build_stream(const sbnn_packed* p, const TileCfg& c, Stream1x1* out) {
    const int G = p->G, GT = c.GT(), KC = c.KC, TM = c.TM();
    const int ntiles = (p->ngroups + GT - 1) / GT, nchunks = (p->Cin + KC - 1) / KC;
    const int HDR = (GT * 2 + 3) / 4, QUAD = 1 + G;
    std::vector<int32_t> blk((size_t)ntiles * (nchunks + 1));
    std::vector<uint32_t> rec;  // 4 words per 16-byte unit
    int max_blk = 0;
    try {
        rec.reserve(((size_t)p->nnz / 4 + (size_t)ntiles * nchunks * (GT + HDR)) * QUAD * 4);
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
                    const int n = hi - lo, nq = (n + 3) / 4;
                    rec[blk_beg * 4 + 2 * s + 0] = (uint32_t)(rec.size() / 4 - blk_beg);
                    rec[blk_beg * 4 + 2 * s + 1] = (uint32_t)nq;
                    for (int qd = 0; qd < nq; ++qd) {
                        const size_t base = rec.size();
                        rec.resize(base + (size_t)QUAD * 4, 0u);  // zero offsets (row 0) and zero weights
                        for (int u = 0; u < 4; ++u) {
                            const int j = lo + qd * 4 + u;
                            if (j >= hi) break;
                            const int cl = p->idx[j] - k * KC;
                            rec[base + u] = (uint32_t)cl * (uint32_t)(TM * 4) | (uint32_t)(((cl >> 2) & 7) << 4);
                            for (int r = 0; r < G; ++r) {
                                const float w = p->val[(size_t)j * G + r];
                                uint32_t bits;
                                memcpy(&bits, &w, 4);
                                rec[base + 4 + u * G + r] = bits;
                            }
                        }
                    }
                }
                max_blk = std::max(max_blk, (int)(rec.size() / 4 - blk_beg));
            }
            blk[(size_t)t * (nchunks + 1) + nchunks] = (int32_t)(rec.size() / 4);
        }
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the 1x1 weight stream");
    }
    if (rec.size() / 4 > 0x7fffffffull) return fail(SBNN_ERR_UNSUPPORTED, "weight stream too large");
    Stream1x1 s;
    s.ntiles = ntiles; s.nchunks = nchunks; s.max_blk = max_blk;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s.rec), std::max<size_t>(rec.size() * 4, 16)));
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&s.blk_ptr), blk.size() * 4);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        return fail(SBNN_ERR_ALLOC, "cudaMalloc: %s", cudaGetErrorString(e));
    }
    if (!rec.empty()) e = cudaMemcpy(s.rec, rec.data(), rec.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s.blk_ptr, blk.data(), blk.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(s.rec);
        cudaFree(s.blk_ptr);
        return fail(SBNN_ERR_CUDA, "cudaMemcpy: %s", cudaGetErrorString(e));
    }
    *out = s;
    return SBNN_OK;
}

sbnn_status get_stream(const sbnn_packed* p, const TileCfg& c, Stream1x1* out) {
    std::lock_guard<std::mutex> lk(p->mu);
    auto it = p->streams1x1.find(c);
    if (it != p->streams1x1.end()) {
        *out = it->second;
        return SBNN_OK;
    }
    sbnn_status st = build_stream(p, c, out);
    if (st == SBNN_OK) p->streams1x1[c] = *out;
    return st;
}

template <class C>
sbnn_status launch(const sbnn_packed* p, const Stream1x1& s, const float* x, float* y, int M, int relu, cudaStream_t st) {
    static std::mutex mu;
    static std::map<int, bool> configured;  // per device
    {
        std::lock_guard<std::mutex> lk(mu);
        int dev = 0;
        cudaGetDevice(&dev);
        if (!configured[dev]) {
            SBNN_CUDA_TRY(cudaFuncSetAttribute(conv1x1_gs_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM));
            configured[dev] = true;
        }
    }
    if (s.max_blk > C::WS_U4)
        return fail(SBNN_ERR_UNSUPPORTED, "internal: weight block %d exceeds buffer %d", s.max_blk, C::WS_U4);
    const long long nblk = (long long)((M + C::TM - 1) / C::TM) * s.ntiles;
    if (nblk > 0x7fffffffLL) return fail(SBNN_ERR_SHAPE, "too many tiles");
    if (prepare_only()) return SBNN_OK;
    dim3 grid((unsigned)nblk);
    conv1x1_gs_kernel<C><<<grid, C::NT, C::SMEM, st>>>(x, y, p->d_bias, s.rec, s.blk_ptr, M, p->Cin, p->Cout,
                                                       p->ngroups, s.nchunks, s.ntiles, relu);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

// The instantiated tile configurations: (G, P, GPW, NW, KC).
#define SBNN_K1_CONFIGS(X) \
    X(1, 8, 4, 8, 64)      \
    X(2, 8, 2, 8, 64)      \
    X(4, 8, 1, 16, 64)     \
    X(4, 8, 2, 8, 64)      \
    X(4, 8, 2, 16, 32)     \
    X(4, 4, 1, 8, 64)      \
    X(4, 4, 2, 8, 64)      \
    X(8, 8, 1, 16, 32)     \
    X(8, 8, 1, 8, 64)      \
    X(8, 4, 1, 8, 64)      \
    X(16, 4, 1, 8, 64)

sbnn_status dispatch(const sbnn_packed* p, const TileCfg& c, const float* x, float* y, int M, int relu, cudaStream_t st) {
    Stream1x1 s;
#define SBNN_TRY_CFG(g, pp, gpw, nw, kc)                                      \
    if (p->G == g && c.P == pp && c.GPW == gpw && c.NW == nw && c.KC == kc) { \
        sbnn_status r = get_stream(p, c, &s);                                 \
        if (r != SBNN_OK) return r;                                           \
        return launch<K1<g, pp, gpw, nw, kc>>(p, s, x, y, M, relu, st);       \
    }
    SBNN_K1_CONFIGS(SBNN_TRY_CFG)
#undef SBNN_TRY_CFG
    return fail(SBNN_ERR_UNSUPPORTED, "no 1x1 kernel instance for G=%d P=%d GPW=%d NW=%d KC=%d", p->G, c.P, c.GPW,
                c.NW, c.KC);
}

// Default tile choice by layer shape.
TileCfg choose_cfg(const sbnn_packed* p, int64_t M) {
    const bool small = M <= 148 * 128;
    switch (p->G) {
        case 1: return {8, 4, 8, 64};
        case 2: return {8, 2, 8, 64};
        case 4: return small ? TileCfg{4, 1, 8, 64} : TileCfg{8, 1, 16, 64};
        case 8: return small ? TileCfg{4, 1, 8, 64} : TileCfg{8, 1, 8, 64};
        default: return {4, 1, 8, 64};
    }
}

sbnn_status check_args(const sbnn_packed* w, const float* x, float* y, int N, int H, int W, int flags) {
    if (!w || !x || !y) return fail(SBNN_ERR_NULL, "packed weights, x_dev and y_dev must not be NULL");
    if (w->KH != 1 || w->KW != 1) return fail(SBNN_ERR_SHAPE, "packed layer is %dx%d, expected 1x1", w->KH, w->KW);
    if (N < 0 || H < 0 || W < 0) return fail(SBNN_ERR_SHAPE, "negative activation shape %dx%dx%d", N, H, W);
    if ((int64_t)N * H * W > 0x7fffffff) return fail(SBNN_ERR_SHAPE, "N*H*W exceeds 2^31-1");
    if (flags & ~(SBNN_RELU | SBNN_BF16_TC | SBNN_BF16_GATHER)) return fail(SBNN_ERR_UNSUPPORTED, "unknown flag bits 0x%x", flags);
    if ((flags & SBNN_BF16_GATHER) && !(flags & SBNN_BF16_TC))
        return fail(SBNN_ERR_UNSUPPORTED, "SBNN_BF16_GATHER selects a variant of SBNN_BF16_TC and needs that flag too");
    if (!aligned16(x) || !aligned16(y)) return fail(SBNN_ERR_ALIGN, "x_dev and y_dev must be 16-byte aligned");
    if (w->Cin % 4) return fail(SBNN_ERR_UNSUPPORTED, "Cin=%d is not a multiple of 4", w->Cin);
    if ((int64_t)N * H * W == 0) return SBNN_OK;
    return check_packed_device(w);
}

}  // namespace

sbnn_status prepare_default_1x1(const sbnn_packed* p) {
    // Build the streams of the default configurations now, so compute calls only enqueue.
    Stream1x1 s;
    for (int64_t M : {int64_t(1), int64_t(1) << 30}) {
        sbnn_status r = get_stream(p, choose_cfg(p, M), &s);
        if (r != SBNN_OK) return r;
    }
    return p->Cin >= 128 ? prepare_default_cm(p) : SBNN_OK;
}

void free_streams_1x1(sbnn_packed* p) {
    for (auto& kv : p->streams1x1) {
        cudaFree(kv.second.rec);
        cudaFree(kv.second.blk_ptr);
    }
    p->streams1x1.clear();
}

}  // namespace sbnn

using namespace sbnn;

extern "C" sbnn_status sbnn_conv1x1_gs(const sbnn_packed* w, const float* x_dev, float* y_dev, int N, int H, int W,
                                       int flags, void* cuda_stream) {
    clear_error();
    sbnn_status st = check_args(w, x_dev, y_dev, N, H, W, flags);
    if (st != SBNN_OK) return st;
    const int64_t M = (int64_t)N * H * W;
    if (M == 0) return SBNN_OK;
    if ((st = check_device()) != SBNN_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    bool done = false;
    if (flags & SBNN_BF16_TC) {
        // dense over the masked weights on the tcgen05 tensor cores, unless the gathered warp-level kernel is asked
        // for or the shape is outside what the dense kernel takes
        if (!(flags & SBNN_BF16_GATHER) && ((st = conv1x1_umma(w, x_dev, y_dev, (int)M, flags & SBNN_RELU, s, &done)) != SBNN_OK || done))
            return st;
        return conv1x1_bf16(w, x_dev, y_dev, (int)M, flags & SBNN_RELU, s);
    }
    if ((st = conv1x1_via_cm(w, x_dev, y_dev, (int)M, flags & SBNN_RELU, s, &done)) != SBNN_OK || done) return st;
    return dispatch(w, choose_cfg(w, M), x_dev, y_dev, (int)M, flags & SBNN_RELU, s);
}

extern "C" sbnn_status sbnn_conv1x1_gs_tuned(const sbnn_packed* w, const float* x_dev, float* y_dev, int N, int H,
                                             int W, int flags, int P, int GPW, int NW, int KC, void* cuda_stream) {
    clear_error();
    sbnn_status st = check_args(w, x_dev, y_dev, N, H, W, flags);
    if (st != SBNN_OK) return st;
    if (flags & SBNN_BF16_TC) return fail(SBNN_ERR_UNSUPPORTED, "tile parameters apply to the fp32 kernel only");
    const int64_t M = (int64_t)N * H * W;
    if (M == 0) return SBNN_OK;
    if ((st = check_device()) != SBNN_OK) return st;
    return dispatch(w, TileCfg{P, GPW, NW, KC}, x_dev, y_dev, (int)M, flags & SBNN_RELU,
                    static_cast<cudaStream_t>(cuda_stream));
}
