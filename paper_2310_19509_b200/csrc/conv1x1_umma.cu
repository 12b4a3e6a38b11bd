// bf16 tensor-core mode of the 1x1 convolution on the 5th-generation tensor cores (tcgen05), flag SBNN_BF16_TC.
//
//   Y[m][o] = act( bias[o] + sum_c bf16(W~[o][c]) * bf16(X[m][c]) ),   W~ = W (.) M  (Section 3.1), fp32 accumulation
//
// The contraction runs DENSE over the masked weights: the pruned entries of W~ are stored as zeros and multiplied.
// The reason is the shape of the method's sparsity.  A group shares its kept input channels over only G = 4..8 output
// channels (Section 3.2), so a contraction that skips pruned channels has an N extent of G: a 128 x 8 x 16 MMA reads
// a 4 KB A slice from shared memory for 16 K MACs, i.e. the tensor core would run at the pace of the shared-memory
// operand read (about 1/8 of its dense rate at G = 8) and every group would need its own gathered copy of A.  Dense
// 128 x 256 tiles reuse each A slice over 256 output channels and are faster than the gathered form up to about
// 87 % sparsity, and faster than the fp32 kernel at every sparsity.  (The gathered warp-level kernel stays available
// behind SBNN_BF16_GATHER.)
//
// Structure, one CTA per SM, persistent over 128 x BN output tiles:
//   warp 0   producer: per 64-channel step two tiled tensor-map copies (A: 128 pixels x 64 channels of the bf16
//            activations, B: BN output channels x 64 channels of the bf16 weights, both K-major with the 128-byte
//            swizzle) onto the stage's "full" mbarrier;
//   warp 1   issues the MMAs: 4 x tcgen05.mma (128 x BN x 16, operands straight from shared memory through
//            descriptors) per stage into one of two accumulators in tensor memory; tcgen05.commit releases the
//            stage ("empty") and, after the last step, publishes the accumulator ("acc_full");
//   warps 2-5 epilogue: tcgen05.ld of the warp's 32 accumulator rows, bias, ReLU, staging of 32 x 32 blocks in
//            shared memory and tiled copies to the NHWC output (full 128-byte rows, asynchronous); then the
//            accumulator is handed back ("acc_empty"), so the epilogue of one tile overlaps the MMAs of the next.
// Every mbarrier wait is bounded; an expired wait records SBNN_ERR_TIMEOUT in the device status word, raises the
// CTA's abort flag, and all warps fall through to the common exit, where the tensor memory is released.
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include <cuda.h>   // CUtensorMap (type only; the encode call is looked up at run time in conv1x1_cm.cu)

#include "common.h"
#include "pipeline.cuh"

namespace sbnn {
namespace {

// ---- tcgen05 primitives ---------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Whole warp: reserves `cols` (a power of two >= 32) columns of tensor memory; the base address lands in *holder.
__device__ __forceinline__ void tmem_alloc(uint32_t* holder_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder_smem)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes (64 bf16) written with the 128-byte
// swizzle, rows 128 bytes apart, groups of 8 rows 1024 bytes apart; `addr` = shared address of the first row's
// 16-byte chunk to start from (the tile itself is 1024-byte aligned, a K offset of 16 elements is +32 bytes).
__device__ __forceinline__ uint64_t operand_desc(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);   // bits  0-13: start address / 16
    d |= (uint64_t)1 << 16;                            // bits 16-29: leading byte offset / 16 (not used by this layout)
    d |= (uint64_t)(1024 >> 4) << 32;                  // bits 32-45: stride byte offset / 16
    d |= (uint64_t)1 << 46;                            // bits 46-47: descriptor version of this architecture
    d |= (uint64_t)2 << 61;                            // bits 61-63: 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
    return (1u << 4)                    // accumulator format fp32
           | (1u << 7) | (1u << 10)     // A and B format bf16
           | ((uint32_t)(n >> 3) << 17) // N / 8
           | ((uint32_t)(128 >> 4) << 24);   // M / 16
}

// One thread: D[tmem] (+)= A[smem] * B[smem]^T, 128 x N x 16.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// The mbarrier receives one arrival once every MMA this thread has issued so far is complete.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Whole warp: 32 consecutive fp32 columns of the warp's 32 tensor-memory lanes (lane l of the warp gets row l).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- tile shape -----------------------------------------------------------------------------------
template <int BN_>
struct UT {
    static constexpr int BM = 128, BN = BN_, BK = 64, UK = 16;
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE = A_BYTES + B_BYTES;
    static constexpr int S = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int NT = 192;                        // producer warp, MMA warp, four epilogue warps
    static constexpr int TMEM_COLS = 2 * BN;              // two accumulators
    static constexpr int CTRL = 256;                      // mbarriers, tensor-memory base, abort flag
    static constexpr int OUT_TILE = 32 * 32 * 4;          // epilogue staging: 32 pixels x 32 output channels fp32, 128-byte swizzled rows
    static constexpr int OUT_BYTES = 4 * 2 * OUT_TILE;    // two such tiles for each of the four epilogue warps
    static constexpr size_t SMEM = (size_t)S * STAGE + OUT_BYTES + CTRL + 1024;   // + slack to align the stages to 1024 bytes
    static_assert(STAGE % 1024 == 0 && A_BYTES % 1024 == 0, "stages must keep the swizzle alignment");
    static_assert((2 * S + 4) * 8 + 8 <= CTRL, "control block");
    static_assert(SMEM <= 227 * 1024, "shared memory");
};

template <int BN>
__global__ void __launch_bounds__(UT<BN>::NT, 1)
conv1x1_umma_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
                    const __grid_constant__ CUtensorMap ymap, const float* __restrict__ bias, int M, int Cout, int nkb, int ntiles_n,
                    int total_tiles, int relu, int* status) {
    // Both operands are stored tile by tile: A as [pixel tile][channel step][128 pixels][64 channels], B as
    // [channel step][output channels, padded to whole tiles][64 channels], so every box is one contiguous block.
    using T = UT<BN>;
    constexpr int S = T::S;
    extern __shared__ unsigned char raw[];
    const uint32_t raw_addr = smem_u32(raw);
    unsigned char* sm = raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);     // stages, 1024-byte aligned
    unsigned char* out_stage = sm + (size_t)S * T::STAGE;                       // 1024-byte aligned as well
    uint64_t* full = reinterpret_cast<uint64_t*>(out_stage + T::OUT_BYTES);
    uint64_t* empty = full + S;
    uint64_t* acc_full = empty + S;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full + a, 1);
            mbar_init(acc_empty + a, 4);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_holder, T::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ---------------- producer ----------------
        int issued = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const int m0 = (t / ntiles_n) * T::BM, n0 = (t % ntiles_n) * BN;
            for (int kb = 0; kb < nkb; ++kb, ++issued) {
                const int s = issued % S;
                if (issued >= S) ok = __all_sync(0xffffffffu, mbar_wait(empty + s, ((issued / S) & 1) ^ 1, abort_flag, status, SBNN_ERR_TIMEOUT));
                if (!ok) break;
                if (lane == 0) {
                    unsigned char* st = sm + (size_t)s * T::STAGE;
                    mbar_arrive_expect_tx(full + s, (uint32_t)T::STAGE);
                    tensor_g2s_2d(st, &amap, 0, ((t / ntiles_n) * nkb + kb) * T::BM, full + s);
                    tensor_g2s_2d(st + T::A_BYTES, &bmap, 0, kb * ntiles_n * BN + n0, full + s);
                }
                __syncwarp();
            }
        }
        if (!ok) {   // gave up: let the copies already issued land before the shared memory is released
            for (int k = max(0, issued - S); k < issued; ++k) {
                bool landed = false;
                for (uint32_t i = 0; i < kWaitLimit && !landed; ++i) landed = mbar_try_wait(full + k % S, (k / S) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        constexpr uint32_t idesc = instr_desc(BN);
        int consumed = 0, it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
            const int a = it & 1, use = it >> 1;
            if (use > 0) ok = __all_sync(0xffffffffu, mbar_wait(acc_empty + a, (use - 1) & 1, abort_flag, status, SBNN_ERR_TIMEOUT));   // epilogue has drained it
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
            for (int kb = 0; kb < nkb; ++kb, ++consumed) {
                const int s = consumed % S;
                ok = __all_sync(0xffffffffu, mbar_wait(full + s, (consumed / S) & 1, abort_flag, status, SBNN_ERR_TIMEOUT));
                if (!ok) break;
                tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t a_addr = smem_u32(sm + (size_t)s * T::STAGE), b_addr = a_addr + T::A_BYTES;
#pragma unroll
                    for (int k = 0; k < T::BK / T::UK; ++k)
                        umma_bf16(d_tmem, operand_desc(a_addr + k * T::UK * 2), operand_desc(b_addr + k * T::UK * 2), idesc,
                                  (kb | k) ? 1u : 0u);
                    umma_commit(empty + s);                 // the stage is free once these MMAs have read it
                }
                __syncwarp();
            }
            if (ok && lane == 0) umma_commit(acc_full + a);   // the accumulator is complete once every MMA of the tile is
            __syncwarp();
        }
    } else {
        // ---------------- epilogue ----------------
        // A warp reads its 32 accumulator rows 32 columns at a time (a lane holds one pixel's 32 channels), adds the
        // bias, applies the ReLU and writes the 32 x 32 block into one of its two staging tiles, whose 128-byte rows
        // are swizzled (16-byte chunk j of row r sits at chunk j ^ (r % 8)) so that the lanes' 16-byte writes fall
        // into distinct banks; a tiled copy then stores the block to Y as 32 full 128-byte rows, in the background.
        // Rows past M and channels past Cout are clipped by the copy.
        const int q = warp & 3;                             // the quarter of the tensor-memory lanes this warp may read
        unsigned char* stage_tiles = out_stage + (size_t)q * 2 * T::OUT_TILE;
        int it = 0, chunk = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++it) {
            const int a = it & 1, use = it >> 1;
            const int m0 = (t / ntiles_n) * T::BM, n0 = (t % ntiles_n) * BN;
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full + a, use & 1, abort_flag, status, SBNN_ERR_TIMEOUT))) break;   // warp-uniform
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * BN);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(taddr + c0, v);
                unsigned char* tile = stage_tiles + (size_t)(chunk & 1) * T::OUT_TILE;
                if (lane == 0) bulk_wait_read_pending1();   // the copy that last read this tile (two chunks ago) is done with it
                __syncwarp();
                tmem_ld_wait();
                if (n0 + c0 < Cout) {                        // warp-uniform; Cout is a multiple of 4
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int n = n0 + c0 + 4 * j;
                        const float4 b4 = n < Cout ? __ldg(reinterpret_cast<const float4*>(bias + n)) : make_float4(0.f, 0.f, 0.f, 0.f);
                        float4 o = make_float4(__uint_as_float(v[4 * j]) + b4.x, __uint_as_float(v[4 * j + 1]) + b4.y,
                                               __uint_as_float(v[4 * j + 2]) + b4.z, __uint_as_float(v[4 * j + 3]) + b4.w);
                        if (relu) o = make_float4(fmaxf(o.x, 0.f), fmaxf(o.y, 0.f), fmaxf(o.z, 0.f), fmaxf(o.w, 0.f));
                        *reinterpret_cast<float4*>(tile + lane * 128 + ((j ^ (lane & 7)) << 4)) = o;
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tensor_s2g_2d(&ymap, n0 + c0, m0 + q * 32, tile);
                        bulk_commit_group();
                    }
                    ++chunk;                                 // counts issued copies: the two tiles alternate between them
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + a);
        }
        if (lane == 0) bulk_wait_all();                     // this thread's copies are complete before the CTA gives up its shared memory
    }
    // common exit: nobody may still be using the tensor memory when it is released
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, T::TMEM_COLS);
}

// X fp32 [M][Cin] -> bf16 (round to nearest even) in the tiled order the kernel's A boxes are read in:
// [pixel tile of 128][channel step of 64][128 pixels][64 channels], pixels past M and channels past Cin as zeros.
// One warp per pixel row; a lane converts 8 consecutive channels (Cin is a multiple of 8) per round of 256.
__global__ void __launch_bounds__(256)
to_bf16_tiled_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ xb, int M, int Cin, int nkb, int rows_padded) {
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (m >= rows_padded) return;
    const float* xr = x + (size_t)m * Cin;
    uint4* tile = reinterpret_cast<uint4*>(xb) + ((size_t)(m >> 7) * nkb * 128 * 64 + (size_t)(m & 127) * 64) / 8;
    for (int c = lane * 8; c < nkb * 64; c += 256) {
        uint4 o = make_uint4(0u, 0u, 0u, 0u);
        if (m < M && c < Cin) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(xr + c)), b = __ldg(reinterpret_cast<const float4*>(xr + c + 4));
            __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
            __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
            o.x = *reinterpret_cast<uint32_t*>(&p0); o.y = *reinterpret_cast<uint32_t*>(&p1);
            o.z = *reinterpret_cast<uint32_t*>(&p2); o.w = *reinterpret_cast<uint32_t*>(&p3);
        }
        tile[(size_t)(c >> 6) * (128 * 64 / 8) + ((c & 63) >> 3)] = o;
    }
}

// fp32 -> bf16 bits, round to nearest even (finite inputs).
uint16_t bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// Output-tile width for a layer (a template instance exists for each).
int tile_width(int Cout) { return Cout > 128 ? 256 : (Cout > 64 ? 128 : 64); }

struct DenseBf16 {
    uint16_t* w = nullptr;   // device, [channel step][Cout padded to whole output tiles][64] bf16: the masked weights, zeros where pruned
};

sbnn_status build_dense_bf16(const sbnn_packed* p, DenseBf16* out) {
    const int BN = tile_width(p->Cout), nkb = (p->Cin + 63) / 64;
    const size_t cout_pad = (size_t)(p->Cout + BN - 1) / BN * BN;
    std::vector<uint16_t> w;
    try {
        w.assign((size_t)nkb * cout_pad * 64, 0);
    } catch (const std::bad_alloc&) {
        return fail(SBNN_ERR_ALLOC, "out of host memory building the dense bf16 weights");
    }
    const int G = p->G;
    for (int g = 0; g < p->ngroups; ++g)
        for (int64_t j = p->group_ptr[g]; j < p->group_ptr[g + 1]; ++j) {
            const int c = p->idx[j];
            for (int r = 0; r < G; ++r)
                w[((size_t)(c >> 6) * cout_pad + (size_t)(g * G + r)) * 64 + (c & 63)] = bf16_rne(p->val[(size_t)j * G + r]);
        }
    DenseBf16 d;
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&d.w), w.size() * 2));
    cudaError_t e = cudaMemcpy(d.w, w.data(), w.size() * 2, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(d.w);
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "uploading the dense bf16 weights: %s", cudaGetErrorString(e));
    }
    *out = d;
    return SBNN_OK;
}

template <int BN>
sbnn_status launch_umma(const sbnn_packed* p, const DenseBf16& d, const __nv_bfloat16* xb, float* y, int M, int relu,
                        cudaStream_t st) {
    using T = UT<BN>;
    sbnn_status r = set_max_dyn_smem(reinterpret_cast<const void*>(&conv1x1_umma_kernel<BN>), (int)T::SMEM);
    if (r != SBNN_OK) return r;
    int* status = nullptr;
    if ((r = async_status_word(&status)) != SBNN_OK) return r;
    if (prepare_only()) return SBNN_OK;
    const int mtiles = (M + T::BM - 1) / T::BM, ntiles_n = (p->Cout + BN - 1) / BN, nkb = (p->Cin + T::BK - 1) / T::BK;
    CUtensorMap amap, bmap;
    {   // A: [mtiles * nkb * 128 rows][64 channels] bf16, a box = the 128 x 64 block of one (pixel tile, channel step)
        const unsigned long long dims[2] = {(unsigned long long)T::BK, (unsigned long long)mtiles * nkb * T::BM};
        const unsigned long long strides[1] = {(unsigned long long)T::BK * 2};
        const unsigned box[2] = {(unsigned)T::BK, (unsigned)T::BM};
        if ((r = encode_tiled_map(&amap, xb, 2, 2, dims, strides, box, true)) != SBNN_OK) return r;
    }
    {   // B: [nkb * padded Cout rows][64 channels] bf16, a box = BN output channels of one channel step
        const unsigned long long dims[2] = {(unsigned long long)T::BK, (unsigned long long)nkb * ntiles_n * BN};
        const unsigned long long strides[1] = {(unsigned long long)T::BK * 2};
        const unsigned box[2] = {(unsigned)T::BK, (unsigned)BN};
        if ((r = encode_tiled_map(&bmap, d.w, 2, 2, dims, strides, box, true)) != SBNN_OK) return r;
    }
    CUtensorMap ymap;
    {   // Y [M][Cout] fp32, stored in boxes of 32 pixels x 32 channels out of swizzled shared-memory tiles
        const unsigned long long dims[2] = {(unsigned long long)p->Cout, (unsigned long long)M};
        const unsigned long long strides[1] = {(unsigned long long)p->Cout * 4};
        const unsigned box[2] = {32u, 32u};
        if ((r = encode_tiled_map(&ymap, y, 4, 2, dims, strides, box, true)) != SBNN_OK) return r;
    }
    const long long total = (long long)mtiles * ntiles_n;
    if (total > 0x7fffffffLL) return fail(SBNN_ERR_SHAPE, "too many tiles");
    int dev = 0, sms = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    SBNN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const unsigned grid = (unsigned)std::min<long long>(total, std::max(sms, 1));
    conv1x1_umma_kernel<BN><<<grid, T::NT, T::SMEM, st>>>(amap, bmap, ymap, p->d_bias, M, p->Cout, nkb,
                                                         ntiles_n, (int)total, relu, status);
    SBNN_CUDA_TRY(cudaGetLastError());
    return SBNN_OK;
}

}  // namespace

// Dense-over-masked-weights bf16 path.  *done = false (and SBNN_OK) when the shape is outside what this kernel takes
// (the caller then uses the gathered kernel): Cin must be a multiple of 8 (16-byte rows for the tensor map), Cout of 4.
sbnn_status conv1x1_umma(const sbnn_packed* p, const float* x, float* y, int M, int relu, cudaStream_t st, bool* done) {
    *done = false;
    if (p->Cin % 8 || p->Cout % 4 || (long long)M * p->Cin > 0x7fffffff0LL) return SBNN_OK;
    DenseBf16* d = nullptr;
    {
        std::lock_guard<std::mutex> lk(p->mu);
        if (!p->umma_weights) {   // first use of the mode on this layer: build the dense bf16 matrix (allocates, copies)
            DenseBf16* n = new (std::nothrow) DenseBf16;
            if (!n) return fail(SBNN_ERR_ALLOC, "out of host memory");
            sbnn_status r = build_dense_bf16(p, n);
            if (r != SBNN_OK) {
                delete n;
                return r;
            }
            p->umma_weights = n;
        }
        d = static_cast<DenseBf16*>(p->umma_weights);
    }
    float* scratch = nullptr;
    const int nkb = (p->Cin + 63) / 64, rows_padded = (M + 127) / 128 * 128;
    sbnn_status r = scratch_workspace((size_t)rows_padded * nkb * 64 * sizeof(__nv_bfloat16), st, &scratch);
    if (r != SBNN_OK) return r;
    __nv_bfloat16* xb = reinterpret_cast<__nv_bfloat16*>(scratch);
    if (!prepare_only()) {
        to_bf16_tiled_kernel<<<(unsigned)(rows_padded / 8), 256, 0, st>>>(x, xb, M, p->Cin, nkb, rows_padded);
        SBNN_CUDA_TRY(cudaGetLastError());
    }
    switch (tile_width(p->Cout)) {
        case 256: r = launch_umma<256>(p, *d, xb, y, M, relu, st); break;
        case 128: r = launch_umma<128>(p, *d, xb, y, M, relu, st); break;
        default: r = launch_umma<64>(p, *d, xb, y, M, relu, st); break;
    }
    if (r == SBNN_OK) *done = true;
    return r;
}

void free_umma_weights(sbnn_packed* p) {
    if (!p->umma_weights) return;
    DenseBf16* d = static_cast<DenseBf16*>(p->umma_weights);
    cudaFree(d->w);
    delete d;
    p->umma_weights = nullptr;
}

}  // namespace sbnn
