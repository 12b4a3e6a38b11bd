// Shared declarations of libsbnn's translation units (not part of the public interface).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "sbnn.h"

namespace sbnn {

// Records the thread-local error text and returns `s`, so call sites can `return fail(...)`.
sbnn_status fail(sbnn_status s, const char* fmt, ...);
void clear_error();

// SBNN_OK if the current device exists and is compute capability 10.x.
sbnn_status check_device();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// True while the calling thread is inside sbnn_prepare: the entry points then run their whole host path (private
// weight layouts, scratch sizing, kernel attributes) but enqueue nothing and touch neither x_dev nor y_dev.
bool prepare_only();
struct PrepareScope {
    PrepareScope();
    ~PrepareScope();
};

// True while the calling thread is inside the MobileNet chain's forward pass: kernels are then launched with
// programmatic stream serialization, i.e. a kernel may become resident and run its set-up while its predecessor in
// the stream drains.  Every kernel launched this way executes grid_dependency_wait() (pipeline.cuh) before it reads or
// writes anything another kernel of the stream touches.
bool chained_launch();
struct ChainedLaunchScope {
    ChainedLaunchScope();
    ~ChainedLaunchScope();
};

// Kernel launch that honours chained_launch().  Arguments are converted to the kernel's parameter types.
template <class... Params, class... Args>
cudaError_t launch_kernel(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (chained_launch()) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

// Raises a kernel's dynamic shared-memory limit to `bytes` on the current device, once per (device, kernel) and size.
sbnn_status set_max_dyn_smem(const void* func, int bytes);

#define SBNN_CUDA_TRY(expr)                                                                         \
    do {                                                                                            \
        cudaError_t e__ = (expr);                                                                   \
        if (e__ != cudaSuccess)                                                                     \
            return ::sbnn::fail(e__ == cudaErrorMemoryAllocation ? SBNN_ERR_ALLOC : SBNN_ERR_CUDA,  \
                                "%s: %s", #expr, cudaGetErrorString(e__));                          \
    } while (0)

// Tile configuration of the group-sparse 1x1 kernel; also the key of the kernel-private weight stream.
struct TileCfg {
    int P;    // pixels per lane (a warp covers 32*P consecutive pixels)
    int GPW;  // groups a warp accumulates at once
    int NW;   // warps per CTA
    int KC;   // input channels staged per pipeline step
    int TM() const { return 32 * P; }
    int GT() const { return NW * GPW; }
    bool operator<(const TileCfg& o) const {
        if (P != o.P) return P < o.P;
        if (GPW != o.GPW) return GPW < o.GPW;
        if (NW != o.NW) return NW < o.NW;
        return KC < o.KC;
    }
};

// Kernel-private re-layout of a packed 1x1 layer for one TileCfg (device memory).
struct Stream1x1 {
    uint4* rec = nullptr;        // record stream, 16-byte units
    int32_t* blk_ptr = nullptr;  // [ntiles][nchunks + 1] offsets into rec
    int ntiles = 0, nchunks = 0;
    int max_blk = 0;             // largest block in 16-byte units
};

// Kernel-private re-layout of a packed 3x3 layer (see conv3x3_gs.cu).
struct Stream3x3 {
    uint4* rec = nullptr;
    int32_t* blk_ptr = nullptr;
    int ntiles = 0, nchunks = 0;
    int max_blk = 0;
    std::vector<int32_t> blk_host;   // host copy of blk_ptr: the block sizes weigh the shares of the persistent CTAs
};

// How one launch of the 3x3 copy-engine kernel deals the channel steps of its tiles to the persistent CTAs
// (device memory; see conv3x3_gs.cu).
struct Plan3x3 {
    int32_t* cta_ptr = nullptr;  // [ncta + 1] offsets into segs
    void* segs = nullptr;
    int ncta = 0;
    int nslots = 0;              // partial-sum slots the split tiles need
    int ncounters = 0;           // split tiles
};

}  // namespace sbnn

struct sbnn_packed {
    int Cout = 0, KH = 0, KW = 0, Cin = 0, G = 0, ngroups = 0;
    int64_t nnz = 0;
    std::vector<int32_t> group_ptr, idx;
    std::vector<float> val, bias;
    std::vector<uint16_t> tap_mask;   // per kept unit, bit t = tap t kept; empty unless packed with tap patterns
    mutable long long kept_taps = -1; // taps kept over all units of a pattern layer (counted on first use, under mu)
    int gi = 1;                       // 4 if every group's kept channels are aligned runs of 4 (the paper's 4 x 4 blocks), else 1
    std::vector<int32_t> block_idx;   // gi == 4: first channel of every run, [nnz / 4]
    // device side (valid when device >= 0)
    int device = -1;
    int32_t* d_group_ptr = nullptr;
    int32_t* d_idx = nullptr;
    float* d_val = nullptr;
    float* d_bias = nullptr;
    // kernel-private layouts, built on first use of a tile configuration
    mutable std::mutex mu;
    mutable std::map<sbnn::TileCfg, sbnn::Stream1x1> streams1x1;
    mutable std::map<sbnn::TileCfg, sbnn::Stream1x1> streams_cm;   // channel-major kernel, see conv1x1_cm.cu
    mutable std::map<long long, sbnn::TileCfg> cfg_cm;             // tile shape chosen for a pixel count (the choice costs a loop over the tiles)
    mutable std::map<int, sbnn::Stream3x3> streams3x3;
    mutable std::map<long long, sbnn::Plan3x3> plans3x3;           // per (stream, row tiles of the launch, CTAs)
    mutable void* bf16_stream = nullptr;  // see conv1x1_bf16.cu
    mutable void* umma_weights = nullptr; // dense bf16 copy of the masked weights, see conv1x1_umma.cu
};

namespace sbnn {
// SBNN_OK if `w` has device copies and they live on the current device (else SBNN_ERR_CUDA, nothing is launched).
sbnn_status check_packed_device(const sbnn_packed* w);
// conv1x1_gs.cu
sbnn_status prepare_default_1x1(const sbnn_packed* p);
void free_streams_1x1(sbnn_packed* p);
// conv1x1_cm.cu
// Builds the weight stream of the tile shape that a launch on M pixels would pick (M <= 0: the many-pixel choice).
sbnn_status prepare_default_cm(const sbnn_packed* p, long long M = 0);
sbnn_status prepare_cm(const sbnn_packed* p, int P, int GPW, int NW, int KC);   // builds the stream of one tile shape
void free_streams_cm(sbnn_packed* p);
// Runs the NHWC call through the channel-major kernel if the shape profits; *done tells whether it did.
sbnn_status conv1x1_via_cm(const sbnn_packed* w, const float* x, float* y, int M, int relu, cudaStream_t st, bool* done);
// Depthwise 3x3 (stride 1) + group-sparse 1x1 in one kernel on channel-major tensors; *done = false (and SBNN_OK) when the
// shape is outside what the fused kernel takes (G = 4, W a multiple of 4, W <= 124).
sbnn_status dwconv3x3_conv1x1_fused_cm(const sbnn_packed* pw, const float* dw_w, const float* dw_b, const float* x, int ldx, float* y,
                                       int ldy, int N, int H, int W, int relu_dw, int relu, cudaStream_t st, bool* done);
sbnn_status read_async_status(int* value);
// Device address of the status word that bounded waits report into (per device).
sbnn_status async_status_word(int** out);
// Fills a 128-byte tensor-map descriptor (CUtensorMap) for tiled copies out of an fp32 (elem_bytes 4) or bf16 (2)
// tensor: `rank` dimensions, innermost first, `strides_bytes` for dimensions 1.. (multiples of 16), `box` = elements
// copied per dimension.  Elements outside the tensor are delivered as zeros.
// With swizzle128 the box's rows (at most 128 bytes) are written to shared memory with the 128-byte swizzle that the
// tcgen05 operand descriptors expect.
sbnn_status encode_tiled_map(void* out, const void* base, int elem_bytes, int rank, const unsigned long long* dims,
                             const unsigned long long* strides_bytes, const unsigned* box, bool swizzle128 = false);
// Per-device scratch buffer for channel-major copies made on behalf of NHWC callers.  Grows on demand with a
// synchronous allocation (the outgrown buffer is kept until the process exits, so work already enqueued or recorded
// on it stays valid); growth while `st` is being captured is refused with SBNN_ERR_UNSUPPORTED.
sbnn_status scratch_workspace(size_t bytes, cudaStream_t st, float** out);
// cm_layers.cu: dense layers on channel-major activations ([C][ld]); arguments validated by the callers
sbnn_status launch_transpose(const float* in, int ld_in, float* out, int ld_out, int R, int Ccols, cudaStream_t st);
sbnn_status launch_dwconv3x3_cm(const float* w, const float* b, const float* x, int ldx, float* y, int ldy, int N, int H,
                                int W, int C, int stride, int relu, cudaStream_t st);
sbnn_status launch_conv3x3_thin_cm(const float* w, const float* b, const float* x, float* y, int ldy, int N, int H, int W,
                                   int Cin, int Cout, int stride, int relu, cudaStream_t st);
sbnn_status launch_avgpool_cm(const float* x, int ldx, float* y, int ldy, int N, int HW, int C, cudaStream_t st);
// conv1x1_small.cu: kernel for launches with few pixels; reads the canonical packed arrays (no private layout)
sbnn_status conv1x1_small(const sbnn_packed* p, const float* x, int ldx, float* y, int ldy, int M, int relu, bool out_cm,
                          cudaStream_t st);
// conv1x1_bf16.cu
sbnn_status conv1x1_bf16(const sbnn_packed* w, const float* x, float* y, int M, int relu, cudaStream_t st);
void free_stream_bf16(sbnn_packed* p);
// conv1x1_umma.cu: bf16 mode as a dense contraction over the masked weights (tcgen05); *done = false if the shape is not taken
sbnn_status conv1x1_umma(const sbnn_packed* w, const float* x, float* y, int M, int relu, cudaStream_t st, bool* done);
void free_umma_weights(sbnn_packed* p);
// conv3x3_gs.cu
sbnn_status prepare_default_3x3(const sbnn_packed* p);
void free_streams_3x3(sbnn_packed* p);
}  // namespace sbnn
