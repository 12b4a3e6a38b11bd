/*
 * sbnn.h — C interface of libsbnn: group-sparse convolution for NVIDIA B200 (sm_100a).
 *
 * The library computes convolutions whose weights are fine-grained group-sparse:
 * G consecutive output channels (one "group") share one 0/1 mask over the input
 * channels, so a "unit" — the G weights (1x1 kernel) or 9*G weights (3x3 kernel)
 * that connect one input channel to one group — is either kept or removed as a
 * whole (the paper's connectivity group pruning, Section 3.2 and Eq. 2, with an
 * input-channel group size of 1).  The result is by definition the ordinary
 * convolution with W~ = W (.) M (Section 3.1); the kernels reach it by visiting
 * kept units only (Algorithm 1).
 *
 * Conventions that hold for every entry point
 *   - Tensors: activations [N][H][W][C] fp32 (NHWC), weights [Cout][KH][KW][Cin]
 *     fp32, as in Algorithm 1's data declaration.  Zero padding (K-1)/2,
 *     cross-correlation (no kernel flip), bias added before the optional ReLU.
 *   - "_host" pointers are ordinary host memory, "_dev" pointers are device
 *     memory of the current CUDA device, 16-byte aligned, owned by the caller.
 *     Input and output buffers must not overlap.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls that create, pack, prepare or free objects may allocate and
 *     synchronise.  A compute call only enqueues kernels on the stream and returns,
 *     provided sbnn_prepare has been called for the layer with a shape at least as
 *     large (sbnn_mobilenet_v1_create does the same for the chain); without it, the
 *     first call of a layer at a new shape or in a new mode may build a private
 *     weight layout or grow the per-device scratch buffer, both synchronously.
 *   - Packed layers and networks belong to the device that was current when they were
 *     packed / created; a compute call made while another device is current returns
 *     SBNN_ERR_CUDA.
 *   - Every function returns an sbnn_status; nothing throws, aborts or exits.
 *     On error no kernel is launched.  sbnn_last_error() gives a thread-local
 *     one-line explanation of the most recent failure.
 *   - There is no CPU fallback: compute calls need a B200-class device
 *     (compute capability 10.x) and fail with SBNN_ERR_ARCH / SBNN_ERR_CUDA
 *     otherwise.  Packing is host-side and works without a device.
 */
#ifndef SBNN_H_
#define SBNN_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SBNN_API __attribute__((visibility("default")))
#else
#define SBNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SBNN_OK = 0,
    SBNN_ERR_NULL = 1,                   /* a required pointer is NULL */
    SBNN_ERR_SHAPE = 2,                  /* a dimension is negative, zero where it may not be, or inconsistent */
    SBNN_ERR_GROUP = 3,                  /* G not in {1,2,4,8,16} or Cout % G != 0 */
    SBNN_ERR_MASK_NOT_GROUP_UNIFORM = 4, /* mask differs inside a group's rows or taps, or holds a value > 1 */
    SBNN_ERR_ALIGN = 5,                  /* a device pointer is not 16-byte aligned */
    SBNN_ERR_UNSUPPORTED = 6,            /* valid request outside what the kernels implement */
    SBNN_ERR_ARCH = 7,                   /* current device is not compute capability 10.x */
    SBNN_ERR_ALLOC = 8,                  /* host or device allocation failed */
    SBNN_ERR_CUDA = 9,                   /* a CUDA runtime call failed or no device is present */
    SBNN_ERR_TIMEOUT = 10,               /* a bounded device-side wait gave up (reported by sbnn_get_async_status) */
    SBNN_ERR_IO = 11                     /* a packed-layer file could not be opened, read or written, or is corrupt */
} sbnn_status;

/* Static name of a status code ("SBNN_OK", ...). Never NULL. */
SBNN_API const char* sbnn_status_str(sbnn_status s);
/* Detail of the calling thread's most recent failing call; "" if none.  Valid until that thread's next call. */
SBNN_API const char* sbnn_last_error(void);

/* ------------------------------------------------------------------------------------------------
 * Packing (Section 3.5: the conversion step that produces the engine's sparse weight format;
 * Algorithm 1's "sparse info SD" is the per-group list of kept input channels).
 * ------------------------------------------------------------------------------------------------ */

/* Opaque packed layer.  Owns a host copy and, if a device was present at pack time, device copies. */
typedef struct sbnn_packed sbnn_packed;

/*
 * Build the group-compressed form of one layer.
 *   W_host    [Cout][KH][KW][Cin] fp32 dense weights (values under a zero mask entry are ignored)
 *   mask_host [Cout][KH][KW][Cin] uint8, 1 = kept.  Must be identical for the G rows of a group and
 *             for all KH*KW taps (a unit is kept or removed as a whole), else
 *             SBNN_ERR_MASK_NOT_GROUP_UNIFORM.
 *   bias_host [Cout] or NULL (= zeros)
 *   KH = KW = 1 or 3.  G in {1,2,4,8,16}, Cout % G == 0.
 * Canonical layout produced (all little-endian host arrays, also uploaded to the device):
 *   group_ptr int32 [Cout/G + 1]   prefix sums of kept units per group
 *   idx       int32 [nnz_units]    kept input channels, ascending inside each group
 *   val       fp32  [nnz_units][KH*KW][G]   weights of a unit: taps outer, the group's channels inner
 *   bias      fp32  [Cout]
 * A kept weight that is numerically zero stays stored (packing follows the mask, not the values).
 * On success *out owns everything; release it with sbnn_packed_free.  If no CUDA device is present the
 * object is host-only (view / unpack work, compute calls return SBNN_ERR_CUDA).
 */
SBNN_API sbnn_status sbnn_pack_weights(const float* W_host, const uint8_t* mask_host, const float* bias_host,
                                       int Cout, int KH, int KW, int Cin, int G, sbnn_packed** out);

/*
 * Kernel-pattern variant of packing (Section 3.3, last paragraph: pattern pruning of Conv3x3 in the manner of
 * PatDNN, one pattern shared by adjacent filters; Section 3.2 for the patterns of a kernel).  Same arguments
 * and layout as sbnn_pack_weights, but the taps of a unit may be masked individually: the mask must still be
 * identical for the G filters of a group (the pattern is shared by the group), a unit is kept if any of its
 * KH*KW taps is, pruned taps are stored as 0.0f in val, and the view's tap_mask records which taps were kept,
 * so that sbnn_unpack_weights returns the mask exactly.  The convolution entry points take the result like
 * any other packed layer (pruned taps are multiplied as zeros; they are not skipped).
 */
SBNN_API sbnn_status sbnn_pack_weights_pattern(const float* W_host, const uint8_t* mask_host, const float* bias_host,
                                               int Cout, int KH, int KW, int Cin, int G, sbnn_packed** out);

typedef struct {
    int Cout, KH, KW, Cin, G, ngroups;
    int64_t nnz_units;
    const int32_t* group_ptr; /* host, borrowed from the sbnn_packed */
    const int32_t* idx;       /* host, borrowed */
    const float* val;         /* host, borrowed */
    const float* bias;        /* host, borrowed */
    const uint16_t* tap_mask; /* host, borrowed: [nnz_units], bit t = tap t of the unit is kept; NULL unless the layer
                                 was packed by sbnn_pack_weights_pattern */
    int gi;                   /* 4 if every group keeps aligned runs of 4 consecutive input channels (the paper's
                                 gi x go = 4 x G blocks, Section 3.2), else 1 */
    const int32_t* block_idx; /* host, borrowed: gi == 4: first channel of every run, [nnz_units / 4] (Algorithm 1's
                                 SD: one index per block); NULL when gi == 1 */
} sbnn_packed_view;

/* Borrow the canonical host arrays; they stay valid until sbnn_packed_free. */
SBNN_API sbnn_status sbnn_packed_get(const sbnn_packed* p, sbnn_packed_view* view);
/* Inverse of packing: writes W (.) M and M (either pointer may be NULL), each [Cout][KH][KW][Cin]. */
SBNN_API sbnn_status sbnn_unpack_weights(const sbnn_packed* p, float* W_host_out, uint8_t* mask_host_out);
/* Frees host and device copies.  NULL is accepted. */
SBNN_API sbnn_status sbnn_packed_free(sbnn_packed* p);

/*
 * Packed layers as files (Section 3.5: the conversion tool writes the pruned model in the engine's own sparse
 * format, which the engine loads at start-up).  sbnn_packed_save writes the canonical arrays of one layer,
 * sbnn_packed_load reads them back into a new packed layer: host copy plus, if a device is present, device copies,
 * exactly as after packing.  File layout, little-endian, no padding:
 *   bytes 0-7    magic 'S' 'B' 'N' 'N' 'P' 'K' 0x01 0x00
 *   int32[8]     format version (1), Cout, KH, KW, Cin, G, has_tap_mask (0 or 1), index_block (0 or 4)
 *   int64        nnz_units
 *   int32        group_ptr[Cout/G + 1]
 *   int32        idx[nnz_units]                 index_block = 0: one index per kept unit
 *                idx[nnz_units / 4]             index_block = 4 (written for layers whose view has gi = 4): the first
 *                                               channel of every aligned run of 4 kept channels, a quarter of the indices
 *   float32      val[nnz_units][KH*KW][G]
 *   float32      bias[Cout]
 *   uint16       tap_mask[nnz_units]            only if has_tap_mask
 *   uint64       FNV-1a (64 bit) of all preceding bytes
 * Loading checks the magic, the version, the checksum and the structure (prefix sums, ascending in-range indices,
 * non-empty tap masks), sets the stored weights of pruned taps to zero (as the packer writes them: kernels that run a
 * whole 3x3 kernel multiply every stored tap), and returns SBNN_ERR_IO for a file that cannot be read, is truncated or corrupt,
 * SBNN_ERR_UNSUPPORTED for another version and SBNN_ERR_SHAPE for inconsistent contents; *out is NULL then.
 */
SBNN_API sbnn_status sbnn_packed_save(const sbnn_packed* p, const char* path);
SBNN_API sbnn_status sbnn_packed_load(const char* path, sbnn_packed** out);

/*
 * Set-up step of the engine for one layer (Section 3.5: the model is converted once, ahead of inference):
 * does now everything that sbnn_conv1x1_gs / sbnn_conv1x1_gs_cm (KH = 1) or sbnn_conv3x3_gs (KH = 3) would
 * otherwise do on first use for activations of up to N x H x W pixels with these flags -- builds the kernels'
 * private weight layouts (for the 1x1 case those of every tile shape the library may choose, whatever the
 * pixel count), raises the kernels' shared-memory limits, and grows the per-device scratch buffer to what
 * the NHWC entry points need for this shape (with SBNN_BF16_TC: what the bf16 mode needs).  Allocates and
 * may synchronise; launches nothing; the activation buffers need not exist yet.  Afterwards compute calls of
 * this layer with no more pixels (3x3: the same W) only enqueue.  Call it once per layer and mode, outside
 * any stream capture.  The scratch buffer never shrinks and an outgrown one is kept until the process exits,
 * so a CUDA graph recorded over an entry point stays valid when a later, larger call makes the buffer grow;
 * growth during a capture is refused with SBNN_ERR_UNSUPPORTED.
 */
SBNN_API sbnn_status sbnn_prepare(const sbnn_packed* w, int N, int H, int W, int flags);

/* ------------------------------------------------------------------------------------------------
 * Group-sparse convolutions (Algorithm 1 for the 1x1 case; Section 3.2's connectivity group
 * pruning of whole 3x3 kernels for the 3x3 case).
 * ------------------------------------------------------------------------------------------------ */

enum {
    SBNN_RELU = 1,    /* apply max(.,0) after the bias */
    SBNN_BF16_TC = 2, /* 1x1 only: round activations and weights to bf16 and contract on tensor cores, fp32 accumulate */
    SBNN_OUT_CM = 4,  /* sbnn_conv1x1_gs_cm only: write the output channel-major, [Cout][ldy] */
    SBNN_BF16_GATHER = 8 /* with SBNN_BF16_TC: contract per group over its kept channels only (warp-level MMA on gathered
                            rows) instead of densely over the masked weights */
};

/*
 * Y[n][y][x][g*G + r] = act( bias[g*G + r] + sum_j val[g][j][r] * X[n][y][x][idx[g][j]] )
 *   w      packed 1x1 layer (KH = KW = 1)
 *   x_dev  [N][H][W][Cin] fp32, y_dev [N][H][W][Cout] fp32
 * Cin must be a multiple of 4 (else SBNN_ERR_UNSUPPORTED).  N*H*W == 0 returns SBNN_OK without a launch.
 * With SBNN_BF16_TC the activations and the kept weights are rounded to bf16 (to nearest even) and the
 * products are summed in fp32 on the tensor cores; bias and ReLU stay fp32.  By default the contraction then runs
 * densely over the masked weights (pruned weights are stored as zeros and multiplied: on the tcgen05 tensor cores
 * that is faster than skipping them, because a group of G <= 8 output channels is too narrow an MMA); this needs
 * Cin % 8 == 0 and Cout % 4 == 0, other shapes -- and every shape when SBNN_BF16_GATHER is added -- run the
 * gathered kernel, which visits kept units only.  Both give the same result up to the order of the fp32 sums.
 * The first call of a layer in either form builds a private re-layout of its weights (allocates and copies
 * synchronously), and both convert X to bf16 in the per-device scratch buffer first.
 */
SBNN_API sbnn_status sbnn_conv1x1_gs(const sbnn_packed* w, const float* x_dev, float* y_dev,
                                     int N, int H, int W, int flags, void* cuda_stream);

/*
 * Same operation with an explicit tile shape, for tuning and for testing every compiled kernel
 * instance: P pixels per lane, GPW groups per warp, NW warps per CTA, KC input channels per
 * pipeline step.  Combinations that were not compiled return SBNN_ERR_UNSUPPORTED.  The first call
 * with a new combination builds a private re-layout of the weights (allocates and copies
 * synchronously); later calls only enqueue.  SBNN_BF16_TC is not accepted here.
 */
SBNN_API sbnn_status sbnn_conv1x1_gs_tuned(const sbnn_packed* w, const float* x_dev, float* y_dev,
                                           int N, int H, int W, int flags, int P, int GPW, int NW, int KC,
                                           void* cuda_stream);

/*
 * Channel-major variant of the 1x1 convolution (same arithmetic as sbnn_conv1x1_gs): the activations
 * are given as xt_dev [Cin][ldx] with the M = N*H*W pixels of a channel contiguous (ldx >= M, a multiple
 * of 4; the padding need not be initialised).  In this layout the kernel's shared-memory tiles are
 * filled by bulk asynchronous copies, which is the fast path for layers bound by arithmetic.
 *   output: y_dev [M][ldy] (pixel-major rows of ldy >= Cout floats), or, with SBNN_OUT_CM, [Cout][ldy]
 *   with ldy >= M; ldy a multiple of 4 in both cases.
 *   P, GPW, NW, KC: tile shape as in sbnn_conv1x1_gs_tuned, or all 0 to let the library choose: the tile
 *   shape whose tiles fill the SMs best for this M, or, when M is so small that even that leaves most SMs
 *   idle (the classifier, batch-1 layers), a kernel that splits the work by 32 pixels x one group instead.
 *   The order of the sums, hence the last bits of the result, can therefore depend on M.
 * sbnn_conv1x1_gs itself takes this path for wide layers (Cin >= 128, M >= 2048): it first copies X
 * into a channel-major scratch buffer kept per device, which it allocates or grows (synchronously) the
 * first time a size is seen.
 * sbnn_to_channel_major converts x_dev [M][C] to xt_dev [C][ld].
 * The scratch buffer is one per device and is also used by the bf16 mode and by sbnn_conv3x3_gs: calls that
 * use it must be ordered on the GPU (same stream, or events); overlapping ones race on it.
 */
SBNN_API sbnn_status sbnn_conv1x1_gs_cm(const sbnn_packed* w, const float* xt_dev, int ldx, float* y_dev, int ldy,
                                        int M, int flags, int P, int GPW, int NW, int KC, void* cuda_stream);
SBNN_API sbnn_status sbnn_to_channel_major(const float* x_dev, float* xt_dev, int M, int C, int ld, void* cuda_stream);

/*
 * 3x3, stride 1, pad 1:
 * Y[n][y][x][g*G + r] = act( bias + sum_j sum_{kh,kw} val[g][j][kh*3+kw][r] * X[n][y+kh-1][x+kw-1][idx[g][j]] ),
 * X taken as zero outside the image.  Shapes as above with KH = KW = 3.  SBNN_BF16_TC is not accepted.
 * W <= 256 and Cin a multiple of 4, else SBNN_ERR_UNSUPPORTED.  The first call with a new image width
 * builds a private re-layout of the weights (allocates and copies synchronously); later calls only enqueue.
 * The input is first copied, channel by channel (image rows padded to a multiple of 4 floats), into a scratch buffer
 * kept per device (allocated or grown synchronously the first time a size is seen).
 */
SBNN_API sbnn_status sbnn_conv3x3_gs(const sbnn_packed* w, const float* x_dev, float* y_dev,
                                     int N, int H, int W, int flags, void* cuda_stream);

/*
 * Channel-major variant of the 3x3 convolution (same arithmetic): the activations are given as xt_dev [Cin][ldx] with
 * the M = N*H*W pixels of a channel contiguous in (n, y, x) order (ldx >= M, a multiple of 4; the padding need not be
 * initialised) -- the layout sbnn_conv1x1_gs_cm reads and, with SBNN_OUT_CM, writes, so 1x1 and 3x3 layers chain
 * without a conversion pass.  This is the layout the pipelined 3x3 kernel stages from; sbnn_conv3x3_gs converts to it first.
 *   output: y_dev [M][ldy] (pixel-major rows of ldy >= Cout floats, ldy a multiple of 4), or, with SBNN_OUT_CM,
 *   [Cout][ldy] with ldy >= M.
 *   flags: SBNN_RELU, SBNN_OUT_CM.
 * W at most 224 (a staged plane row is at most 256 floats), Cin a multiple of 4, else SBNN_ERR_UNSUPPORTED.  For widths that are not multiples of 4 the planes are
 * first copied into the per-device scratch buffer with their rows padded to whole 16-byte units (one extra pass).  The
 * partial sums of tiles that are shared between CTAs live in the per-device scratch buffer (see sbnn_conv1x1_gs_cm for its rules); the first call
 * with a new width builds a private re-layout of the weights and a work plan (allocates and copies synchronously).
 */
SBNN_API sbnn_status sbnn_conv3x3_gs_cm(const sbnn_packed* w, const float* xt_dev, int ldx, float* y_dev, int ldy,
                                        int N, int H, int W, int flags, void* cuda_stream);

/* ------------------------------------------------------------------------------------------------
 * Dense supporting layers of MobileNet-v1 (Section 3.2 names the operators; they stay dense here).
 * ------------------------------------------------------------------------------------------------ */

/*
 * Depthwise 3x3, pad 1, stride 1 or 2:
 * Y[n][y][x][c] = act( b[c] + sum_{kh,kw} w[kh][kw][c] * X[n][s*y+kh-1][s*x+kw-1][c] ).
 *   w_dev [3][3][C], b_dev [C] or NULL, x_dev [N][H][W][C], y_dev [N][Ho][Wo][C], Ho = (H-1)/s + 1.
 * C must be a multiple of 4.
 */
SBNN_API sbnn_status sbnn_dwconv3x3(const float* w_dev, const float* b_dev, const float* x_dev, float* y_dev,
                                    int N, int H, int W, int C, int stride, int flags, void* cuda_stream);

/*
 * The same depthwise convolution on channel-major tensors, as the MobileNet chain runs it: xt_dev [C][ldx] with the
 * pixels of a channel contiguous (index (n*H + y)*W + x), yt_dev [C][ldy] likewise for the output; ldx >= N*H*W,
 * ldy >= N*Ho*Wo, both multiples of 4, both tensors 16-byte aligned; H and W must be divisible by the stride
 * (else SBNN_ERR_UNSUPPORTED).  w_dev [3][3][C], b_dev [C] or NULL.  Any C.  The kernel is chosen by shape
 * (row blocks of 4 for wide maps, column strips for the 14- and 7-wide maps, one output per thread otherwise).
 */
SBNN_API sbnn_status sbnn_dwconv3x3_cm(const float* w_dev, const float* b_dev, const float* xt_dev, int ldx, float* yt_dev,
                                       int ldy, int N, int H, int W, int C, int stride, int flags, void* cuda_stream);

/*
 * Depthwise 3x3 (stride 1, pad 1, dense) followed by a group-sparse 1x1 convolution, as one kernel: the two principal
 * layers of the network (Section 3.2), which follow each other in every block, without the depthwise output ever being
 * written to memory.  Channel-major tensors as in sbnn_dwconv3x3_cm / sbnn_conv1x1_gs_cm:
 *   xt_dev [Cin][ldx] input of the depthwise layer, yt_dev [Cout][ldy] output of the pointwise layer (always channel-major),
 *   dw_w_dev [3][3][Cin], dw_b_dev [Cin] or NULL, pw a packed 1x1 layer with pw->Cin = Cin,
 *   dw_flags / pw_flags: SBNN_RELU or 0 for the activation after each of the two layers.
 * Result: what sbnn_dwconv3x3_cm followed by sbnn_conv1x1_gs_cm gives, up to the order of the fp32 sums (the depthwise
 * result is rounded to fp32 once, as when it is stored).  Takes G = 4 layers and image widths that are multiples of 4
 * up to 124; other shapes return SBNN_ERR_UNSUPPORTED (run the two layers one after the other then).  The first call
 * of a layer builds a private re-layout of its weights (allocates and copies synchronously).
 */
SBNN_API sbnn_status sbnn_dwconv3x3_conv1x1_gs_cm(const sbnn_packed* pw, const float* dw_w_dev, const float* dw_b_dev,
                                                  const float* xt_dev, int ldx, float* yt_dev, int ldy, int N, int H, int W,
                                                  int dw_flags, int pw_flags, void* cuda_stream);

/*
 * Depthwise 3x3 with 3:9 kernel patterns (Section 3.2, DwConv3x3; Algorithm 2): in every row of a kernel the
 * middle weight stays and either the first or the third column is pruned, one pattern per block of go
 * consecutive channels (the paper's PatternInfo; go = 16, or 8 or 4 for channel counts that need it).
 *
 * sbnn_pack_dw_pattern (host only): from dense weights W_host [3][3][C] and mask_host [3][3][C] (1 = kept)
 * writes pattern_host_out [C/go] (bit kh set = the THIRD column of row kh is pruned and the first is kept;
 * clear = the first is pruned) and w6_host_out [3][2][C] (per row: the surviving side weight, then the
 * middle weight).  A mask that is not such a pattern, or that differs inside a block, gives
 * SBNN_ERR_MASK_NOT_GROUP_UNIFORM.  The paper's additional dense ("full-1") pattern is not part of this format:
 * dense channels go through sbnn_dwconv3x3.
 *
 * sbnn_dwconv3x3_pattern: Y as in sbnn_dwconv3x3 with the pruned weights taken as zero; six loads and six
 * FMAs per output.  w6_dev, b_dev, x_dev, y_dev 16-byte aligned device pointers, pattern_dev a device byte array;
 * x_dev [N][H][W][C], y_dev [N][Ho][Wo][C]; stride 1 or 2; go in {4, 8, 16}, C a multiple of go.
 */
SBNN_API sbnn_status sbnn_pack_dw_pattern(const float* W_host, const uint8_t* mask_host, int C, int go,
                                          uint8_t* pattern_host_out, float* w6_host_out);
SBNN_API sbnn_status sbnn_dwconv3x3_pattern(const float* w6_dev, const uint8_t* pattern_dev, int go, const float* b_dev,
                                            const float* x_dev, float* y_dev, int N, int H, int W, int C, int stride,
                                            int flags, void* cuda_stream);

/*
 * Dense 3x3, pad 1, stride 1 or 2, for thin inputs (the network's first layer, Cin = 3):
 *   w_dev [Cout][3][3][Cin], b_dev [Cout] or NULL, x_dev [N][H][W][Cin], y_dev [N][Ho][Wo][Cout].
 * Cin <= 4 and Cout a multiple of 8 and <= 64; other shapes return SBNN_ERR_UNSUPPORTED.
 * x_dev needs 4-byte alignment only.
 */
SBNN_API sbnn_status sbnn_conv3x3_dense(const float* w_dev, const float* b_dev, const float* x_dev, float* y_dev,
                                        int N, int H, int W, int Cin, int Cout, int stride, int flags,
                                        void* cuda_stream);

/* Global average pool: x_dev [N][HW][C] -> y_dev [N][C], C a multiple of 4. */
SBNN_API sbnn_status sbnn_avgpool(const float* x_dev, float* y_dev, int N, int HW, int C, void* cuda_stream);

/* ------------------------------------------------------------------------------------------------
 * MobileNet-v1 (width 1.0, 224x224x3) forward chain (Section 3.5: the sparse inference engine's
 * forward pass; Tables 3 and 4 prune the 13 pointwise layers only).
 * ------------------------------------------------------------------------------------------------ */

typedef struct sbnn_mbv1 sbnn_mbv1;

#define SBNN_MBV1_NUM_BLOCKS 13
#define SBNN_MBV1_NUM_LAYERS 29 /* conv0, 13 x (dw, pw), pool, fc */

/*
 * Bind weights and allocate the two ping-pong activation workspaces for up to max_batch images.
 *   pw[13]        packed pointwise layers, in network order (borrowed; must outlive the network)
 *   fc            packed classifier, 1000 x 1024, any G dividing 1000 (normally a full mask)
 *   dw_w_dev[13]  depthwise weights [3][3][C]; dw_b_dev[13] their biases [C]  (device, borrowed)
 *   conv0_w_dev   [32][3][3][3], conv0_b_dev [32]                               (device, borrowed)
 * Shapes are checked against the network's layer table.
 */
SBNN_API sbnn_status sbnn_mobilenet_v1_create(const sbnn_packed* const* pw, const sbnn_packed* fc,
                                              const float* const* dw_w_dev, const float* const* dw_b_dev,
                                              const float* conv0_w_dev, const float* conv0_b_dev,
                                              int max_batch, sbnn_mbv1** out);

/*
 * Enqueue the whole forward pass for N <= max_batch images on one stream:
 * conv0 -> 13 x (depthwise 3x3 -> group-sparse 1x1) -> average pool -> classifier.
 *   x_dev [N][224][224][3] fp32 (4-byte aligned is enough), logits_dev [N][1000] fp32.
 * Every conv but the classifier applies ReLU.  No host synchronisation.
 * The second call with the same (x_dev, logits_dev, N) records the 29 launches into a CUDA graph (captured on a
 * stream the network owns; nothing of the caller's stream is touched) and from then on such calls launch that
 * graph on cuda_stream, which shortens the gaps between the kernels; up to 8 triples are kept.  If recording
 * fails, or if cuda_stream is itself being captured, the launches are issued one by one as on the first call.
 * Calls on one network are serialised on the host by a lock; the workspaces make concurrent forwards of one
 * network on different streams invalid in any case.
 */
SBNN_API sbnn_status sbnn_mobilenet_v1_forward(sbnn_mbv1* net, const float* x_dev, float* logits_dev,
                                               int N, void* cuda_stream);

/*
 * Run a single layer of the chain on caller-provided input (for layer-isolated checks):
 * layer 0 = conv0, 2i-1 = dw_i, 2i = pw_i (i = 1..13), 27 = pool, 28 = fc.
 * in_dev / out_dev are NHWC buffers of that layer's input / output shape for N images.
 */
SBNN_API sbnn_status sbnn_mobilenet_v1_run_layer(sbnn_mbv1* net, int layer, const float* in_dev, float* out_dev,
                                                 int N, void* cuda_stream);

/*
 * The same layer in the chain's own activation layout, without conversions (what forward launches):
 * in_dev and out_dev are channel-major, [C][ld] with ld = N*side*side rounded up to a multiple of 4 and
 * the pixel index n*side*side + y*side + x (the pool's output has side 1: [1024][N rounded up to 4]).
 * Exceptions: layer 0 reads the NHWC image, the classifier (layer 28) writes [N][1000].
 */
SBNN_API sbnn_status sbnn_mobilenet_v1_run_layer_cm(sbnn_mbv1* net, int layer, const float* in_dev, float* out_dev,
                                                    int N, void* cuda_stream);

/*
 * The first last_layer + 1 layers of the forward pass (Section 3.5), launched exactly as sbnn_mobilenet_v1_forward
 * launches them (same kernels, same workspaces, no CUDA graph of the library's own), with the output of layer
 * last_layer written to out_dev in the chain's layout: channel-major [Cout][ld], ld = N*side*side rounded up to 4
 * (the pool: [1024][N rounded up to 4]; layer 28: the logits [N][1000]).  Gives access to every intermediate
 * activation of the chain, and, by timing consecutive prefixes, to the cost of each layer inside a step.  The call
 * only enqueues; it may be captured into a caller's CUDA graph.  out_dev: 16-byte aligned device memory of the caller.
 */
SBNN_API sbnn_status sbnn_mobilenet_v1_forward_prefix(sbnn_mbv1* net, const float* x_dev, float* out_dev, int N,
                                                      int last_layer, void* cuda_stream);

/* Shape of a layer of the chain: input side, input channels, output side, output channels. */
SBNN_API sbnn_status sbnn_mobilenet_v1_layer_shape(int layer, int* Hin, int* Cin, int* Hout, int* Cout);

SBNN_API sbnn_status sbnn_mobilenet_v1_free(sbnn_mbv1* net);

/*
 * Classifier head without any allocation: logits = classifier(mean over HW of x).
 * (The paper has no counterpart; this entry point exists for deployment only.)
 *
 * Who needs it: callers that may not allocate device memory at the point where they run the head --
 * a serving loop with a latency budget that a cudaMalloc (an implicit device synchronisation) would
 * break, a plug-in living inside another framework's capped memory pool, an application that has
 * frozen its device memory map after start-up.  The ordinary route (sbnn_avgpool, then
 * sbnn_conv1x1_gs) needs a pooled [N][Cin] buffer from the caller; here that buffer is a fixed
 * array of SBNN_HEAD_NOALLOC_MAX_FLOATS floats (256 KiB) inside the library image, resident on every
 * GPU that loads the library until the process exits.
 *
 *   fc          packed 1x1 classifier (any Cout; Cin a multiple of 4), packed while a device was present
 *   x_dev       [N][HW][Cin] fp32, logits_dev [N][Cout] fp32; no ReLU
 *   N * Cin must not exceed SBNN_HEAD_NOALLOC_MAX_FLOATS (e.g. 64 images x 1024 channels), else
 *   SBNN_ERR_SHAPE and nothing is launched.
 * The call uses no cudaMalloc/cudaFree and no allocating library routine; it enqueues two kernels.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, once per
 * device): make that first call outside of any stream capture.  All calls on a device share the one
 * array, which keeps the previous call's values (every element read is rewritten first, nothing
 * needs to start at zero): two calls whose kernels may overlap on the GPU (different streams) race
 * on it -- keep calls on one stream or order them with events.
 */
#define SBNN_HEAD_NOALLOC_MAX_FLOATS 65536
SBNN_API sbnn_status sbnn_head_noalloc(const sbnn_packed* fc, const float* x_dev, float* logits_dev,
                                       int N, int HW, void* cuda_stream);

/*
 * Synchronise the stream and report device-side trouble: SBNN_ERR_CUDA if a kernel failed,
 * SBNN_ERR_TIMEOUT if a bounded wait inside a kernel expired, else SBNN_OK.
 */
SBNN_API sbnn_status sbnn_get_async_status(void* cuda_stream);

/*
 * Diagnostic for the bounded waits of the pipelined kernels: enqueues a one-warp kernel that waits, with a
 * cap of 2000 polls, on a barrier nothing completes.  The kernel gives up, records SBNN_ERR_TIMEOUT in the
 * device status word and returns normally; the next sbnn_get_async_status on the stream reports
 * SBNN_ERR_TIMEOUT once (the word is cleared by that call) and the context stays usable.
 */
SBNN_API sbnn_status sbnn_selftest_wait_timeout(void* cuda_stream);

/*
 * Diagnostic for the roofline of the arithmetic-bound kernels (the paper gives no counterpart: it quotes
 * latencies only, Tables 3 and 4): enqueues a kernel in which 4 CTAs of 512 threads per SM each run
 * `iterations` rounds of 32 packed fp32 FMAs (fma.rn.f32x2, the instruction the convolution kernels use) on
 * registers only, and writes to *flop_out (host, may be NULL) the floating-point operations it performs.
 * Timing it with events on `cuda_stream` gives the FP32 rate this GPU sustains at its current clocks.
 */
SBNN_API sbnn_status sbnn_selftest_fma_rate(int iterations, double* flop_out, void* cuda_stream);

/*
 * Debug aid (the paper has no counterpart): checks the DEVICE copies of a packed layer on the device -- prefix sums
 * monotone and spanning the kept units, indices ascending inside [0, Cin) -- with one thread per group.  A violation
 * sets the device status word; the next sbnn_get_async_status on the stream then returns SBNN_ERR_SHAPE once.  The
 * kernel never traps and reads nothing outside the arrays it is given, so it is safe to run on memory suspected
 * of having been overwritten.  sbnn_debug_poke_device_index is the test hook that goes with it: it overwrites one
 * index of the device copy (the host copy and the private layouts stay as they are) and returns the previous value.
 */
SBNN_API sbnn_status sbnn_debug_check_packed(const sbnn_packed* w, void* cuda_stream);

/*
 * Debug aid (host arithmetic only, needs no GPU; the paper has no counterpart): the work plan of the pipelined 3x3
 * kernel behind sbnn_conv3x3_gs.  That kernel runs `ncta` persistent CTAs; the channel steps of all tiles
 * (group tile `by` outermost, then row tile `bx`, then step k) are laid end to end and cut into `ncta` consecutive
 * shares of equal weight, where step k of group tile `by` weighs block_ptr[by][k+1] - block_ptr[by][k] (the 16-byte
 * words of weights it multiplies) plus a constant.  block_ptr is [ntiles][nchunks + 1], host, non-decreasing per tile.
 * Output: cta_ptr_out [ncta + 1] (host): CTA c owns segments cta_ptr_out[c] .. cta_ptr_out[c+1]-1; segs_out (host,
 * room for seg_capacity segments of 8 ints): {bx, by, k0, k1, part, nparts, slot, counter} -- steps [k0, k1) of tile
 * (bx, by); a tile cut into nparts > 1 segments gets nparts consecutive partial-sum slots from `slot` and one arrival
 * counter (each part stores its sums, the part that arrives last adds them in part order and finishes the tile).
 * *nsegs = segments produced; *nslots, *ncounters (may be NULL) = slots and counters the plan needs.
 * Errors: SBNN_ERR_NULL, SBNN_ERR_SHAPE (non-positive sizes, decreasing block_ptr, seg_capacity too small: *nsegs is
 * still set), SBNN_ERR_ALLOC.
 */
SBNN_API sbnn_status sbnn_debug_plan_conv3x3(const int32_t* block_ptr, int ntiles, int nchunks, int nrow, int ncta,
                                             int32_t* cta_ptr_out, int32_t* segs_out, int seg_capacity, int* nsegs,
                                             int* nslots, int* ncounters);
SBNN_API sbnn_status sbnn_debug_poke_device_index(sbnn_packed* w, long long unit, int value, int* previous);

/*
 * Test hook: overwrite the device number recorded in a packed layer, so that the refusal of compute calls
 * on weights that live on another device can be exercised on a machine with a single GPU.  Not for
 * production use: the device copies themselves do not move.  *previous (may be NULL) receives the number that
 * was recorded, so the test can put it back before freeing the layer.
 */
SBNN_API sbnn_status sbnn_debug_set_packed_device(sbnn_packed* w, int device, int* previous);

#ifdef __cplusplus
}
#endif
#endif /* SBNN_H_ */
