// MobileNet-v1 (width 1.0, 224x224x3) forward chain: the engine's forward pass of Section 3.5
// with the 13 pointwise layers group-sparse (the layers Tables 3 and 4 prune) and everything
// else dense.  Launches only: conv0 -> 13 x (depthwise, pointwise) -> pool -> classifier on one
// stream over two ping-pong workspaces.  Between the image and the pooled features every
// activation is kept channel-major ([C][ld], the pixels of a channel contiguous), the layout in
// which the group-sparse 1x1 kernel's tiles are plain row copies; no layer transposes anything.
#include <new>

#include "common.h"

namespace sbnn {
namespace {

struct LayerShape {
    int kind;  // 0 conv0, 1 dw, 2 pw, 3 pool, 4 fc
    int hin, cin, hout, cout, stride;
};

// Network table (Howard et al. 2017, Table 1).
struct Table {
    LayerShape t[SBNN_MBV1_NUM_LAYERS];
    Table() {
        static const int chans[SBNN_MBV1_NUM_BLOCKS][3] = {
            {32, 64, 1},   {64, 128, 2},  {128, 128, 1}, {128, 256, 2}, {256, 256, 1}, {256, 512, 2}, {512, 512, 1},
            {512, 512, 1}, {512, 512, 1}, {512, 512, 1}, {512, 512, 1}, {512, 1024, 2}, {1024, 1024, 1}};
        int n = 0, h = 112;
        t[n++] = {0, 224, 3, 112, 32, 2};
        for (int i = 0; i < SBNN_MBV1_NUM_BLOCKS; ++i) {
            const int ci = chans[i][0], co = chans[i][1], s = chans[i][2];
            t[n++] = {1, h, ci, h / s, ci, s};
            h /= s;
            t[n++] = {2, h, ci, h, co, 1};
        }
        t[n++] = {3, 7, 1024, 1, 1024, 1};
        t[n++] = {4, 1, 1024, 1, 1000, 1};
    }
};

const LayerShape* layer_table() {
    static const Table tab;
    return tab.t;
}

inline int round4(long long v) { return (int)((v + 3) / 4 * 4); }

}  // namespace
}  // namespace sbnn

struct sbnn_mbv1 {
    const sbnn_packed* pw[SBNN_MBV1_NUM_BLOCKS];
    const sbnn_packed* fc;
    const float* dw_w[SBNN_MBV1_NUM_BLOCKS];
    const float* dw_b[SBNN_MBV1_NUM_BLOCKS];
    const float* c0_w;
    const float* c0_b;
    int max_batch;
    int device;
    float* ws[2];  // ping-pong activation buffers
    // Forward calls replay a CUDA graph of the 29 launches once a (x, logits, N) triple has been seen twice:
    // the first call runs plainly (and builds whatever is built lazily), the second is captured on a private
    // stream and instantiated, later ones only launch the graph on the caller's stream.
    struct GraphKey {
        const float* x;
        float* y;
        int n;
        bool operator<(const GraphKey& o) const {
            if (x != o.x) return x < o.x;
            if (y != o.y) return y < o.y;
            return n < o.n;
        }
    };
    struct GraphEntry {
        cudaGraphExec_t exec = nullptr;
        int seen = 0;
        bool failed = false;
    };
    std::mutex mu;
    std::map<GraphKey, GraphEntry> graphs;
    cudaStream_t capture_stream = nullptr;
};

using namespace sbnn;

extern "C" sbnn_status sbnn_mobilenet_v1_layer_shape(int layer, int* Hin, int* Cin, int* Hout, int* Cout) {
    clear_error();
    if (layer < 0 || layer >= SBNN_MBV1_NUM_LAYERS) return fail(SBNN_ERR_SHAPE, "layer %d out of range", layer);
    const LayerShape& L = layer_table()[layer];
    if (Hin) *Hin = L.hin;
    if (Cin) *Cin = L.cin;
    if (Hout) *Hout = L.hout;
    if (Cout) *Cout = L.cout;
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_mobilenet_v1_create(const sbnn_packed* const* pw, const sbnn_packed* fc,
                                                const float* const* dw_w_dev, const float* const* dw_b_dev,
                                                const float* conv0_w_dev, const float* conv0_b_dev, int max_batch,
                                                sbnn_mbv1** out) {
    clear_error();
    if (!pw || !fc || !dw_w_dev || !dw_b_dev || !conv0_w_dev || !conv0_b_dev || !out)
        return fail(SBNN_ERR_NULL, "all arguments must be non-NULL");
    *out = nullptr;
    if (max_batch <= 0) return fail(SBNN_ERR_SHAPE, "max_batch=%d must be positive", max_batch);
    const LayerShape* T = layer_table();
    for (int i = 0; i < SBNN_MBV1_NUM_BLOCKS; ++i) {
        const LayerShape& L = T[2 + 2 * i];
        if (!pw[i] || !dw_w_dev[i] || !dw_b_dev[i]) return fail(SBNN_ERR_NULL, "block %d has a NULL weight pointer", i + 1);
        if (pw[i]->KH != 1 || pw[i]->Cin != L.cin || pw[i]->Cout != L.cout)
            return fail(SBNN_ERR_SHAPE, "pointwise layer %d is %d->%d (k=%d), expected %d->%d 1x1", i + 1, pw[i]->Cin,
                        pw[i]->Cout, pw[i]->KH, L.cin, L.cout);
        if (!aligned16(dw_w_dev[i]) || !aligned16(dw_b_dev[i]))
            return fail(SBNN_ERR_ALIGN, "depthwise weights of block %d not 16-byte aligned", i + 1);
    }
    if (fc->KH != 1 || fc->Cin != 1024 || fc->Cout != 1000) return fail(SBNN_ERR_SHAPE, "classifier must be 1024->1000 1x1");
    sbnn_status st = check_device();
    if (st != SBNN_OK) return st;
    // The kernel-private weight layouts of the channel-major 1x1 kernel are built here, not in forward.
    for (int i = 0; i < SBNN_MBV1_NUM_BLOCKS; ++i) {
        if ((st = check_packed_device(pw[i])) != SBNN_OK) return st;
        const int hw = layer_table()[2 + 2 * i].hin;                 // the block's pointwise layer is entry 2 + 2*i
        if ((st = prepare_default_cm(pw[i], (long long)max_batch * hw * hw)) != SBNN_OK) return st;
        if ((st = prepare_default_cm(pw[i], (long long)hw * hw)) != SBNN_OK) return st;   // and the batch-1 choice
    }
    if ((st = check_packed_device(fc)) != SBNN_OK) return st;
    if ((st = prepare_default_cm(fc, max_batch)) != SBNN_OK) return st;
    sbnn_mbv1* n = new (std::nothrow) sbnn_mbv1;
    if (!n) return fail(SBNN_ERR_ALLOC, "out of host memory");
    for (int i = 0; i < SBNN_MBV1_NUM_BLOCKS; ++i) {
        n->pw[i] = pw[i];
        n->dw_w[i] = dw_w_dev[i];
        n->dw_b[i] = dw_b_dev[i];
    }
    n->fc = fc; n->c0_w = conv0_w_dev; n->c0_b = conv0_b_dev; n->max_batch = max_batch;
    n->ws[0] = n->ws[1] = nullptr;
    cudaGetDevice(&n->device);
    if (cudaStreamCreateWithFlags(&n->capture_stream, cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        n->capture_stream = nullptr;   // forward then always launches plainly
    }
    // Largest activation: pw1's output, 112*112*64 floats per image (+ row padding of the layout).
    const size_t bytes = ((size_t)max_batch * 112 * 112 * 64 + 4 * 1024) * sizeof(float);
    for (int i = 0; i < 2; ++i) {
        cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&n->ws[i]), bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            sbnn_mobilenet_v1_free(n);
            return fail(SBNN_ERR_ALLOC, "workspace of %zu bytes: %s", bytes, cudaGetErrorString(e));
        }
    }
    *out = n;
    return SBNN_OK;
}

namespace {

// SBNN_OK if the network's weights and workspaces live on the current device.
sbnn_status check_net_device(const sbnn_mbv1* net) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "no usable CUDA device");
    }
    if (dev != net->device)
        return fail(SBNN_ERR_CUDA, "the network was created on device %d, the current device is %d", net->device, dev);
    return SBNN_OK;
}

// One layer on channel-major buffers.  in: channel-major [Cin][ld_in] (layer 0: the NHWC image);
// out: channel-major [Cout][ld_out] (pool: [N][C]; classifier: [N][1000], reading the pooled [N][C]).
sbnn_status run_cm(sbnn_mbv1* net, int layer, const float* in, float* out, int N, void* stream) {
    const LayerShape& L = layer_table()[layer];
    const int blk = (layer - 1) / 2;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int ld_in = round4((long long)N * L.hin * L.hin), ld_out = round4((long long)N * L.hout * L.hout);
    switch (L.kind) {
        case 0: return launch_conv3x3_thin_cm(net->c0_w, net->c0_b, in, out, ld_out, N, L.hin, L.hin, L.cin, L.cout, L.stride, 1, st);
        case 1: return launch_dwconv3x3_cm(net->dw_w[blk], net->dw_b[blk], in, ld_in, out, ld_out, N, L.hin, L.hin, L.cin, L.stride, 1, st);
        case 2: return sbnn_conv1x1_gs_cm(net->pw[blk], in, ld_in, out, ld_out, N * L.hin * L.hin, SBNN_RELU | SBNN_OUT_CM, 0, 0, 0, 0, stream);
        case 3: return launch_avgpool_cm(in, ld_in, out, round4(N), N, L.hin * L.hin, L.cin, st);
        default: {   // classifier: pooled features [1024][ld] in, logits [N][1000] out (few pixels: the entry point picks the kernel)
            return sbnn_conv1x1_gs_cm(net->fc, in, round4(N), out, L.cout, N, 0, 0, 0, 0, 0, stream);
        }
    }
}

}  // namespace

extern "C" sbnn_status sbnn_mobilenet_v1_run_layer(sbnn_mbv1* net, int layer, const float* in, float* outp, int N,
                                                   void* stream) {
    clear_error();
    if (!net || !in || !outp) return fail(SBNN_ERR_NULL, "net, in_dev and out_dev must not be NULL");
    if (layer < 0 || layer >= SBNN_MBV1_NUM_LAYERS) return fail(SBNN_ERR_SHAPE, "layer %d out of range", layer);
    if (N < 0 || N > net->max_batch) return fail(SBNN_ERR_SHAPE, "N=%d outside [0, max_batch=%d]", N, net->max_batch);
    if (N == 0) return SBNN_OK;
    sbnn_status r = check_net_device(net);
    if (r != SBNN_OK) return r;
    // The chain's kernels work on channel-major buffers; this entry point takes and returns NHWC, so
    // it converts on the way in and out through the network's own workspaces.
    const LayerShape& L = layer_table()[layer];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int M_in = N * L.hin * L.hin, M_out = N * L.hout * L.hout;
    const int ld_in = round4(M_in), ld_out = round4(M_out);
    const float* src = in;
    if (L.kind != 0) {                                                                   // NHWC [M][C] -> [C][ld]
        if ((r = launch_transpose(in, L.cin, net->ws[0], ld_in, M_in, L.cin, st)) != SBNN_OK) return r;
        src = net->ws[0];
    }
    if (L.kind == 4) return run_cm(net, layer, src, outp, N, stream);                    // classifier writes [N][1000] directly
    if ((r = run_cm(net, layer, src, net->ws[1], N, stream)) != SBNN_OK) return r;
    return launch_transpose(net->ws[1], ld_out, outp, L.cout, L.cout, M_out, st);        // [C][ld] -> NHWC
}

extern "C" sbnn_status sbnn_mobilenet_v1_run_layer_cm(sbnn_mbv1* net, int layer, const float* in, float* outp, int N,
                                                      void* stream) {
    clear_error();
    if (!net || !in || !outp) return fail(SBNN_ERR_NULL, "net, in_dev and out_dev must not be NULL");
    if (layer < 0 || layer >= SBNN_MBV1_NUM_LAYERS) return fail(SBNN_ERR_SHAPE, "layer %d out of range", layer);
    if (N < 0 || N > net->max_batch) return fail(SBNN_ERR_SHAPE, "N=%d outside [0, max_batch=%d]", N, net->max_batch);
    if (!aligned16(in) || !aligned16(outp)) return fail(SBNN_ERR_ALIGN, "in_dev and out_dev must be 16-byte aligned");
    if (N == 0) return SBNN_OK;
    sbnn_status r = check_net_device(net);
    if (r != SBNN_OK) return r;
    return run_cm(net, layer, in, outp, N, stream);
}

namespace {

// Layers 0 .. last on the ping-pong workspaces; the output of layer `last` goes to out_dev.
sbnn_status forward_plain(sbnn_mbv1* net, const float* x_dev, float* out_dev, int N, void* stream,
                          int last = SBNN_MBV1_NUM_LAYERS - 1) {
    // The kernels are launched with programmatic stream serialization: each may become resident and run its
    // set-up (barrier initialisation, weight fetches) while its predecessor drains, and waits for the
    // predecessor's completion before it touches an activation buffer.
    ChainedLaunchScope chained;
    const float* cur = x_dev;
    for (int l = 0; l <= last; ++l) {
        float* dst = (l == last) ? out_dev : net->ws[l & 1];
        sbnn_status st = run_cm(net, l, cur, dst, N, stream);
        if (st != SBNN_OK) return st;
        cur = dst;
    }
    return SBNN_OK;
}

void drop_graphs(sbnn_mbv1* net) {
    for (auto& kv : net->graphs)
        if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    net->graphs.clear();
}

constexpr size_t kMaxGraphs = 8;

}  // namespace

extern "C" sbnn_status sbnn_mobilenet_v1_forward(sbnn_mbv1* net, const float* x_dev, float* logits_dev, int N,
                                                 void* stream) {
    clear_error();
    if (!net || !x_dev || !logits_dev) return fail(SBNN_ERR_NULL, "net, x_dev and logits_dev must not be NULL");
    if (N < 0 || N > net->max_batch) return fail(SBNN_ERR_SHAPE, "N=%d outside [0, max_batch=%d]", N, net->max_batch);
    if (!aligned16(logits_dev)) return fail(SBNN_ERR_ALIGN, "logits_dev must be 16-byte aligned");
    if (N == 0) return SBNN_OK;
    sbnn_status dr = check_net_device(net);
    if (dr != SBNN_OK) return dr;
    cudaStream_t user = static_cast<cudaStream_t>(stream);
    // A caller that is itself capturing gets the plain launches recorded into its own graph.
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(user, &cs) != cudaSuccess) cudaGetLastError();
    if (cs != cudaStreamCaptureStatusNone) return forward_plain(net, x_dev, logits_dev, N, stream);

    std::lock_guard<std::mutex> lk(net->mu);
    if (net->graphs.size() >= kMaxGraphs && !net->graphs.count({x_dev, logits_dev, N})) drop_graphs(net);
    sbnn_mbv1::GraphEntry& e = net->graphs[{x_dev, logits_dev, N}];
    if (e.exec) {
        SBNN_CUDA_TRY(cudaGraphLaunch(e.exec, user));
        return SBNN_OK;
    }
    if (e.failed || e.seen++ == 0 || !net->capture_stream) return forward_plain(net, x_dev, logits_dev, N, stream);
    // second call with these buffers: record the launches on the private stream (nothing runs there)
    cudaGraph_t graph = nullptr;
    sbnn_status r = SBNN_ERR_CUDA;
    if (cudaStreamBeginCapture(net->capture_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        r = forward_plain(net, x_dev, logits_dev, N, net->capture_stream);
        if (cudaStreamEndCapture(net->capture_stream, &graph) != cudaSuccess || !graph) r = SBNN_ERR_CUDA;
    }
    if (r == SBNN_OK && cudaGraphInstantiate(&e.exec, graph, 0) != cudaSuccess) {
        e.exec = nullptr;
        r = SBNN_ERR_CUDA;
    }
    if (graph) cudaGraphDestroy(graph);
    if (r != SBNN_OK) {          // no graph for these buffers: keep launching plainly
        cudaGetLastError();
        clear_error();
        e.failed = true;
        return forward_plain(net, x_dev, logits_dev, N, stream);
    }
    SBNN_CUDA_TRY(cudaGraphLaunch(e.exec, user));
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_mobilenet_v1_forward_prefix(sbnn_mbv1* net, const float* x_dev, float* out_dev, int N,
                                                        int last_layer, void* stream) {
    clear_error();
    if (!net || !x_dev || !out_dev) return fail(SBNN_ERR_NULL, "net, x_dev and out_dev must not be NULL");
    if (last_layer < 0 || last_layer >= SBNN_MBV1_NUM_LAYERS) return fail(SBNN_ERR_SHAPE, "layer %d out of range", last_layer);
    if (N < 0 || N > net->max_batch) return fail(SBNN_ERR_SHAPE, "N=%d outside [0, max_batch=%d]", N, net->max_batch);
    if (!aligned16(out_dev)) return fail(SBNN_ERR_ALIGN, "out_dev must be 16-byte aligned");
    if (out_dev == net->ws[0] || out_dev == net->ws[1]) return fail(SBNN_ERR_SHAPE, "out_dev must not be a workspace of the network");
    if (N == 0) return SBNN_OK;
    sbnn_status r = check_net_device(net);
    if (r != SBNN_OK) return r;
    std::lock_guard<std::mutex> lk(net->mu);
    return forward_plain(net, x_dev, out_dev, N, stream, last_layer);
}

extern "C" sbnn_status sbnn_mobilenet_v1_free(sbnn_mbv1* net) {
    clear_error();
    if (!net) return SBNN_OK;
    drop_graphs(net);
    if (net->capture_stream) cudaStreamDestroy(net->capture_stream);
    cudaFree(net->ws[0]);
    cudaFree(net->ws[1]);
    cudaGetLastError();
    delete net;
    return SBNN_OK;
}
