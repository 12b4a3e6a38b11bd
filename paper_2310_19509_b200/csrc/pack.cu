// Status strings, error text, and the host-side packer of group-sparse weights
// (the conversion step of Section 3.5; Algorithm 1's "sparse info" becomes the
// per-group list of kept input channels).
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <utility>

#include "common.h"

namespace sbnn {

static thread_local char g_err[512] = "";

sbnn_status fail(sbnn_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

void clear_error() { g_err[0] = 0; }

sbnn_status check_device() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(e));
    }
    static std::mutex mu;
    static std::map<int, int> major_of;
    int major = 0;
    {
        std::lock_guard<std::mutex> lk(mu);
        auto it = major_of.find(dev);
        if (it == major_of.end()) {
            e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
            if (e != cudaSuccess) {
                cudaGetLastError();
                return fail(SBNN_ERR_CUDA, "cannot query device %d: %s", dev, cudaGetErrorString(e));
            }
            major_of[dev] = major;
        } else {
            major = it->second;
        }
    }
    if (major != 10)
        return fail(SBNN_ERR_ARCH, "device %d has compute capability %d.x; this library is built for 10.x", dev, major);
    return SBNN_OK;
}

sbnn_status check_packed_device(const sbnn_packed* w) {
    if (w->device < 0) return fail(SBNN_ERR_CUDA, "packed weights have no device copy (packed without a CUDA device)");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(SBNN_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(e));
    }
    if (dev != w->device)
        return fail(SBNN_ERR_CUDA, "weights were packed on device %d, the current device is %d", w->device, dev);
    return SBNN_OK;
}

static thread_local int g_prepare_depth = 0;
bool prepare_only() { return g_prepare_depth > 0; }
PrepareScope::PrepareScope() { ++g_prepare_depth; }
PrepareScope::~PrepareScope() { --g_prepare_depth; }

static thread_local int g_chained_depth = 0;
bool chained_launch() { return g_chained_depth > 0; }
ChainedLaunchScope::ChainedLaunchScope() { ++g_chained_depth; }
ChainedLaunchScope::~ChainedLaunchScope() { --g_chained_depth; }

sbnn_status set_max_dyn_smem(const void* func, int bytes) {
    static std::mutex mu;
    static std::map<std::pair<int, const void*>, int> limit;
    int dev = 0;
    SBNN_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    int& cur = limit[{dev, func}];
    if (bytes > cur) {
        SBNN_CUDA_TRY(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        cur = bytes;
    }
    return SBNN_OK;
}

static bool supported_group(int G) { return G == 1 || G == 2 || G == 4 || G == 8 || G == 16; }

template <typename T>
static sbnn_status upload(T** dst, const std::vector<T>& src) {
    // At least one whole unit of the widest group (16 floats): kernels that fetch a unit ahead read unit 0 of an
    // empty layer, which must be addressable (and is zero).
    const size_t bytes = std::max<size_t>(src.size() * sizeof(T), 64);
    SBNN_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(dst), bytes));
    if (src.size() * sizeof(T) < 64) SBNN_CUDA_TRY(cudaMemset(*dst, 0, bytes));
    if (!src.empty()) SBNN_CUDA_TRY(cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice));
    return SBNN_OK;
}

}  // namespace sbnn

using namespace sbnn;

extern "C" const char* sbnn_status_str(sbnn_status s) {
    switch (s) {
        case SBNN_OK: return "SBNN_OK";
        case SBNN_ERR_NULL: return "SBNN_ERR_NULL";
        case SBNN_ERR_SHAPE: return "SBNN_ERR_SHAPE";
        case SBNN_ERR_GROUP: return "SBNN_ERR_GROUP";
        case SBNN_ERR_MASK_NOT_GROUP_UNIFORM: return "SBNN_ERR_MASK_NOT_GROUP_UNIFORM";
        case SBNN_ERR_ALIGN: return "SBNN_ERR_ALIGN";
        case SBNN_ERR_UNSUPPORTED: return "SBNN_ERR_UNSUPPORTED";
        case SBNN_ERR_ARCH: return "SBNN_ERR_ARCH";
        case SBNN_ERR_ALLOC: return "SBNN_ERR_ALLOC";
        case SBNN_ERR_CUDA: return "SBNN_ERR_CUDA";
        case SBNN_ERR_TIMEOUT: return "SBNN_ERR_TIMEOUT";
        case SBNN_ERR_IO: return "SBNN_ERR_IO";
    }
    return "SBNN_ERR_UNKNOWN";
}

extern "C" const char* sbnn_last_error(void) { return g_err; }

namespace {
// The paper's own Conv1x1 format groups gi = 4 consecutive input channels with the go = G output channels of a group
// (Section 3.2) and stores one index per block (Algorithm 1's SD).  A layer whose every group keeps aligned runs of 4
// channels is such a layer: record the block size and the per-block index list, a quarter of the per-channel one.
void detect_blocks(sbnn_packed* p) {
    p->gi = 1;
    p->block_idx.clear();
    if (p->Cin % 4 || p->nnz == 0 || p->nnz % 4) return;
    for (int g = 0; g < p->ngroups; ++g) {
        const int64_t lo = p->group_ptr[g], hi = p->group_ptr[g + 1];
        if ((hi - lo) % 4) return;
        for (int64_t u = lo; u < hi; u += 4)
            if (p->idx[u] % 4 || p->idx[u + 1] != p->idx[u] + 1 || p->idx[u + 2] != p->idx[u] + 2 || p->idx[u + 3] != p->idx[u] + 3) return;
    }
    p->block_idx.resize(p->nnz / 4);
    for (int64_t b = 0; b < p->nnz / 4; ++b) p->block_idx[b] = p->idx[4 * b];
    p->gi = 4;
}

// Last step of packing and of loading: device copies of the canonical arrays and the default private layouts, if
// there is a device; *out owns p afterwards (on failure p is freed).
sbnn_status finish_packed(sbnn_packed* p, sbnn_packed** out) {
    try {
        detect_blocks(p);
    } catch (const std::bad_alloc&) {
        p->gi = 1;
        p->block_idx.clear();
    }
    int ndev = 0, dev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0 || cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        *out = p;
        return SBNN_OK;
    }
    sbnn_status st = SBNN_OK;
    p->device = dev;
    if ((st = upload(&p->d_group_ptr, p->group_ptr)) != SBNN_OK || (st = upload(&p->d_idx, p->idx)) != SBNN_OK ||
        (st = upload(&p->d_val, p->val)) != SBNN_OK || (st = upload(&p->d_bias, p->bias)) != SBNN_OK) {
        sbnn_packed_free(p);
        return st;
    }
    st = (p->KH == 1) ? prepare_default_1x1(p) : prepare_default_3x3(p);
    if (st != SBNN_OK) {
        sbnn_packed_free(p);
        return st;
    }
    *out = p;
    return SBNN_OK;
}

// tap_patterns = false: a unit's mask is one value for all taps (connectivity pruning only).
// tap_patterns = true: the taps of a unit may differ (kernel patterns), but not between the G filters of the group;
// a unit is kept if any of its taps is, pruned taps are stored as zeros and remembered in tap_mask.
sbnn_status pack_impl(const float* W, const uint8_t* mask, const float* bias, int Cout, int KH, int KW, int Cin, int G,
                      bool tap_patterns, sbnn_packed** out) {
    clear_error();
    if (!W || !mask || !out) return fail(SBNN_ERR_NULL, "W_host, mask_host and out must not be NULL");
    *out = nullptr;
    if (Cout <= 0 || Cin <= 0) return fail(SBNN_ERR_SHAPE, "Cout=%d and Cin=%d must be positive", Cout, Cin);
    if (!((KH == 1 && KW == 1) || (KH == 3 && KW == 3)))
        return fail(SBNN_ERR_SHAPE, "kernel %dx%d: only 1x1 and 3x3", KH, KW);
    if (!supported_group(G)) return fail(SBNN_ERR_GROUP, "G=%d not in {1,2,4,8,16}", G);
    if (Cout % G) return fail(SBNN_ERR_GROUP, "Cout=%d is not a multiple of G=%d", Cout, G);

    sbnn_packed* p = new (std::nothrow) sbnn_packed;
    if (!p) return fail(SBNN_ERR_ALLOC, "out of host memory");
    p->Cout = Cout; p->KH = KH; p->KW = KW; p->Cin = Cin; p->G = G; p->ngroups = Cout / G;
    const int taps = KH * KW;
    const int64_t row = (int64_t)taps * Cin;  // elements per output channel
    try {
        p->group_ptr.assign(p->ngroups + 1, 0);
        p->bias.assign(Cout, 0.0f);
        if (bias) memcpy(p->bias.data(), bias, sizeof(float) * Cout);
        // Pass 1: validate the mask's structure and count the kept units.
        std::vector<uint16_t> unit_taps((size_t)p->ngroups * Cin, 0);   // bit t = tap t of the unit is kept
        for (int g = 0; g < p->ngroups; ++g) {
            const uint8_t* m0 = mask + (int64_t)g * G * row;  // first row, first tap
            int kept = 0;
            for (int c = 0; c < Cin; ++c) {
                unsigned bits = 0;
                for (int t = 0; t < taps; ++t) {
                    const uint8_t ref = m0[(int64_t)t * Cin + c];
                    if (ref > 1) {
                        delete p;
                        return fail(SBNN_ERR_MASK_NOT_GROUP_UNIFORM, "mask value %d at group %d channel %d is not 0/1", ref, g, c);
                    }
                    if (!tap_patterns && ref != m0[c]) {
                        delete p;
                        return fail(SBNN_ERR_MASK_NOT_GROUP_UNIFORM, "mask of group %d differs at row 0 tap %d channel %d", g, t, c);
                    }
                    for (int r = 1; r < G; ++r)
                        if (m0[(int64_t)r * row + (int64_t)t * Cin + c] != ref) {
                            delete p;
                            return fail(SBNN_ERR_MASK_NOT_GROUP_UNIFORM,
                                        "mask of group %d differs at row %d tap %d channel %d", g, r, t, c);
                        }
                    bits |= (unsigned)ref << t;
                }
                unit_taps[(size_t)g * Cin + c] = (uint16_t)bits;
                kept += bits != 0;
            }
            p->group_ptr[g + 1] = p->group_ptr[g] + kept;
        }
        p->nnz = p->group_ptr[p->ngroups];
        p->idx.resize(p->nnz);
        p->val.resize((size_t)p->nnz * taps * G);
        if (tap_patterns) p->tap_mask.resize(p->nnz);
        // Pass 2: emit ascending indices and the [taps][G] value block of every kept unit.
        for (int g = 0; g < p->ngroups; ++g) {
            const float* w0 = W + (int64_t)g * G * row;
            int64_t u = p->group_ptr[g];
            for (int c = 0; c < Cin; ++c) {
                const unsigned bits = unit_taps[(size_t)g * Cin + c];
                if (!bits) continue;
                p->idx[u] = c;
                if (tap_patterns) p->tap_mask[u] = (uint16_t)bits;
                float* v = p->val.data() + (size_t)u * taps * G;
                for (int t = 0; t < taps; ++t)
                    for (int r = 0; r < G; ++r)
                        v[t * G + r] = ((bits >> t) & 1u) ? w0[(int64_t)r * row + (int64_t)t * Cin + c] : 0.0f;
                ++u;
            }
        }
    } catch (const std::bad_alloc&) {
        delete p;
        return fail(SBNN_ERR_ALLOC, "out of host memory while packing");
    }

    return finish_packed(p, out);
}
}  // namespace

extern "C" sbnn_status sbnn_pack_weights(const float* W, const uint8_t* mask, const float* bias, int Cout, int KH,
                                         int KW, int Cin, int G, sbnn_packed** out) {
    return pack_impl(W, mask, bias, Cout, KH, KW, Cin, G, false, out);
}

extern "C" sbnn_status sbnn_pack_weights_pattern(const float* W, const uint8_t* mask, const float* bias, int Cout, int KH,
                                                 int KW, int Cin, int G, sbnn_packed** out) {
    return pack_impl(W, mask, bias, Cout, KH, KW, Cin, G, true, out);
}

extern "C" sbnn_status sbnn_packed_get(const sbnn_packed* p, sbnn_packed_view* v) {
    clear_error();
    if (!p || !v) return fail(SBNN_ERR_NULL, "packed and view must not be NULL");
    v->Cout = p->Cout; v->KH = p->KH; v->KW = p->KW; v->Cin = p->Cin; v->G = p->G; v->ngroups = p->ngroups;
    v->nnz_units = p->nnz;
    v->group_ptr = p->group_ptr.data();
    v->idx = p->idx.data();
    v->val = p->val.data();
    v->bias = p->bias.data();
    v->tap_mask = p->tap_mask.empty() ? nullptr : p->tap_mask.data();
    v->gi = p->gi;
    v->block_idx = p->block_idx.empty() ? nullptr : p->block_idx.data();
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_unpack_weights(const sbnn_packed* p, float* W, uint8_t* mask) {
    clear_error();
    if (!p) return fail(SBNN_ERR_NULL, "packed must not be NULL");
    const int taps = p->KH * p->KW, G = p->G;
    const int64_t row = (int64_t)taps * p->Cin;
    if (W) memset(W, 0, sizeof(float) * row * p->Cout);
    if (mask) memset(mask, 0, (size_t)row * p->Cout);
    for (int g = 0; g < p->ngroups; ++g)
        for (int64_t u = p->group_ptr[g]; u < p->group_ptr[g + 1]; ++u) {
            const int c = p->idx[u];
            const float* v = p->val.data() + (size_t)u * taps * G;
            for (int t = 0; t < taps; ++t)
                for (int r = 0; r < G; ++r) {
                    int64_t o = ((int64_t)g * G + r) * row + (int64_t)t * p->Cin + c;
                    if (W) W[o] = v[t * G + r];
                    if (mask) mask[o] = p->tap_mask.empty() ? 1 : (uint8_t)((p->tap_mask[u] >> t) & 1u);
                }
        }
    return SBNN_OK;
}

// ---- packed-layer files ------------------------------------------------------------------------------------
namespace {
const unsigned char kFileMagic[8] = {'S', 'B', 'N', 'N', 'P', 'K', 1, 0};

// FNV-1a, 64 bit, over the bytes of the file that precede the checksum.
struct Fnv {
    uint64_t h = 1469598103934665603ull;
    void add(const void* data, size_t n) {
        const unsigned char* b = static_cast<const unsigned char*>(data);
        for (size_t i = 0; i < n; ++i) h = (h ^ b[i]) * 1099511628211ull;
    }
};

struct FileCloser {
    FILE* f;
    ~FileCloser() { if (f) fclose(f); }
};
}  // namespace

extern "C" sbnn_status sbnn_packed_save(const sbnn_packed* p, const char* path) {
    clear_error();
    if (!p || !path) return fail(SBNN_ERR_NULL, "packed and path must not be NULL");
    FileCloser fc{fopen(path, "wb")};
    if (!fc.f) return fail(SBNN_ERR_IO, "cannot open %s for writing", path);
    Fnv sum;
    bool ok = true;
    auto put = [&](const void* d, size_t n) {
        sum.add(d, n);
        ok = ok && (n == 0 || fwrite(d, 1, n, fc.f) == n);
    };
    const bool blocks = p->gi == 4 && !p->block_idx.empty();   // indices are then stored once per run of 4
    const int32_t hdr[8] = {1, p->Cout, p->KH, p->KW, p->Cin, p->G, p->tap_mask.empty() ? 0 : 1, blocks ? 4 : 0};
    const int64_t nnz = p->nnz;
    put(kFileMagic, 8);
    put(hdr, sizeof(hdr));
    put(&nnz, 8);
    put(p->group_ptr.data(), p->group_ptr.size() * 4);
    if (blocks) put(p->block_idx.data(), p->block_idx.size() * 4);
    else put(p->idx.data(), p->idx.size() * 4);
    put(p->val.data(), p->val.size() * 4);
    put(p->bias.data(), p->bias.size() * 4);
    put(p->tap_mask.data(), p->tap_mask.size() * 2);
    const uint64_t h = sum.h;
    ok = ok && fwrite(&h, 1, 8, fc.f) == 8;
    ok = ok && fflush(fc.f) == 0;
    if (!ok) return fail(SBNN_ERR_IO, "short write to %s", path);
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_packed_load(const char* path, sbnn_packed** out) {
    clear_error();
    if (!path || !out) return fail(SBNN_ERR_NULL, "path and out must not be NULL");
    *out = nullptr;
    FileCloser fc{fopen(path, "rb")};
    if (!fc.f) return fail(SBNN_ERR_IO, "cannot open %s", path);
    Fnv sum;
    bool ok = true;
    auto get = [&](void* d, size_t n) {
        ok = ok && (n == 0 || fread(d, 1, n, fc.f) == n);
        if (ok) sum.add(d, n);
    };
    unsigned char magic[8];
    int32_t hdr[8];
    int64_t nnz = 0;
    get(magic, 8);
    get(hdr, sizeof(hdr));
    get(&nnz, 8);
    if (!ok) return fail(SBNN_ERR_IO, "%s is too short to be a packed layer", path);
    if (memcmp(magic, kFileMagic, 8) != 0) return fail(SBNN_ERR_IO, "%s is not a packed-layer file (bad magic)", path);
    if (hdr[0] != 1) return fail(SBNN_ERR_UNSUPPORTED, "%s has format version %d, this library reads version 1", path, hdr[0]);
    const int Cout = hdr[1], KH = hdr[2], KW = hdr[3], Cin = hdr[4], G = hdr[5], has_taps = hdr[6], file_gi = hdr[7];
    if (Cout <= 0 || Cin <= 0 || !((KH == 1 && KW == 1) || (KH == 3 && KW == 3)) || !supported_group(G) || Cout % G ||
        (has_taps != 0 && has_taps != 1) || (file_gi != 0 && file_gi != 4) || (file_gi == 4 && (nnz % 4 || Cin % 4)) || nnz < 0 ||
        nnz > (int64_t)(Cout / G) * Cin)
        return fail(SBNN_ERR_SHAPE, "%s: inconsistent header (Cout=%d KH=%d KW=%d Cin=%d G=%d units=%lld)", path, Cout, KH, KW, Cin,
                    G, (long long)nnz);
    sbnn_packed* p = new (std::nothrow) sbnn_packed;
    if (!p) return fail(SBNN_ERR_ALLOC, "out of host memory");
    p->Cout = Cout; p->KH = KH; p->KW = KW; p->Cin = Cin; p->G = G; p->ngroups = Cout / G; p->nnz = nnz;
    const int taps = KH * KW;
    try {
        p->group_ptr.resize(p->ngroups + 1);
        p->idx.resize(nnz);
        p->val.resize((size_t)nnz * taps * G);
        p->bias.resize(Cout);
        if (has_taps) p->tap_mask.resize(nnz);
    } catch (const std::bad_alloc&) {
        delete p;
        return fail(SBNN_ERR_ALLOC, "out of host memory while loading %s", path);
    }
    get(p->group_ptr.data(), p->group_ptr.size() * 4);
    if (file_gi == 4) {   // one index per run of 4 consecutive channels
        std::vector<int32_t> blk;
        try {
            blk.resize(nnz / 4);
        } catch (const std::bad_alloc&) {
            delete p;
            return fail(SBNN_ERR_ALLOC, "out of host memory while loading %s", path);
        }
        get(blk.data(), blk.size() * 4);
        for (int64_t b = 0; ok && b < nnz / 4; ++b)
            for (int e = 0; e < 4; ++e) p->idx[4 * b + e] = blk[b] + e;
    } else {
        get(p->idx.data(), p->idx.size() * 4);
    }
    get(p->val.data(), p->val.size() * 4);
    get(p->bias.data(), p->bias.size() * 4);
    get(p->tap_mask.data(), p->tap_mask.size() * 2);
    uint64_t stored = 0;
    const uint64_t computed = sum.h;
    const bool have_sum = ok && fread(&stored, 1, 8, fc.f) == 8;
    unsigned char extra;
    const bool trailing = have_sum && fread(&extra, 1, 1, fc.f) == 1;
    sbnn_status st = SBNN_OK;
    if (!ok || !have_sum) st = fail(SBNN_ERR_IO, "%s is truncated", path);
    else if (trailing) st = fail(SBNN_ERR_IO, "%s has bytes after the checksum", path);
    else if (stored != computed) st = fail(SBNN_ERR_IO, "%s: checksum mismatch (file is corrupt)", path);
    // structure: prefix sums, ascending in-range indices, tap masks inside the kernel and not empty
    if (st == SBNN_OK && (p->group_ptr[0] != 0 || p->group_ptr[p->ngroups] != nnz))
        st = fail(SBNN_ERR_SHAPE, "%s: group_ptr does not span the kept units", path);
    for (int g = 0; st == SBNN_OK && g < p->ngroups; ++g) {
        const int64_t lo = p->group_ptr[g], hi = p->group_ptr[g + 1];
        if (lo > hi || hi > nnz) st = fail(SBNN_ERR_SHAPE, "%s: group_ptr is not monotone at group %d", path, g);
        for (int64_t u = lo; st == SBNN_OK && u < hi; ++u) {
            if (p->idx[u] < 0 || p->idx[u] >= Cin || (u > lo && p->idx[u] <= p->idx[u - 1]))
                st = fail(SBNN_ERR_SHAPE, "%s: indices of group %d are not ascending inside [0, Cin)", path, g);
            else if (has_taps && (p->tap_mask[u] == 0 || (p->tap_mask[u] >> taps) != 0))
                st = fail(SBNN_ERR_SHAPE, "%s: tap mask of unit %lld is empty or reaches outside the kernel", path, (long long)u);
        }
    }
    if (st != SBNN_OK) {
        delete p;
        return st;
    }
    // The weights of pruned taps are zeros, as the packer writes them: kernels that run a whole 3x3 kernel multiply them.
    if (has_taps) {
        for (int64_t u = 0; u < nnz; ++u)
            for (int t = 0; t < taps; ++t)
                if (!((p->tap_mask[u] >> t) & 1u))
                    for (int r = 0; r < p->G; ++r) p->val[((size_t)u * taps + t) * p->G + r] = 0.0f;
    }
    return finish_packed(p, out);
}

extern "C" sbnn_status sbnn_packed_free(sbnn_packed* p) {
    clear_error();
    if (!p) return SBNN_OK;
    if (p->device >= 0) {
        int cur = 0;
        bool sw = cudaGetDevice(&cur) == cudaSuccess && cur != p->device && cudaSetDevice(p->device) == cudaSuccess;
        free_streams_1x1(p);
        free_streams_cm(p);
        free_stream_bf16(p);
        free_umma_weights(p);
        free_streams_3x3(p);
        cudaFree(p->d_group_ptr);
        cudaFree(p->d_idx);
        cudaFree(p->d_val);
        cudaFree(p->d_bias);
        if (sw) cudaSetDevice(cur);
        cudaGetLastError();
    }
    delete p;
    return SBNN_OK;
}

extern "C" sbnn_status sbnn_get_async_status(void* stream) {
    clear_error();
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail(SBNN_ERR_CUDA, "stream failed: %s", cudaGetErrorString(e));
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(SBNN_ERR_CUDA, "pending error: %s", cudaGetErrorString(e));
    int word = 0;
    sbnn_status st = read_async_status(&word);
    if (st != SBNN_OK) return st;
    if (word == SBNN_ERR_TIMEOUT) return fail(SBNN_ERR_TIMEOUT, "a bounded wait inside a kernel gave up");
    if (word) return fail((sbnn_status)word, "a device-side check failed (device status %d)", word);
    return SBNN_OK;
}
