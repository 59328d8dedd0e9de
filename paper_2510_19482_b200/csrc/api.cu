// extern "C" boundary: argument validation, blob registry, scratch management, dispatch.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <unordered_map>
#include <vector>
#include <utility>

#include "common.cuh"

namespace elutq {

namespace {

thread_local int g_last_cuda_error = 0;
thread_local unsigned g_test_flags = 0;        // set around one call by elutq_test_wait_expiry
thread_local unsigned g_test_wait_limit = 0;
std::atomic<unsigned long long> g_launches{0};

struct BlobMeta { int q, G, N, K; };
std::mutex g_mu;
std::unordered_map<const void*, BlobMeta> g_blobs;

struct Scratch { void* ptr = nullptr; size_t bytes = 0; };
// Buffers that a larger request has replaced.  They are kept until elutq_release_scratch: a CUDA graph captured
// earlier holds their addresses as kernel arguments, and work enqueued earlier may still be running on them.
std::vector<void*> g_parked;
// keyed by (device, stream, kind): kind 0 = arrival counters (always zero between calls), 1 = X staging,
// 2 = Y staging, 3 = K-split partial sums.  Counters live in a buffer of their own so that no other data
// is ever written where a later call with a different shape expects zeroed counters.
std::map<std::tuple<int, void*, int>, Scratch> g_scratch;
int g_num_sms[64] = {};

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return ELUTQ_ERR_CUDA;
}

int check_shape(int q, int G, int N, int K) {
    if (N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    if (q < 1 || q > 4) return ELUTQ_ERR_SHAPE;
    if (G != 32 && G != 64 && G != 128) return ELUTQ_ERR_SHAPE;
    if (K % G != 0) return ELUTQ_ERR_SHAPE;
    return ELUTQ_OK;
}

int num_sms() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (g_num_sms[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        g_num_sms[dev] = n;
    }
    return g_num_sms[dev];
}

// Workspace layout: a 256-byte control area (word 0 = device status), then the partial sums.
size_t counters_bytes(int, int) { return 256; }
size_t partials_bytes(int M, int N, int K) {
    const size_t n_rb = (size_t)(N + kTileRows - 1) / kTileRows;
    const size_t n_kc = (size_t)(K + kChunkK - 1) / kChunkK;
    // M = 1: one partial per 512-column chunk (none when there is a single chunk);
    // M > 1: one per 256-column half chunk
    const size_t chunks = (M == 1) ? (n_kc > 1 ? n_kc : 0) : 2 * n_kc;
    return chunks * (size_t)M * n_rb * kTileRows * sizeof(float);
}

int lookup_blob(const void* packed, int N, int K, BlobMeta* out, bool force_read = false) {
    if (!force_read) {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_blobs.find(packed);
        if (it != g_blobs.end() && it->second.N == N && it->second.K == K) {
            *out = it->second;
            return ELUTQ_OK;
        }
        // unknown address, or an entry left by a blob that has since been freed and its address
        // reused: read the header that is there now
    }
    uint32_t hdr[ELUTQ_HEADER_BYTES / 4];
    cudaError_t e = cudaMemcpy(hdr, packed, sizeof(hdr), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (hdr[0] != (uint32_t)kMagic || hdr[1] != (uint32_t)kVersion) return ELUTQ_ERR_SHAPE;
    BlobMeta m{(int)hdr[2], (int)hdr[3], (int)hdr[4], (int)hdr[5]};
    if (check_shape(m.q, m.G, m.N, m.K) != ELUTQ_OK || m.N != N || m.K != K) return ELUTQ_ERR_SHAPE;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_blobs[packed] = m;
    }
    *out = m;
    return ELUTQ_OK;
}

// Library-owned scratch of at least `bytes` for (current device, stream, kind); counters zeroed on (re)allocation.
// A buffer that has to grow is replaced, never freed (see g_parked).  Nothing is allocated while the stream is being
// captured: the request fails with ELUTQ_ERR_BUFFER_TOO_SMALL instead (reserve before capturing).
int get_scratch(void* stream, int kind, size_t bytes, bool zero, void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    std::lock_guard<std::mutex> lk(g_mu);
    Scratch& s = g_scratch[std::make_tuple(dev, stream, kind)];
    if (s.bytes < bytes) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing((cudaStream_t)stream, &cap);
        if (e != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
        if (cap != cudaStreamCaptureStatusNone) return ELUTQ_ERR_BUFFER_TOO_SMALL;
        size_t want = bytes < (1u << 20) ? (1u << 20) : bytes;
        void* fresh = nullptr;
        e = cudaMalloc(&fresh, want);
        if (e != cudaSuccess) return cuda_fail(e);
        if (zero) {
            e = cudaMemsetAsync(fresh, 0, want, (cudaStream_t)stream);
            if (e != cudaSuccess) { cudaFree(fresh); return cuda_fail(e); }
        }
        if (s.ptr) g_parked.push_back(s.ptr);
        s.ptr = fresh;
        s.bytes = want;
    }
    *out = s.ptr;
    return ELUTQ_OK;
}

// Device-side address of a pinned, mapped host pointer, or nullptr when the device cannot address it.
const void* host_device_pointer(const void* host) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) return nullptr;
    return at.devicePointer;
}

// dst[0 .. bytes) = src[0 .. bytes), 16 bytes per thread (bytes is a multiple of 16 for K % 8 == 0; the tail is
// copied by halves).  src is host memory addressed by the device.
__global__ void __launch_bounds__(256) copy_in_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, size_t bytes) {
    grid_launch_dependents();
    grid_dependency_wait();          // stream order: whatever preceded the call (it may have produced X) is complete
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
    if (i + 16 <= bytes) *reinterpret_cast<uint4*>(dst + i) = *reinterpret_cast<const uint4*>(src + i);
    else
        for (size_t j = i; j < bytes; j += 2) *reinterpret_cast<uint16_t*>(dst + j) = *reinterpret_cast<const uint16_t*>(src + j);
}

int launch_copy_in(const void* src, void* dst, size_t bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((bytes + 16 * 256 - 1) / (16 * 256)));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, copy_in_kernel, reinterpret_cast<const uint8_t*>(src), reinterpret_cast<uint8_t*>(dst), bytes);
    count_launch(1);
    return (int)e;
}

// Which kernel family a batched call runs on (the crossover depends on the shape: see ELUTQ_TENSOR_MIN_M_NARROW).
bool takes_tensor_path(int M, int N, int G, unsigned flags) {
    const unsigned lut_variants = ELUTQ_FLAG_PLAIN_G4 | ELUTQ_FLAG_CLUSTER_REDUCE | ELUTQ_FLAG_MIRROR | ELUTQ_FLAG_LUT_ONLY |
                                  ELUTQ_FLAG_TABLE_F16 | ELUTQ_FLAG_TABLE_I8;
    if (G != 128 || (flags & lut_variants)) return false;
    return M >= ELUTQ_TENSOR_MIN_M || (M >= ELUTQ_TENSOR_MIN_M_NARROW && N <= ELUTQ_TENSOR_NARROW_N);
}

int run_gemm(const void* X, const void* packed, void* Y, int M, int N, int K, unsigned flags,
             void* workspace, size_t workspace_bytes, bool own_workspace, void* stream) {
    if (!X || !packed || !Y) return ELUTQ_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    if ((flags & ELUTQ_FLAG_SKIP_OFFSET) && (flags & ELUTQ_FLAG_OFFSET_ONLY)) return ELUTQ_ERR_INVALID_ARG;
    if (flags & ~0x3ffu) return ELUTQ_ERR_INVALID_ARG;
    if ((flags & ELUTQ_FLAG_TABLE_F16) && (flags & ELUTQ_FLAG_TABLE_I8)) return ELUTQ_ERR_INVALID_ARG;
    if ((flags & ELUTQ_FLAG_PLAIN_G4) && (flags & ELUTQ_FLAG_MIRROR)) return ELUTQ_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(packed, 16) || !aligned(Y, 16)) return ELUTQ_ERR_ALIGN;
    BlobMeta m;
    int st = lookup_blob(packed, N, K, &m);
    if (st != ELUTQ_OK) return st;
    if ((flags & (ELUTQ_FLAG_PLAIN_G4 | ELUTQ_FLAG_MIRROR | ELUTQ_FLAG_TABLE_F16 | ELUTQ_FLAG_TABLE_I8)) && m.G != 128) return ELUTQ_ERR_UNSUPPORTED;
    // decode-kernel variants exist for M = 1 only
    if ((flags & (ELUTQ_FLAG_PLAIN_G4 | ELUTQ_FLAG_MIRROR | ELUTQ_FLAG_CLUSTER_REDUCE)) && M > 1) return ELUTQ_ERR_UNSUPPORTED;

    const size_t cb = counters_bytes(M, N), pb = partials_bytes(M, N, K);
    void* counters = workspace;
    void* partials = nullptr;
    if (own_workspace) {
        st = get_scratch(stream, 0, cb, true, &counters);
        if (st != ELUTQ_OK) return st;
        st = get_scratch(stream, 3, pb ? pb : 16, false, &partials);
        if (st != ELUTQ_OK) return st;
    } else {
        if (!workspace) return ELUTQ_ERR_INVALID_ARG;
        if (!aligned(workspace, 16)) return ELUTQ_ERR_ALIGN;
        if (workspace_bytes < cb + pb) return ELUTQ_ERR_BUFFER_TOO_SMALL;
        partials = reinterpret_cast<uint8_t*>(workspace) + cb;
    }

    const Geo g = make_geo(m.q, m.G, N, K);
    GemmArgs a;
    a.X = reinterpret_cast<const __half*>(X);
    a.tiles = reinterpret_cast<const uint8_t*>(packed) + ELUTQ_HEADER_BYTES;
    a.Y = Y;
    a.counters = reinterpret_cast<unsigned*>(counters);
    a.partials = reinterpret_cast<float*>(partials);
    a.M = M; a.N = N; a.K = K;
    a.n_rb = g.n_rb; a.n_kc = g.n_kc;
    a.flags = flags | g_test_flags;
    a.wait_limit = g_test_wait_limit;
    a.items_q = 0; a.items_r = 0; a.active_warps = 0; a.ranges = 0; a.rb_q = 0; a.rb_r = 0; a.cpc = 1; a.cluster_reduce = 0;
    const int sms = num_sms();
    int ce;
    if (M == 1) ce = launch_lut_gemv(a, m.q, m.G, sms, (cudaStream_t)stream);
    else if (takes_tensor_path(M, N, m.G, flags)) ce = launch_hlq_mma(a, m.q, m.G, sms, (cudaStream_t)stream);
    else ce = launch_lut_gemm(a, m.q, m.G, sms, (cudaStream_t)stream);
    if (ce == (int)cudaErrorNotSupported) return ELUTQ_ERR_UNSUPPORTED;
    if (ce != 0) return cuda_fail((cudaError_t)ce);
    return ELUTQ_OK;
}

}  // namespace

void count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Helpers for entry points that live in other translation units.
int blob_meta(const void* packed, int N, int K, int* q, int* G) {
    BlobMeta m;
    const int st = lookup_blob(packed, N, K, &m);
    if (st != ELUTQ_OK) return st;
    *q = m.q;
    *G = m.G;
    return ELUTQ_OK;
}
int note_cuda_error(int cuda_error) { return cuda_fail((cudaError_t)cuda_error); }
int device_sm_count() { return num_sms(); }

}  // namespace elutq

using namespace elutq;

extern "C" {

const char* elutq_status_string(int status) {
    switch (status) {
        case ELUTQ_OK: return "ok";
        case ELUTQ_ERR_INVALID_ARG: return "invalid argument";
        case ELUTQ_ERR_SHAPE: return "shape or format mismatch";
        case ELUTQ_ERR_ALIGN: return "misaligned pointer";
        case ELUTQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case ELUTQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case ELUTQ_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

int elutq_last_cuda_error(void) { return g_last_cuda_error; }

unsigned long long elutq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int elutq_packed_bytes(int q, int G, int N, int K, size_t* bytes) {
    if (!bytes) return ELUTQ_ERR_INVALID_ARG;
    int st = check_shape(q, G, N, K);
    if (st != ELUTQ_OK) return st;
    *bytes = make_geo(q, G, N, K).total_bytes;
    return ELUTQ_OK;
}

int elutq_pack(const uint8_t* planes, const void* scales, const void* offsets, int q, int G, int N, int K,
               void* packed, size_t packed_bytes, void* stream) {
    if (!planes || !scales || !offsets || !packed) return ELUTQ_ERR_INVALID_ARG;
    int st = check_shape(q, G, N, K);
    if (st != ELUTQ_OK) return st;
    if (!aligned(planes, 8) || !aligned(scales, 2) || !aligned(offsets, 2) || !aligned(packed, 16)) return ELUTQ_ERR_ALIGN;
    const Geo g = make_geo(q, G, N, K);
    if (packed_bytes < g.total_bytes) return ELUTQ_ERR_BUFFER_TOO_SMALL;
    int ce = launch_pack(planes, reinterpret_cast<const __half*>(scales), reinterpret_cast<const __half*>(offsets), g,
                         reinterpret_cast<uint8_t*>(packed), (cudaStream_t)stream);
    if (ce != 0) return cuda_fail((cudaError_t)ce);
    std::lock_guard<std::mutex> lk(g_mu);
    g_blobs[packed] = BlobMeta{q, G, N, K};
    return ELUTQ_OK;
}

int elutq_unpack(const void* packed, int N, int K, uint8_t* planes, void* scales, void* offsets, void* stream) {
    if (!packed || !planes || !scales || !offsets) return ELUTQ_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(planes, 8) || !aligned(scales, 2) || !aligned(offsets, 2)) return ELUTQ_ERR_ALIGN;
    BlobMeta m;
    int st = lookup_blob(packed, N, K, &m);
    if (st != ELUTQ_OK) return st;
    const Geo g = make_geo(m.q, m.G, N, K);
    int ce = launch_unpack(reinterpret_cast<const uint8_t*>(packed), g, planes, reinterpret_cast<__half*>(scales),
                           reinterpret_cast<__half*>(offsets), (cudaStream_t)stream);
    if (ce != 0) return cuda_fail((cudaError_t)ce);
    return ELUTQ_OK;
}

int elutq_describe(const void* packed, int N, int K, int* q, int* G) {
    if (!packed || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    BlobMeta m;
    int st = lookup_blob(packed, N, K, &m, true);     // always the header that is there now, never a remembered one
    if (st != ELUTQ_OK) return st;
    if (q) *q = m.q;
    if (G) *G = m.G;
    return ELUTQ_OK;
}

int elutq_forget(const void* packed) {
    if (!packed) return ELUTQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_mu);
    g_blobs.erase(packed);
    return ELUTQ_OK;
}

int elutq_workspace_bytes(int M, int N, int K, size_t* bytes) {
    if (!bytes || M <= 0 || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    *bytes = counters_bytes(M, N) + partials_bytes(M, N, K);
    return ELUTQ_OK;
}

int elutq_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes == 0) return ELUTQ_ERR_INVALID_ARG;
    if (!aligned(workspace, 16)) return ELUTQ_ERR_ALIGN;
    cudaError_t e = cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    return ELUTQ_OK;
}

int elutq_lut_gemm(const void* X, const void* packed, void* Y, int M, int N, int K, void* stream) {
    return run_gemm(X, packed, Y, M, N, K, 0u, nullptr, 0, true, stream);
}

int elutq_lut_gemm_bias(const void* X, const void* packed, void* Y, int M, int N, int K, int accumulate, void* stream) {
    const unsigned flags = ELUTQ_FLAG_OFFSET_ONLY | (accumulate ? ELUTQ_FLAG_ACCUMULATE : 0u);
    return run_gemm(X, packed, Y, M, N, K, flags, nullptr, 0, true, stream);
}

int elutq_lut_gemm_f32(const void* X, const void* packed, float* Y, int M, int N, int K, unsigned flags, void* stream) {
    return run_gemm(X, packed, Y, M, N, K, flags | ELUTQ_FLAG_OUT_F32, nullptr, 0, true, stream);
}

int elutq_lut_gemm_ws(const void* X, const void* packed, void* Y, int M, int N, int K, unsigned flags,
                      void* workspace, size_t workspace_bytes, void* stream) {
    return run_gemm(X, packed, Y, M, N, K, flags, workspace, workspace_bytes, false, stream);
}

int elutq_lut_gemm_host(const void* X_host, const void* packed, void* Y_host, int M, int N, int K, void* stream) {
    if (!X_host || !packed || !Y_host) return ELUTQ_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    const size_t xb = (size_t)M * K * sizeof(__half), yb = (size_t)M * N * sizeof(__half);
    void *xd = nullptr, *yd = nullptr;
    int st = get_scratch(stream, 1, xb, false, &xd);
    if (st != ELUTQ_OK) return st;
    // Pinned host buffers that the device can address (any cudaHostAlloc / registered memory under unified
    // addressing): a small kernel pulls X across the bus into the staging buffer and the epilogue stores Y straight
    // into host memory, both chained to the GEMM kernels by programmatic dependent launch.  This avoids the two
    // copy-engine operations per call, which cost several microseconds each for a few kilobytes.
    // Only for small transfers (decode and small batches): large ones are faster through the copy engines
    // (measured on the prefill step: 69 against 21 GB/s).
    const bool small = xb + yb <= ((size_t)1 << 20);
    const void* x_map = small ? host_device_pointer(X_host) : nullptr;
    void* y_map = small ? const_cast<void*>(host_device_pointer(Y_host)) : nullptr;
    if (x_map && y_map && aligned(x_map, 16) && aligned(y_map, 16)) {
        int ce = launch_copy_in(x_map, xd, xb, (cudaStream_t)stream);
        if (ce != 0) return cuda_fail((cudaError_t)ce);
        return run_gemm(xd, packed, y_map, M, N, K, 0u, nullptr, 0, true, stream);
    }
    st = get_scratch(stream, 2, yb, false, &yd);
    if (st != ELUTQ_OK) return st;
    cudaError_t e = cudaMemcpyAsync(xd, X_host, xb, cudaMemcpyHostToDevice, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    st = run_gemm(xd, packed, yd, M, N, K, 0u, nullptr, 0, true, stream);
    if (st != ELUTQ_OK) return st;
    e = cudaMemcpyAsync(Y_host, yd, yb, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    return ELUTQ_OK;
}

int elutq_test_wait_expiry(const void* X, const void* packed, float* Y, int M, int N, int K, unsigned wait_limit, void* stream) {
    if (M < ELUTQ_TENSOR_MIN_M || M > 128 || wait_limit == 0) return ELUTQ_ERR_UNSUPPORTED;   // the one-token-tile schedule only
    if (K < 3 * 128) return ELUTQ_ERR_UNSUPPORTED;                                           // a wait needs a third K step
    g_test_flags = kFlagTestNoMma;
    g_test_wait_limit = wait_limit;
    const int st = run_gemm(X, packed, Y, M, N, K, ELUTQ_FLAG_OUT_F32, nullptr, 0, true, stream);
    g_test_flags = 0;
    g_test_wait_limit = 0;
    return st;
}

int elutq_device_status(void* stream, int* status) {
    if (!status) return ELUTQ_ERR_INVALID_ARG;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    void* ptr = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_scratch.find(std::make_tuple(dev, stream, 0));
        if (it != g_scratch.end()) ptr = it->second.ptr;
    }
    *status = 0;
    e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!ptr) return ELUTQ_OK;
    unsigned word = 0;
    e = cudaMemcpy(&word, ptr, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    *status = (int)word;
    return ELUTQ_OK;
}

int elutq_release_scratch(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    cudaError_t first = cudaSuccess;
    for (auto& kv : g_scratch) {
        if (kv.second.ptr) {
            cudaError_t e = cudaFree(kv.second.ptr);
            if (e != cudaSuccess && first == cudaSuccess) first = e;
        }
    }
    g_scratch.clear();
    for (void* p : g_parked) {
        cudaError_t e = cudaFree(p);
        if (e != cudaSuccess && first == cudaSuccess) first = e;
    }
    g_parked.clear();
    if (first != cudaSuccess) return cuda_fail(first);
    return ELUTQ_OK;
}

int elutq_takes_tensor_path(int M, int N, int K, int G, unsigned flags) {
    (void)K;
    return M > 1 && takes_tensor_path(M, N, G, flags) ? 1 : 0;
}

int elutq_reserve(int M, int N, int K, void* stream) {
    if (M <= 0 || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    void* p = nullptr;
    int st = get_scratch(stream, 0, counters_bytes(M, N), true, &p);
    if (st != ELUTQ_OK) return st;
    const size_t pb = partials_bytes(M, N, K);
    st = get_scratch(stream, 3, pb ? pb : 16, false, &p);
    if (st != ELUTQ_OK) return st;
    st = get_scratch(stream, 1, (size_t)M * K * sizeof(__half), false, &p);
    if (st != ELUTQ_OK) return st;
    return get_scratch(stream, 2, (size_t)M * N * sizeof(__half), false, &p);
}

int elutq_scratch_address(void* stream, int kind, void** ptr, size_t* bytes) {
    if (!ptr || kind < 0 || kind > 3) return ELUTQ_ERR_INVALID_ARG;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_scratch.find(std::make_tuple(dev, stream, kind));
    *ptr = it == g_scratch.end() ? nullptr : it->second.ptr;
    if (bytes) *bytes = it == g_scratch.end() ? 0 : it->second.bytes;
    return ELUTQ_OK;
}

}  // extern "C"
