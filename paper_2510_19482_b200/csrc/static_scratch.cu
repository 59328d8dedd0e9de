// elutq_lut_gemm_static: the product of elutq_lut_gemm for callers that must not allocate.
//
// Some users of this library run where a device allocation is off the table: a plugin inside a host
// runtime that hands out all device memory from its own arena at start-up and treats any driver
// allocation as a bug, a latency-critical decode loop that cannot take the device-wide stall of a
// cudaMalloc / cudaFree, or a process that runs under a fixed memory budget.  The other entry points
// get their K-split scratch either from the caller (elutq_lut_gemm_ws) or from buffers the library
// allocates on demand; this one keeps its scratch in a fixed array that is part of the loaded module.
//
// The array below is device memory that every GPU loading the library holds until the process exits
// (4 MiB per GPU).  In host code its name is only a handle: the device address is obtained once per
// device with cudaGetSymbolAddress while that device is current, and that address is what the kernels
// receive.  All calls on a device share the array and it keeps whatever the last call left in it; the
// kernels overwrite every partial sum they later read, so nothing has to be cleared, but two calls
// that overlap on the GPU (different streams) would race on it.
#include <mutex>

#include "common.cuh"

#define ELUTQ_STATIC_SCRATCH_BYTES (4u << 20)

static __device__ __align__(256) unsigned char g_static_scratch[ELUTQ_STATIC_SCRATCH_BYTES];

namespace {

std::mutex g_static_mu;
void* g_static_ptr[64] = {};   // device address of g_static_scratch, per device ordinal

// Device address of the scratch array on the current device (looked up on the first call per device).
int static_scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return elutq::note_cuda_error((int)e);
    if (dev < 0 || dev >= 64) return ELUTQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return elutq::note_cuda_error((int)e);
        if (!p) return ELUTQ_ERR_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return ELUTQ_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int elutq_lut_gemm_static(const void* X, const void* packed, void* Y, int M, int N, int K, void* stream) {
    using namespace elutq;
    if (!X || !packed || !Y) return ELUTQ_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return ELUTQ_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(packed) || !aligned16(Y)) return ELUTQ_ERR_ALIGN;

    // K-split partial sums: one fp32 per (K chunk, activation row, padded output row); chunks are
    // 512 columns wide for M = 1 and 256 columns wide for M > 1
    const size_t n_rb = ((size_t)N + kTileRows - 1) / kTileRows;
    const size_t n_kc = ((size_t)K + kChunkK - 1) / kChunkK;
    const size_t chunks = (M == 1) ? (n_kc > 1 ? n_kc : 0) : 2 * n_kc;
    const size_t need = chunks * (size_t)M * n_rb * kTileRows * sizeof(float);
    if (need > ELUTQ_STATIC_SCRATCH_BYTES) return ELUTQ_ERR_BUFFER_TOO_SMALL;   // shape exceeds the built-in scratch

    int q = 0, G = 0;
    int st = blob_meta(packed, N, K, &q, &G);
    if (st != ELUTQ_OK) return st;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != ELUTQ_OK) return st;

    GemmArgs a;
    a.X = reinterpret_cast<const __half*>(X);
    a.tiles = reinterpret_cast<const uint8_t*>(packed) + ELUTQ_HEADER_BYTES;
    a.Y = Y;
    a.partials = reinterpret_cast<float*>(scratch);
    a.counters = nullptr;
    a.M = M; a.N = N; a.K = K;
    a.n_rb = (int)n_rb; a.n_kc = (int)n_kc;
    a.flags = 0u;
    a.items_q = 0; a.items_r = 0; a.active_warps = 0;
    a.ranges = 0; a.rb_q = 0; a.rb_r = 0; a.cpc = 1; a.cluster_reduce = 0; a.wait_limit = 0;
    const int sms = device_sm_count();
    const int ce = (M == 1) ? launch_lut_gemv(a, q, G, sms, (cudaStream_t)stream)
                            : launch_lut_gemm(a, q, G, sms, (cudaStream_t)stream);
    if (ce != 0) return note_cuda_error(ce);
    return ELUTQ_OK;
}
