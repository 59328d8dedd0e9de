// Shared declarations of the CUDA side: layout geometry, launch descriptors, PTX helpers.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "elutq.h"

namespace elutq {

constexpr int kTileRows = 16;     // output rows per tile (one per lane of a half-warp)
constexpr int kChunkK = 512;      // input columns per tile (64 byte-columns)
constexpr int kMagic = 0x51544C45;
constexpr int kVersion = 1;

// Geometry of the device layout "v1" for one layer.
//   tile = 16 rows x 512 k, stored kc-major (tile = kc * n_rb + rb).
//   Inside a tile: plane vectors uint4 V[2q][32 lanes], then parameter words u32 P[gl*(q+1)/2][32 lanes].
//   lane = 16*h + l: row 16*rb + l, super-groups (128 k each) h and h+2 of the chunk.
//   Step i of a super-group visits column tau(l,i) = w*((a+v)%nsg) + (r+ii)%w,
//   a = l/w, r = l%w, v = i/w, ii = i%w, w = G/8 columns per quantisation group, nsg = 128/G.
struct Geo {
    int q, G, N, K;
    int w, nsg, gl;          // columns per group, groups per super-group, groups per lane
    int n_rb, n_kc;
    int tile_bytes, plane_bytes;
    size_t total_bytes;
};

__host__ __device__ inline Geo make_geo(int q, int G, int N, int K) {
    Geo g;
    g.q = q; g.G = G; g.N = N; g.K = K;
    g.w = G / 8; g.nsg = 128 / G; g.gl = 2 * g.nsg;
    g.n_rb = (N + kTileRows - 1) / kTileRows;
    g.n_kc = (K + kChunkK - 1) / kChunkK;
    g.plane_bytes = 32 * 32 * q;
    g.tile_bytes = g.plane_bytes + 32 * 2 * g.gl * (q + 1);
    g.total_bytes = (size_t)ELUTQ_HEADER_BYTES + (size_t)g.n_kc * g.n_rb * g.tile_bytes;
    return g;
}

// Column visited by lane-row l at step i of a super-group.
__host__ __device__ inline int tau_of(int l, int i, int w, int nsg) {
    const int a = l / w, r = l % w, v = i / w, ii = i % w;
    return w * ((a + v) % nsg) + (r + ii) % w;
}

// Descriptor of one GEMM call handed to the kernel launchers.
struct GemmArgs {
    const __half* X;         // [M][K]
    const uint8_t* tiles;    // packed + header
    void* Y;                 // fp16 or fp32 [M][N]
    float* partials;         // [n_kc][M][n_rb*16] (unused when n_kc == 1)
    unsigned* counters;      // control words of the scratch (may be null): word 0 = device status (0 = fine)
    int M, N, K;
    int n_rb, n_kc;
    unsigned flags;
    int items_q, items_r;    // items per CTA: CTA b owns items_q (+1 if b < items_r) consecutive items
    int active_warps;        // warps that take items (item stride); the rest only help build tables
    int ranges, rb_q, rb_r;  // aligned partition: every chunk is cut into the same `ranges` row ranges (0 = flat
                             // partition of the item list); range r holds rb_q (+1 if r < rb_r) row blocks;
                             // CTA b = group * ranges + r, group = `cpc` consecutive chunks
    int cpc;                 // chunks per CTA in the aligned partition
    int cluster_reduce;      // 1: launched as clusters of n_kc CTAs (one per chunk, same row range): partials stay in
                             //    shared memory and are reduced through distributed shared memory
    unsigned wait_limit;     // poll limit of the tensor-core kernel's bounded waits (0: the default)
};

// Kernel launchers (defined in the .cu files); return a cudaError_t value.
int launch_pack(const uint8_t* planes, const __half* scales, const __half* offsets,
                const Geo& g, uint8_t* packed, cudaStream_t stream);
int launch_unpack(const uint8_t* packed, const Geo& g, uint8_t* planes, __half* scales,
                  __half* offsets, cudaStream_t stream);
int launch_lut_gemv(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream);
int launch_lut_gemm(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream);
int launch_hlq_mma(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream);

// col0 / cols restrict the reduction to output columns [col0, col0 + cols) (cols = 0: all N columns).
int launch_finalize(const GemmArgs& a, int n_chunks, bool pdl, cudaStream_t stream, int col0 = 0, int cols = 0);
void count_launch(unsigned n = 1);

// api.cu helpers shared with other translation units: blob description (registry or header read),
// recording a CUDA error for elutq_last_cuda_error(), SM count of the current device.
int blob_meta(const void* packed, int N, int K, int* q, int* G);
int note_cuda_error(int cuda_error);
int device_sm_count();

// ---- PTX helpers -------------------------------------------------------------------------

// Streaming (read-once) global loads at base + compile-time byte offset.
template <int IMM>
__device__ __forceinline__ uint4 ldg_stream_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4+%5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "n"(IMM));
    return v;
}
template <int IMM>
__device__ __forceinline__ uint32_t ldg_stream_u32(const void* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1+%2];" : "=r"(v) : "l"(p), "n"(IMM));
    return v;
}
// The same loads under a run-time condition (on == 0: no access, the registers keep their values).
template <int IMM>
__device__ __forceinline__ void ldg_stream_v4_if(uint4& v, const void* p, uint32_t on) {
    asm volatile("{\n\t.reg .pred pq;\n\tsetp.ne.u32 pq, %6, 0;\n\t"
                 "@pq ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4+%5];\n\t}"
                 : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w) : "l"(p), "n"(IMM), "r"(on));
}
template <int IMM>
__device__ __forceinline__ void ldg_stream_u32_if(uint32_t& v, const void* p, uint32_t on) {
    asm volatile("{\n\t.reg .pred pq;\n\tsetp.ne.u32 pq, %3, 0;\n\t"
                 "@pq ld.global.nc.L1::no_allocate.u32 %0, [%1+%2];\n\t}" : "+r"(v) : "l"(p), "n"(IMM), "r"(on));
}
// Compile-time loop: f(IntC<I>) for I in [0, N); IntC<I> converts to a constant int.
template <int V>
struct IntC {
    static constexpr int value = V;
    __host__ __device__ constexpr operator int() const { return V; }
};
template <int I, int N, class F>
__device__ __forceinline__ void static_for(F&& f) {
    if constexpr (I < N) {
        f(IntC<I>{});
        static_for<I + 1, N>(f);
    }
}
// prmt.b32 in its default mode: result byte k = byte (sel nibble k & 7) of {b:a}, or that byte's
// sign bit replicated when the nibble's bit 3 is set.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// Packed fp32x2 add (one instruction for two independent fp32 additions, round to nearest even).
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 c;
    asm("{\n\t.reg .b64 ra, rb, rc;\n\t"
        "mov.b64 ra, {%2, %3};\n\t"
        "mov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rc, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rc;\n\t}"
        : "=f"(c.x), "=f"(c.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return c;
}
// Writes one finished output value Y[idx] (fp32 or fp16, optionally accumulating).
__device__ __forceinline__ void store_out(const GemmArgs& a, size_t idx, float y) {
    if (a.flags & ELUTQ_FLAG_OUT_F32) {
        float* Yf = reinterpret_cast<float*>(a.Y);
        Yf[idx] = (a.flags & ELUTQ_FLAG_ACCUMULATE) ? Yf[idx] + y : y;
    } else {
        __half* Yh = reinterpret_cast<__half*>(a.Y);
        if (a.flags & ELUTQ_FLAG_ACCUMULATE) y += __half2float(Yh[idx]);
        Yh[idx] = __float2half_rn(y);
    }
}
// Thread-block cluster helpers (distributed shared memory).
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(const float* local_smem_ptr, unsigned cta_rank) {
    const uint32_t local = (uint32_t)__cvta_generic_to_shared(local_smem_ptr);
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(cta_rank));
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}
// Device status codes (word 0 of the control area; read back by elutq_device_status / elutq_chain_status).
constexpr unsigned kStatusWaitExpired = 0x7C05u;    // a bounded wait ran out
constexpr unsigned kStatusBlobMismatch = 0x7C0Bu;
// Internal flag (never accepted from callers; set by elutq_test_wait_expiry only): the tensor-core kernel's issuing
// thread issues no MMA and no commit, so that the other threads' bounded waits for MMA completion run out.
constexpr unsigned kFlagTestNoMma = 0x20000000u;   // the blob header does not describe what the kernel was launched for

// Every GEMM kernel compares the header of the blob it was handed with the geometry it was launched for before it
// reads any tile: a stale description of an address that now holds another blob must never turn into reads
// past the end of the buffer.  `tiles` points just behind the 128-byte header.  On mismatch the status word is
// raised and the caller returns without touching the tiles (every thread sees the same header, so a CTA
// leaves as a whole).
__device__ __forceinline__ void blob_header_load(const uint8_t* tiles, uint4& h0, uint2& h1) {
    h0 = __ldg(reinterpret_cast<const uint4*>(tiles - ELUTQ_HEADER_BYTES));
    h1 = __ldg(reinterpret_cast<const uint2*>(tiles - ELUTQ_HEADER_BYTES + 16));
}
__device__ __forceinline__ bool blob_header_ok(const uint4& h0, const uint2& h1, int q, int G, int N, int K) {
    return h0.x == (uint32_t)kMagic && h0.y == (uint32_t)kVersion && h0.z == (uint32_t)q && h0.w == (uint32_t)G &&
           h1.x == (uint32_t)N && h1.y == (uint32_t)K;
}
__device__ __forceinline__ bool blob_header_matches(const uint8_t* tiles, int q, int G, int N, int K, unsigned* status) {
    uint4 h0;
    uint2 h1;
    blob_header_load(tiles, h0, h1);
    const bool ok = blob_header_ok(h0, h1, q, G, N, K);
    if (!ok && status != nullptr && threadIdx.x == 0) atomicExch(status, kStatusBlobMismatch);
    return ok;
}

// Programmatic dependent launch: wait for the preceding grid's memory, allow the next grid to start.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace elutq
