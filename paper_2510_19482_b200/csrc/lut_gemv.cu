// M = 1 decode kernel: bit-serial LUT GEMV over HLQ weights (Appendix B procedure, Eq. 3 parameters).
//
// Work decomposition
//   item  = one tile of the packed layout: 16 output rows x 512 input columns (all q planes,
//           their scales and offsets), processed by one warp.
//   CTA   = 16 warps; owns a contiguous range of the kc-major item list, so it needs the
//           activation tables of one K chunk at a time (rebuilt when the range crosses a chunk).
//   lane  = 16*h + l: output row l of the tile, super-groups h and h+2 (128 columns each).
//
// Tables (step "LUT build"): for every byte-column c of the chunk (8 activations) the 256
// partial sums T[p][c] = sum_i bit_i(p) * x[8c+i] are formed as A[p & 15] + B[p >> 4], the two
// g = 4 tables of the column's half-slices, and stored at byte offset p*256 + c*4.  All lanes
// of a warp therefore address bank c: the packed layout rotates each row's bytes so that at
// every step the 32 lanes of a warp use 32 different columns (no bank conflicts), and the
// address is a single byte-permute of (weight byte, lane column).
//
// Look-up / accumulate: per (group, plane) the lane sums its 16 (G=128) table entries in fp32,
// multiplies by the group's per-plane scale, adds offset * group activation sum, and the two
// half-warps are combined with one shuffle.
//
// K split: one partial per K chunk goes to the workspace; the warp that arrives last at a row
// block (arrival counter, wraps to zero) adds the partials in a fixed order and writes Y.
#include "common.cuh"

namespace elutq {

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kTableBytes = 256 * 256;           // 256 entries x 64 columns x 4 bytes
constexpr int kSmemBytes = kTableBytes + 64;     // + up to 16 group sums

template <int Q, int G>
struct Cfg {
    static constexpr int W = G / 8;              // byte-columns per quantisation group
    static constexpr int NSG = 128 / G;          // groups per super-group
    static constexpr int GL = 2 * NSG;           // groups per lane
    static constexpr int NV = 2 * Q;             // 16-byte plane vectors per lane
    static constexpr int NPW = GL * (Q + 1) / 2; // parameter words per lane
    static constexpr int PLANE_BYTES = 1024 * Q;
    static constexpr int TILE_BYTES = PLANE_BYTES + 128 * NPW;
};

template <int Q, int G>
struct Item {
    uint4 v[Cfg<Q, G>::NV];
    uint32_t p[Cfg<Q, G>::NPW];
};

template <int Q, int G>
__device__ __forceinline__ void load_item(Item<Q, G>& it, const uint8_t* tile, int lane, bool planes) {
    using C = Cfg<Q, G>;
    if (planes) {
#pragma unroll
        for (int i = 0; i < C::NV; ++i) it.v[i] = ldg_stream_v4(tile + (i * 32 + lane) * 16);
    }
#pragma unroll
    for (int i = 0; i < C::NPW; ++i) it.p[i] = ldg_stream_u32(tile + C::PLANE_BYTES + (i * 32 + lane) * 4);
}

// Builds the 64 fused tables of chunk kc and the chunk's group sums.  512 threads:
// thread -> column c = tid & 63 and two high nibbles {2*hq, 2*hq+1}, hq = tid >> 6.
template <int G, bool PLAIN>
__device__ __forceinline__ void build_tables(uint8_t* smem, const __half* __restrict__ X, int kc, int K, int tid) {
    constexpr int W = G / 8;
    float* T = reinterpret_cast<float*>(smem);
    float* gsum = reinterpret_cast<float*>(smem + kTableBytes);
    const int c = tid & 63, hq = tid >> 6;
    const int k0 = kc * kChunkK + c * 8;
    float x[8];
    if (k0 < K) {
        const uint4 raw = *reinterpret_cast<const uint4*>(X + k0);
        const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = 0.f;
    }
    float A[16];
    A[0] = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int p = 0; p < (1 << b); ++p) A[p | (1 << b)] = A[p] + x[b];
    float total = 0.f;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int hi = 2 * hq + hh;
        float Bv = 0.f;
#pragma unroll
        for (int b = 0; b < 4; ++b) Bv += ((hi >> b) & 1) ? x[4 + b] : 0.f;
        if (PLAIN) {
            // unfused variant: entry p holds A[lo] in rows with hi == 0 and B[hi] in rows with lo == 0
            // (only those rows are addressed by the plain g = 4 look-ups)
#pragma unroll
            for (int lo = 0; lo < 16; ++lo) T[(hi * 16 + lo) * 64 + c] = (hi == 0) ? A[lo] : (lo == 0 ? Bv : 0.f);
        } else {
#pragma unroll
            for (int lo = 0; lo < 16; ++lo) T[(hi * 16 + lo) * 64 + c] = A[lo] + Bv;
        }
        total = A[15] + Bv;
    }
    if (hq == 7) {  // warps 14 and 15 hold entry 255 = sum of the column's 8 activations
#pragma unroll
        for (int off = W / 2; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
        if ((c % W) == 0) gsum[c / W] = total;
    }
}

template <int Q, int G, bool PLAIN>
__global__ void __launch_bounds__(kThreads, 2) lut_gemv_kernel(const GemmArgs a) {
    using C = Cfg<Q, G>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const float* gsum = reinterpret_cast<const float*>(smem + kTableBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = lane >> 4, l = lane & 15;
    const long long total = (long long)a.n_kc * a.n_rb;   // < 2^31 (checked by the launcher)
    const int first = (int)(total * blockIdx.x / gridDim.x);
    const int last = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const bool use_planes = !(a.flags & ELUTQ_FLAG_OFFSET_ONLY);
    const bool use_offset = !(a.flags & ELUTQ_FLAG_SKIP_OFFSET);

    // byte offset of the lane's column inside a 256-byte table row, per step
    uint32_t col[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) col[i] = 4u * (16 * h + tau_of(l, i, C::W, C::NSG));

    Item<Q, G> cur, nxt;
    int it = first + warp;
    if (it < last) load_item<Q, G>(nxt, a.tiles + (size_t)it * C::TILE_BYTES, lane, use_planes);

    // weights do not depend on the previous kernel in the stream; X, Y and the workspace do
    grid_launch_dependents();
    grid_dependency_wait();

    const int n_pad = a.n_rb * kTileRows;
    int seg = first;
    while (seg < last) {
        const int kc = seg / a.n_rb;
        const int seg_end = min(last, (kc + 1) * a.n_rb);
        __syncthreads();
        build_tables<G, PLAIN>(smem, a.X, kc, a.K, tid);
        __syncthreads();

        float S[C::GL];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int v = 0; v < C::NSG; ++v)
                S[u * C::NSG + v] = use_offset ? gsum[C::NSG * (h + 2 * u) + (l / C::W + v) % C::NSG] : 0.f;

        while (it < seg_end) {
            cur = nxt;
            const int nit = it + kWarps;
            if (nit < last) load_item<Q, G>(nxt, a.tiles + (size_t)nit * C::TILE_BYTES, lane, use_planes);

            float prm[C::GL * (Q + 1)];
#pragma unroll
            for (int i = 0; i < C::NPW; ++i) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&cur.p[i]));
                prm[2 * i] = f.x;
                prm[2 * i + 1] = f.y;
            }
            float y = 0.f;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
#pragma unroll
                for (int v = 0; v < C::NSG; ++v) {
                    const int gidx = u * C::NSG + v;
                    if (use_planes) {
#pragma unroll
                        for (int j = 0; j < Q; ++j) {
                            const uint4 vec = cur.v[u * Q + j];
                            const uint32_t wd[4] = {vec.x, vec.y, vec.z, vec.w};
                            float acc = 0.f;
                            if (!PLAIN) {
#pragma unroll
                                for (int ii = 0; ii < C::W; ++ii) {
                                    const int i = v * C::W + ii;
                                    const uint32_t off = __byte_perm(wd[i >> 2], col[i], 0x5504 + 0x10 * (i & 3));
                                    acc += *reinterpret_cast<const float*>(smem + off + u * 128);
                                }
                            } else {
#pragma unroll
                                for (int ii = 0; ii < C::W; ++ii) {
                                    const int i = v * C::W + ii;
                                    const uint32_t off = __byte_perm(wd[i >> 2], col[i], 0x5504 + 0x10 * (i & 3));
                                    acc += *reinterpret_cast<const float*>(smem + (off & 0x0fffu) + u * 128);   // low nibble table
                                    acc += *reinterpret_cast<const float*>(smem + (off & 0xf0ffu) + u * 128);   // high nibble table
                                }
                            }
                            y = fmaf(prm[gidx * (Q + 1) + j], acc, y);
                        }
                    }
                    y = fmaf(prm[gidx * (Q + 1) + Q], S[gidx], y);
                }
            }
            y += __shfl_xor_sync(0xffffffffu, y, 16);

            const int rb = it - kc * a.n_rb;
            const int row = rb * kTileRows + l;
            bool write_out = (a.n_kc == 1);
            if (!write_out) {
                if (h == 0) a.partials[(size_t)kc * n_pad + row] = y;
                __threadfence();
                __syncwarp();
                unsigned old = 0;
                if (lane == 0) old = atomicInc(a.counters + rb, (unsigned)(a.n_kc - 1));
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == (unsigned)(a.n_kc - 1)) {   // last chunk to arrive: fixed-order sum
                    __threadfence();
                    float sum = 0.f;
                    for (int kk = h; kk < a.n_kc; kk += 2) sum += __ldcg(a.partials + (size_t)kk * n_pad + row);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 16);
                    y = sum;
                    write_out = true;
                }
            }
            if (write_out && h == 0 && row < a.N) {
                if (a.flags & ELUTQ_FLAG_OUT_F32) {
                    float* Yf = reinterpret_cast<float*>(a.Y);
                    Yf[row] = (a.flags & ELUTQ_FLAG_ACCUMULATE) ? Yf[row] + y : y;
                } else {
                    __half* Yh = reinterpret_cast<__half*>(a.Y);
                    if (a.flags & ELUTQ_FLAG_ACCUMULATE) y += __half2float(Yh[row]);
                    Yh[row] = __float2half_rn(y);
                }
            }
            it = nit;
        }
        seg = seg_end;
    }
}

template <int Q, int G, bool PLAIN>
int launch_one(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(lut_gemv_kernel<Q, G, PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return (int)e;
        configured[dev] = true;
    }
    const long long total = (long long)a.n_kc * a.n_rb;
    if (total >= (1LL << 31) - kWarps) return (int)cudaErrorInvalidValue;
    long long grid = (total + kWarps - 1) / kWarps;
    if (grid > num_sms) grid = 2LL * num_sms;
    if (grid > total) grid = total;
    if (grid < 1) grid = 1;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, G, PLAIN>, a);
    count_launch(1);
    return (int)e;
}

template <int Q>
int launch_q(const GemmArgs& a, int G, int num_sms, cudaStream_t stream) {
    switch (G) {
        case 32: return launch_one<Q, 32, false>(a, num_sms, stream);
        case 64: return launch_one<Q, 64, false>(a, num_sms, stream);
        case 128:
            return (a.flags & ELUTQ_FLAG_PLAIN_G4) ? launch_one<Q, 128, true>(a, num_sms, stream)
                                                   : launch_one<Q, 128, false>(a, num_sms, stream);
        default: return (int)cudaErrorInvalidValue;
    }
}

}  // namespace

int launch_lut_gemv(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream) {
    switch (q) {
        case 1: return launch_q<1>(a, G, num_sms, stream);
        case 2: return launch_q<2>(a, G, num_sms, stream);
        case 3: return launch_q<3>(a, G, num_sms, stream);
        case 4: return launch_q<4>(a, G, num_sms, stream);
        default: return (int)cudaErrorInvalidValue;
    }
}

}  // namespace elutq
