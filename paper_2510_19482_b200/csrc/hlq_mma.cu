// Prefill-sized batches (M >= 64): dequantise-and-contract on the 5th-generation tensor cores.
//
// For large M the look-up path is bound by the shared-memory look-up rate (it does M look-ups per
// weight byte), while Y = X W_hat^T is then a genuine dense contraction.  This kernel rebuilds each
// weight tile in fp16 from the packed bit-planes and runs it through tcgen05.mma:
//
//   CTA tile   128 weight rows (UMMA M) x NT tokens (UMMA N = 64, 128 or 256), K walked in steps of 256
//              (half a packed tile: super-groups 2u and 2u+1 of a 512-column chunk)
//   A operand  W_hat tile, 128 x 256 fp16, K-major, no swizzle: core matrices of 8 rows x 16 bytes,
//              [row group][k8] order (leading byte offset 128, stride byte offset 4096).  One warp
//              dequantises one packed item (16 rows): lane (h, l) owns row l and super-group h, and every
//              packed byte (8 consecutive k of one row) becomes exactly one 16-byte core-matrix row.
//   dequant    the BCQ / mirror form of Appendix D: W_hat = z^ + sum_j (-s_j/2) * (+-1), where the +-1.0
//              fp16 operand is built by dropping the weight bit into the sign position of 1.0 - two
//              integer instructions and one HFMA2 per pair of weights and plane.  z^ = z + (1/2) sum s_j
//              is formed in fp32 and rounded once.
//   B operand  X tile, NT x 256 fp16, same canonical layout
//   D          fp32 in tensor memory (128 lanes x NT columns); read back with tcgen05.ld, then either
//              written to Y (one rounding to fp16) or, with a K split, to the fp32 partial buffer that the
//              shared finalize kernel reduces in ascending order.
//
// Every wait is bounded: if the MMA-completion barrier does not flip within the limit the CTA raises the
// status word, skips the remaining work, still releases its tensor memory and returns.
#include "common.cuh"

namespace elutq {

namespace {

constexpr int kMmaThreads = 256;
constexpr int kTileN = 128;                 // weight rows per CTA (UMMA M)
constexpr int kStepK = 256;                 // K per step
constexpr int kABytes = kTileN * kStepK * 2;
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// K-major, no-swizzle shared-memory matrix descriptor: start address, leading (K) and stride (row group)
// byte offsets in 16-byte units, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(128u >> 4) << 16) | ((uint64_t)(4096u >> 4) << 32) |
           ((uint64_t)1 << 46);
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

template <int Q, int NT>
__global__ void __launch_bounds__(kMmaThreads, 1) hlq_mma_kernel(const GemmArgs a, const int splits) {
    constexpr int NPW = 2 * (Q + 1) / 2 + ((2 * (Q + 1)) % 2);      // parameter words per lane at G = 128: Q + 1
    constexpr int PLANE_BYTES = 1024 * Q;
    constexpr int TILE_BYTES = PLANE_BYTES + 128 * (Q + 1);
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sA = smem;
    uint8_t* sB = smem + kABytes;
    uint64_t* mbar = reinterpret_cast<uint64_t*>(smem + kABytes + NT * kStepK * 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mbar + 1);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = lane >> 4, l = lane & 15;
    const int n_tile = blockIdx.x, m_tile = blockIdx.y, split = blockIdx.z;
    const int m0 = m_tile * NT;
    const int n_steps = 2 * a.n_kc;                                   // half chunks
    const int step0 = (int)((long long)n_steps * split / splits);
    const int step1 = (int)((long long)n_steps * (split + 1) / splits);
    const bool use_planes = !(a.flags & ELUTQ_FLAG_OFFSET_ONLY);
    const bool use_offset = !(a.flags & ELUTQ_FLAG_SKIP_OFFSET);

    // ---- set-up: tensor memory, completion barrier --------------------------------------------
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)NT) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(mbar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = *tmem_slot;

    grid_launch_dependents();
    grid_dependency_wait();

    // instruction descriptor: D = fp32, A = B = fp16, both K-major, N = NT, M = 128
    constexpr uint32_t idesc = (1u << 4) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(kTileN >> 4) << 24);
    const uint32_t a_addr = smem_u32(sA), b_addr = smem_u32(sB), bar_addr = smem_u32(mbar);

    const int rb = n_tile * (kTileN / kTileRows) + warp;               // this warp's row block
    const bool rb_valid = rb < a.n_rb;
    // destination of this lane's core-matrix rows: row group 2*warp + l/8, row l%8; column added per byte
    const uint32_t a_row_off = (uint32_t)((2 * warp + (l >> 3)) * 32) * 128u + (uint32_t)(l & 7) * 16u;

    uint32_t phase = 0;
    bool ok = true;
    for (int step = step0; step < step1 && ok; ++step) {
        const int kc = step >> 1, u = step & 1;

        // ---- A: dequantise this warp's item half into the core-matrix layout ----------------------
        if (rb_valid && use_planes | use_offset) {
            const uint8_t* tile = a.tiles + ((size_t)kc * a.n_rb + rb) * TILE_BYTES;
            uint4 vec[Q];
            uint32_t pw[NPW];
            static_for<0, Q>([&](auto j) { vec[j] = ldg_stream_v4<0>(tile + ((u * Q + j) * 32 + lane) * 16); });
            static_for<0, NPW>([&](auto i) { pw[i] = ldg_stream_u32<0>(tile + PLANE_BYTES + (i * 32 + lane) * 4); });
            // record of this half: halves [u*(Q+1) .. u*(Q+1)+Q] = s_0..s_{Q-1}, z
            float sc[Q + 1];
#pragma unroll
            for (int c = 0; c <= Q; ++c) {
                float lo_v = 0.f, hi_v = 0.f;
#pragma unroll
                for (int uu = 0; uu < 2; ++uu) {
                    const int e = uu * (Q + 1) + c;
                    const uint32_t wv = pw[e >> 1];
                    const float f = __half2float(__ushort_as_half((unsigned short)((e & 1) ? (wv >> 16) : (wv & 0xffffu))));
                    if (uu == 0) lo_v = f; else hi_v = f;
                }
                sc[c] = u ? hi_v : lo_v;
            }
            float zhat = use_offset ? sc[Q] : 0.f;
            __half2 sneg[Q];
#pragma unroll
            for (int j = 0; j < Q; ++j) {
                const float sj = use_planes ? sc[j] : 0.f;
                zhat += 0.5f * sj;
                sneg[j] = __float2half2_rn(-0.5f * sj);               // exact halving of an fp16 value
            }
            const __half2 z2 = __float2half2_rn(zhat);
            const uint32_t kSign = 0x80008000u, kOne = 0x3C003C00u;
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                __half2 accA[8], accB[8];        // accA[t] = weights (byte 0, byte 2) at bit t; accB: (byte 1, byte 3)
#pragma unroll
                for (int t = 0; t < 8; ++t) { accA[t] = z2; accB[t] = z2; }
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const uint32_t wv = (wi == 0) ? vec[j].x : (wi == 1) ? vec[j].y : (wi == 2) ? vec[j].z : vec[j].w;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        // bits t and t+16 (bytes 0, 2) / t+8 and t+24 (bytes 1, 3) moved to the fp16 sign positions of 1.0
                        const uint32_t xa = ((wv << (15 - t)) & kSign) | kOne;
                        const uint32_t xb = ((wv << (7 - t)) & kSign) | kOne;
                        accA[t] = __hfma2(sneg[j], *reinterpret_cast<const __half2*>(&xa), accA[t]);
                        accB[t] = __hfma2(sneg[j], *reinterpret_cast<const __half2*>(&xb), accB[t]);
                    }
                }
                // regroup: a core-matrix row = the 8 weights of one byte (t = 0..7)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const __half2* src = (b & 1) ? accB : accA;
                    const uint32_t sel = (b & 2) ? 0x7632u : 0x5410u;          // high or low halves
                    uint4 out;
                    out.x = __byte_perm(*reinterpret_cast<const uint32_t*>(&src[0]), *reinterpret_cast<const uint32_t*>(&src[1]), sel);
                    out.y = __byte_perm(*reinterpret_cast<const uint32_t*>(&src[2]), *reinterpret_cast<const uint32_t*>(&src[3]), sel);
                    out.z = __byte_perm(*reinterpret_cast<const uint32_t*>(&src[4]), *reinterpret_cast<const uint32_t*>(&src[5]), sel);
                    out.w = __byte_perm(*reinterpret_cast<const uint32_t*>(&src[6]), *reinterpret_cast<const uint32_t*>(&src[7]), sel);
                    const int ii = 4 * wi + b;                                  // step -> byte column (G = 128 rotation)
                    const int cc = 16 * h + ((l + ii) & 15);
                    *reinterpret_cast<uint4*>(sA + a_row_off + (uint32_t)cc * 128u) = out;
                }
            }
        } else {
            // rows beyond N (or nothing to contribute): zero rows
#pragma unroll
            for (int ii = 0; ii < 16; ++ii)
                *reinterpret_cast<uint4*>(sA + a_row_off + (uint32_t)(16 * h + ((l + ii) & 15)) * 128u) = make_uint4(0, 0, 0, 0);
        }

        // ---- B: activation tile, tokens m0 .. m0+NT-1, columns step*256 .. +255 -----------------------
        {
            const int k_base = step * kStepK;
#pragma unroll 4
            for (int idx = tid; idx < NT * 32; idx += kMmaThreads) {
                const int tok = idx >> 5, c = idx & 31;
                const int m = m0 + tok, k = k_base + c * 8;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (m < a.M && k < a.K) v = *reinterpret_cast<const uint4*>(a.X + (size_t)m * a.K + k);
                *reinterpret_cast<uint4*>(sB + (uint32_t)((tok >> 3) * 32 + c) * 128u + (uint32_t)(tok & 7) * 16u) = v;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> visible to the tensor core
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();

        // ---- MMA: 16 K = 16 slices, issued by one thread; completion arrives on the barrier -------------
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int kk = 0; kk < kStepK / 16; ++kk) {
                const uint64_t da = make_desc(a_addr + kk * 256), db = make_desc(b_addr + kk * 256);
                const uint32_t accumulate = (step != step0 || kk != 0) ? 1u : 0u;
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                             :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         :: "r"(bar_addr) : "memory");
        }
        // everybody waits for the tensor core to finish reading the tiles before they are overwritten
        ok = mbar_wait(bar_addr, phase);
        phase ^= 1u;
    }
    if (!ok && a.counters != nullptr && lane == 0) atomicExch(a.counters, 0x7C05u);   // status word: wait ran out

    // ---- epilogue: TMEM -> registers -> Y or partials ---------------------------------------------
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok && step1 > step0) {
        const int lane_grp = warp & 3, col_half = warp >> 2;            // TMEM lanes 32*lane_grp.., half of the columns
        const int n = n_tile * kTileN + lane_grp * 32 + lane;
        const size_t n_pad = (size_t)a.n_rb * kTileRows;
#pragma unroll 1
        for (int c0 = col_half * (NT / 2); c0 < (col_half + 1) * (NT / 2); c0 += 32) {
            uint32_t r[32];
            const uint32_t taddr = tmem_d + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)c0;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                         "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                         "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                           "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                           "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                           "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (n < a.N) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int m = m0 + c0 + i;
                    if (m < a.M) {
                        const float v = __uint_as_float(r[i]);
                        if (splits == 1) store_out(a, (size_t)m * a.N + n, v);
                        else a.partials[((size_t)split * a.M + m) * n_pad + n] = v;
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"((uint32_t)NT) : "memory");
}

template <int Q, int NT>
int launch_mma_nt(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    constexpr int kSmem = kABytes + NT * kStepK * 2 + 64;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(hlq_mma_kernel<Q, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return (int)e;
        configured[dev] = true;
    }
    const int n_tiles = (a.N + kTileN - 1) / kTileN, m_tiles = (a.M + NT - 1) / NT;
    // K split only while the tile count leaves SMs idle (partials cost M*N*4 bytes per split)
    int splits = 1;
    const int n_steps = 2 * a.n_kc;
    while (splits * 2 <= n_steps && (long long)n_tiles * m_tiles * splits * 2 <= 2LL * num_sms && splits < 16) splits *= 2;
    if (debug_env("ELUTQ_DEBUG_MMA_SPLITS") > 0) splits = debug_env("ELUTQ_DEBUG_MMA_SPLITS");
    if (splits > n_steps) splits = n_steps;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_tiles, (unsigned)m_tiles, (unsigned)splits);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = debug_env("ELUTQ_DEBUG_NO_PDL") > 0 ? 0 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, hlq_mma_kernel<Q, NT>, a, splits);
    count_launch(1);
    if (e != cudaSuccess || splits == 1) return (int)e;
    return launch_finalize(a, splits, cfg.numAttrs != 0, stream);
}

template <int Q>
int launch_mma_q(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    if (a.M <= 64) return launch_mma_nt<Q, 64>(a, num_sms, stream);
    if (a.M <= 128) return launch_mma_nt<Q, 128>(a, num_sms, stream);
    return launch_mma_nt<Q, 256>(a, num_sms, stream);
}

}  // namespace

// Largest K split the tensor-core path may pick for (M, N, K): sizes the partial buffer.
int mma_max_splits() { return 16; }

int launch_hlq_mma(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream) {
    if (G != 128) return (int)cudaErrorNotSupported;
    switch (q) {
        case 1: return launch_mma_q<1>(a, num_sms, stream);
        case 2: return launch_mma_q<2>(a, num_sms, stream);
        case 3: return launch_mma_q<3>(a, num_sms, stream);
        case 4: return launch_mma_q<4>(a, num_sms, stream);
        default: return (int)cudaErrorInvalidValue;
    }
}

}  // namespace elutq
