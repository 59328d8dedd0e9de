// Batches of ELUTQ_TENSOR_MIN_M rows or more at G = 128: dequantise-and-contract on the 5th-generation tensor cores.
//
// For large M the look-up path is bound by the shared-memory look-up rate (it does M look-ups per
// weight byte), while Y = X W_hat^T is then a genuine dense contraction.  This kernel rebuilds each
// weight tile in fp16 from the packed bit-planes and runs it through tcgen05.mma:
//
//   CTA tile   TT x 128 tokens (UMMA M = 128, TT = 1 or 2 accumulators) x NW weight rows (UMMA N = 128
//              or 256), K walked in steps of 128 (one super-group of a 512-column chunk).  Weight rows are
//              the wide dimension on purpose: a packed weight is 8x smaller than an fp16 activation, so the
//              activation tile is what the L2 has to feed again and again; two token tiles share one
//              dequantised weight tile, which halves both the dequantisation work and the weight traffic.
//   A operand  X tile, 128 tokens x 128 k fp16, K-major with the 128-byte swizzle: two blocks of 64 k, a
//              token row is 128 contiguous bytes whose 16-byte chunks are XOR-ed with (token mod 8).  A
//              quarter-warp copies the 8 chunks of one token: four full 32-byte sectors on the global side,
//              eight different bank groups on the shared side.  Two stages, filled by cp.async one step
//              ahead of the MMAs that read them.
//   B operand  W_hat tile, NW x 128 fp16, kept as two halves of 64 k, each K-major without swizzle: core
//              matrices of 8 rows x 16 bytes in [row group][k8] order (leading byte offset 128, stride byte
//              offset 1024).  A warp dequantises two packed items (32 rows): lane 16*i + l owns row l of
//              item i and the step's super-group, and every packed byte (8 consecutive k of one row)
//              becomes exactly one 16-byte core-matrix row.  Each half has its own completion barrier, so
//              the tensor core reads one half while the threads rebuild the other.
//   dequant    the BCQ / mirror form of Appendix D: W_hat = z^ + sum_j (+-)(-s_j/2), in registers.  For a plane
//              byte (8 weights) and each of its 4 weight pairs: one integer multiply moves the pair's two bits
//              to the fp16 sign positions, one logic operation flips the signs of the packed -s_j/2, one
//              packed fp16 add accumulates (measured 8-30 % faster than a shared-memory table of +-1.0 factors,
//              which competes with the tensor core for shared-memory bandwidth).  z^ = z + (1/2) sum s_j is
//              formed in fp32 and rounded once.
//   D          fp32 in tensor memory (lane = token, column = weight row, one block of NW columns per token
//              tile); read back with tcgen05.ld, then either written to Y (one rounding to fp16, 16-byte
//              stores) or, with a K split, to the fp32 partial buffer that the shared finalize kernel
//              reduces in ascending order.
//
//   schedules  M <= 128: one token tile, whole weight tile double-buffered, one CTA barrier per step.  M > 128: two token
//              tiles per CTA and a ninth warp that issues the MMAs; the eight producer warps hand each dequantised
//              half over through an mbarrier (one arrival per warp), no CTA-wide barrier in the step.  With an even
//              number of 256-token tiles the CTAs run as pairs (cluster of two, `cta_group::2`, UMMA M = 256): both
//              CTAs of a pair work on the same weight tile with their own tokens, each dequantises half of its rows,
//              and the half steps run through rings of four slots (see the kernel).
//
// Every wait is bounded: a thread whose MMA-completion barrier does not flip within the limit raises the
// status word and stops waiting; it still joins every CTA barrier, and the CTA releases its tensor memory.
#include "common.cuh"

namespace elutq {

namespace {

constexpr int kMmaThreads = 256;               // measured: 512 threads (two warps per item pair) are 4-8 % slower
constexpr int kTileM = 128;                  // tokens per accumulator (UMMA M)
constexpr int kStepK = 128;                  // K per step
constexpr int kXTileBytes = kTileM * kStepK * 2;   // one token tile of one step: 2 blocks of [128 tokens][128 bytes]
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptors (version 1).  Addresses and offsets are in 16-byte units.
// K-major, no swizzle: leading (K direction) offset 128 bytes, stride (row group) offset 1024 bytes.
__device__ __forceinline__ uint64_t desc_noswizzle(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(128u >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) |
           ((uint64_t)1 << 46);
}
// K-major, 128-byte swizzle: rows of 128 bytes, row groups of 1024 bytes; the leading offset is not used.
__device__ __forceinline__ uint64_t desc_swizzle128(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024u >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

// 32 consecutive outputs of one token row: Y (fp16 or fp32, optionally accumulating) or the fp32 partials.
__device__ __forceinline__ void store_row32(const GemmArgs& a, int m, int n0, const uint32_t (&r)[32], int splits,
                                            int split, size_t n_pad, bool y_vec_ok) {
    if (splits > 1) {
        float* dst = a.partials + ((size_t)split * a.M + m) * n_pad + n0;
#pragma unroll
        for (int i = 0; i < 32; i += 4)
            if ((size_t)(n0 + i) < n_pad)
                *reinterpret_cast<uint4*>(dst + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
        return;
    }
    if (y_vec_ok) {                        // fp16 output, no accumulation, N a multiple of 8, Y 16-byte aligned
        __half* dst = reinterpret_cast<__half*>(a.Y) + (size_t)m * a.N + n0;
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
            if (n0 + i < a.N) {
                uint32_t p[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const __half2 v = __floats2half2_rn(__uint_as_float(r[i + 2 * t]), __uint_as_float(r[i + 2 * t + 1]));
                    p[t] = *reinterpret_cast<const uint32_t*>(&v);
                }
                *reinterpret_cast<uint4*>(dst + i) = make_uint4(p[0], p[1], p[2], p[3]);
            }
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (n0 + i < a.N) store_out(a, (size_t)m * a.N + n0 + i, __uint_as_float(r[i]));
}

// NW = weight rows per CTA (UMMA N: 128 or 256); TT = token tiles of 128 per CTA (1 or 2).
// WS (TT = 2 only) = warp-specialised form: a ninth warp issues the MMAs, the eight producer warps hand each finished
// half over through an mbarrier (one arrival per warp) instead of a CTA-wide barrier.
//
// CG = 2 (with WS): a pair of CTAs (thread-block cluster of two along the token dimension, one SM pair) works on one
// weight tile with `tcgen05.mma.cta_group::2`, UMMA M = 256: each CTA holds its own 2 x 128 tokens (A operand rows and
// accumulator lanes) and dequantises only its half of the tile's weight rows (the tensor core reads the two halves of
// B from the two CTAs' shared memory), so the dequantisation per MMA is halved.  The issuer warp of the leader CTA
// (cluster rank 0) waits for the arrivals of all 16 producer warps (the peer's arrive through the cluster window) and
// commits each half's MMAs to the "done" barriers of both CTAs.
template <int Q, int NW, int TT, bool WS = false, int CG = 1>
__global__ void __launch_bounds__(kMmaThreads + (WS ? 32 : 0), 1) hlq_mma_kernel(const GemmArgs a, const int splits, const int n_tile0) {
    static_assert(!WS || TT == 2, "the warp-specialised form exists for two token tiles only");
    static_assert(CG == 1 || (WS && CG == 2), "the CTA-pair form builds on the warp-specialised one");
    constexpr int NWL = NW / CG;                         // weight rows dequantised by this CTA
    constexpr int NPW = Q + 1;                           // parameter words per lane at G = 128
    constexpr int PLANE_BYTES = 1024 * Q;
    constexpr int TILE_BYTES = PLANE_BYTES + 128 * (Q + 1);
    constexpr int PAIRS = NWL / 32;                      // item pairs per step: 8 or 4
    constexpr int WPP = (kMmaThreads / 32) / PAIRS;      // warps sharing one item pair: 1 or 2
    constexpr int NB = 8 / WPP;                          // plane bytes per lane and half step
    constexpr int W_HALF_BYTES = NWL * 64 * 2;           // one half (64 k) of this CTA's part of the weight tile
    constexpr int X_STAGE_BYTES = TT * kXTileBytes;
    constexpr int W_BYTES = NWL * kStepK * 2;
    constexpr int XS = (TT == 1) ? 3 : 2;                // activation stages
    constexpr int WB = (TT == 1 || CG == 2) ? 2 : 1;     // whole weight tiles (each of two halves); the pair form uses them as a ring of four halves
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sX = smem;                                  // A operand stages
    uint8_t* sW = smem + XS * X_STAGE_BYTES;             // B operand
    uint64_t* mbar = reinterpret_cast<uint64_t*>(sW + WB * W_BYTES);        // [2]: one per weight-tile half (TT = 2)
                                                                            //      or per weight tile (TT = 1)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mbar + 8);            // WS: mbar[2], mbar[3] = "half is ready"; pair form: [0..3] done, [4..7] ready

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int l = lane & 15;
    // CTA pairs are neighbours in x, so the pair form puts the token tiles there
    const int n_tile = n_tile0 + (CG == 2 ? blockIdx.y : blockIdx.x), m_tile = (CG == 2 ? blockIdx.x : blockIdx.y), split = blockIdx.z;
    const int m0 = m_tile * (TT * kTileM);
    const int n_steps = 4 * a.n_kc;                                   // super-groups
    const int step0 = (int)((long long)n_steps * split / splits);
    const int step1 = (int)((long long)n_steps * (split + 1) / splits);
    const bool use_planes = !(a.flags & ELUTQ_FLAG_OFFSET_ONLY);
    const bool use_offset = !(a.flags & ELUTQ_FLAG_SKIP_OFFSET);

    // the blob is still the one this launch was planned for (checked before anything is allocated or read)
    if (!blob_header_matches(a.tiles, Q, 128, a.N, a.K, a.counters)) return;

    // ---- set-up: tensor memory, completion barriers ---------------------------------------------
    uint32_t cta_rank = 0;                               // rank in the CTA pair (0 = leader)
    if constexpr (CG == 2) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(cta_rank));
    if (warp == 0) {
        if constexpr (CG == 2) {     // the same warp of both CTAs of the pair allocates (same columns in both)
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)(TT * NW)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)(TT * NW)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(mbar)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(mbar + 1)) : "memory");
        if constexpr (CG == 2) {
#pragma unroll
            for (int i = 2; i < 4; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(mbar + i)) : "memory");
#pragma unroll
            for (int i = 4; i < 8; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 16;" :: "r"(smem_u32(mbar + i)) : "memory");
        } else {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" :: "r"(smem_u32(mbar + 2)) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" :: "r"(smem_u32(mbar + 3)) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if constexpr (CG == 2) cluster_barrier();            // the peer's barriers are initialised before anyone arrives on them
    else __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = *tmem_slot;

    // instruction descriptor: D = fp32, A = B = fp16, both K-major, M = 128 tokens, N = NW weight rows
    constexpr uint32_t idesc = (1u << 4) | ((uint32_t)(NW >> 3) << 17) | ((uint32_t)((CG * kTileM) >> 4) << 24);
    const uint32_t x_addr = smem_u32(sX), w_addr = smem_u32(sW), bar_addr = smem_u32(mbar);

    // Asynchronous copy of the activation tile(s) of one step into a stage.  Thread (token r = tid / 8 + RPP p,
    // chunk j = tid % 8): 16 bytes at k = step*128 + kb*64 + 8 j, stored at chunk j ^ (r & 7) of row r.  Rows
    // beyond M and columns beyond K are zero-filled by a copy of source size 0 (its address is clamped to a
    // valid row, nothing is read), so the loop carries no branches.
    constexpr int RPP = kMmaThreads / 8;            // token rows per pass
    constexpr int NPASS = kTileM / RPP;
    const __half* x_src[TT * NPASS];
    uint32_t x_live = 0;                            // bit (tt * NPASS + p): the row exists
    {
        const int j = tid & 7, r0 = tid >> 3;
#pragma unroll
        for (int tt = 0; tt < TT; ++tt)
#pragma unroll
            for (int p = 0; p < NPASS; ++p) {
                const int m = m0 + tt * kTileM + p * RPP + r0;
                x_src[tt * NPASS + p] = a.X + (size_t)(m < a.M ? m : a.M - 1) * a.K + j * 8;
                if (m < a.M) x_live |= 1u << (tt * NPASS + p);
            }
    }
    auto copy_x = [&](int step, int stage) {
        const int j = tid & 7, r0 = tid >> 3;
        const uint32_t dst0 = x_addr + (uint32_t)stage * X_STAGE_BYTES + (uint32_t)r0 * 128u + (uint32_t)((j ^ (r0 & 7)) * 16);
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
            const int k = step * kStepK + kb * 64;                     // k + 8 j < K for every j or for none (K % 64 == 0)
            const uint32_t live = (k < a.K) ? x_live : 0u;
            const int koff = (k < a.K) ? k : 0;
#pragma unroll
            for (int tt = 0; tt < TT; ++tt) {
#pragma unroll
                for (int p = 0; p < NPASS; ++p) {                       // (r0 + RPP p) & 7 == r0 & 7
                    const uint32_t dst = dst0 + (uint32_t)(tt * kXTileBytes + kb * (kTileM * 128) + p * RPP * 128);
                    const uint32_t nbytes = ((live >> (tt * NPASS + p)) & 1u) ? 16u : 0u;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                                 :: "r"(dst), "l"(x_src[tt * NPASS + p] + koff), "r"(nbytes) : "memory");
                }
            }
        }
    };

    // Weights of the current step live in registers; the next step's are requested while this one is dequantised.
    // Lane 16 i + l reads what packed lane (h, l) of item i owns: plane vectors of half u, parameter words.
    const int pair = warp % PAIRS;                        // item pair of this warp
    const int bsel = warp / PAIRS;                        // which NB bytes of the 16 (only when two warps share a pair)
    const int item = 2 * pair + (lane >> 4);
    const int rb = n_tile * (NW / kTileRows) + (int)cta_rank * (NWL / kTileRows) + item;
    uint4 vec[Q];
    uint32_t pw[NPW];
    auto load_weights = [&](int step) {
        const int kc = step >> 2, sg = step & 3, h = sg & 1, u = sg >> 1;
        if (rb < a.n_rb) {
            const uint8_t* tile = a.tiles + ((size_t)kc * a.n_rb + rb) * TILE_BYTES;
            const int pl = 16 * h + l;
            static_for<0, Q>([&](auto j) { vec[j] = ldg_stream_v4<0>(tile + ((u * Q + j) * 32 + pl) * 16); });
            static_for<0, NPW>([&](auto i) { pw[i] = ldg_stream_u32<0>(tile + PLANE_BYTES + (i * 32 + pl) * 4); });
        }
    };

    // The packed weights do not depend on the previous kernel in the stream (X, Y and the partial buffer do):
    // the first step's vectors are requested before the dependency wait.
    if (step0 < step1 && warp < kMmaThreads / 32) load_weights(step0);
    grid_launch_dependents();
    grid_dependency_wait();

    // The packed layout rotates a lane's 16 plane bytes (byte i covers 16-byte column (l + i) mod 16 of the
    // super-group, which keeps the look-up kernels free of bank conflicts).  Here the halves of the weight tile
    // are fixed k ranges, so each vector is rotated left by l bytes once per step: byte c then covers column c.
    auto unrotate = [&]() {
        const int ws = l >> 2, sh = (l & 3) * 8;
#pragma unroll
        for (int j = 0; j < Q; ++j) {
            const uint32_t v0 = vec[j].x, v1 = vec[j].y, v2 = vec[j].z, v3 = vec[j].w;
            const uint32_t a0 = (ws & 1) ? v3 : v0, a1 = (ws & 1) ? v0 : v1, a2 = (ws & 1) ? v1 : v2, a3 = (ws & 1) ? v2 : v3;
            const uint32_t t0 = (ws & 2) ? a2 : a0, t1 = (ws & 2) ? a3 : a1, t2 = (ws & 2) ? a0 : a2, t3 = (ws & 2) ? a1 : a3;
            vec[j].x = __funnelshift_l(t3, t0, sh);
            vec[j].y = __funnelshift_l(t0, t1, sh);
            vec[j].z = __funnelshift_l(t1, t2, sh);
            vec[j].w = __funnelshift_l(t2, t3, sh);
        }
    };

    // One thread's view of a completion barrier: every thread polls for itself; a thread whose wait runs out
    // raises the status word once and stops waiting, but keeps taking part in every CTA-wide barrier.
    bool ok = true;
    const uint32_t wait_limit = a.wait_limit ? a.wait_limit : kWaitLimit;
    auto wait_mma = [&](int which, uint32_t parity) {
        if (!ok) return;
        if (!mbar_wait(bar_addr + 8u * which, parity, wait_limit)) {
            ok = false;
            if (a.counters != nullptr) atomicExch(a.counters, 0x7C05u);
        }
    };

    // The issuer's wait for the producers' arrivals; in a CTA pair the peer's arrivals (and what they release) come
    // through the cluster, so the wait acquires at cluster scope.
    auto wait_ready = [&](int which, uint32_t parity) {
        if (!ok) return;
        bool done = false;
        if constexpr (CG == 2) {
            for (uint32_t i = 0; i < wait_limit && !done; ++i) {
                uint32_t r;
                asm volatile("{\n\t.reg .pred p;\n\t"
                             "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                             "selp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(r) : "r"(bar_addr + 8u * which), "r"(parity) : "memory");
                done = r != 0;
            }
        } else {
            done = mbar_wait(bar_addr + 8u * which, parity, wait_limit);
        }
        if (!done) {
            ok = false;
            if (a.counters != nullptr) atomicExch(a.counters, 0x7C05u);
        }
    };

    // Parameters of the step's super-group for this lane's row, decoded once per step: halves
    // [u*(Q+1) .. u*(Q+1)+Q] of the parameter words = s_0..s_{Q-1}, z.
    uint32_t sneg[Q];                                              // (-s_j/2, -s_j/2) as packed fp16
    __half2 z2;                                                    // (z^, z^)
    auto decode_params = [&](int step) {
        const int u = (step & 3) >> 1;
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
#pragma unroll
        for (int j = 0; j < Q; ++j) {
            const float sj = use_planes ? sc[j] : 0.f;
            zhat += 0.5f * sj;
            const __half2 h2 = __float2half2_rn(-0.5f * sj);           // exact halving of an fp16 value
            sneg[j] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        z2 = __float2half2_rn(zhat);
    };

    // Dequantise half hb (64 k) of this lane's row into half hb of weight tile wt (BCQ form, in registers).
    auto dequant_half_to = [&](int hb, uint8_t* buf) {
        const uint32_t row_off = (uint32_t)((2 * item + (l >> 3)) * 8) * 128u + (uint32_t)(l & 7) * 16u;
        if (rb < a.n_rb && (use_planes | use_offset)) {
#pragma unroll
            for (int bi = 0; bi < NB; ++bi) {
                __half2 acc[4] = {z2, z2, z2, z2};
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const uint32_t w0 = hb ? vec[j].z : vec[j].x, w1 = hb ? vec[j].w : vec[j].y;
                    const int gb = bsel * NB + bi;                              // byte of the half: 0..7
                    const uint32_t byte = (((gb & 4) ? w1 : w0) >> (8 * (gb & 3))) & 0xffu;
                    // +-s_j/2 for the byte's 8 weights: one multiply moves bits 2p and 2p+1 to the fp16 sign
                    // positions 15 and 31 (the two shifted copies of an 8-bit value do not overlap), one logic
                    // operation flips the signs of the packed -s_j/2, one packed add accumulates
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const uint32_t t = byte * ((1u << (15 - 2 * p)) + (1u << (30 - 2 * p)));
                        const uint32_t term = (t & 0x80008000u) ^ sneg[j];
                        acc[p] = __hadd2(acc[p], *reinterpret_cast<const __half2*>(&term));
                    }
                }
                const int cc = bsel * NB + bi;                          // 16-byte column inside the half (0..7)
                *reinterpret_cast<uint4*>(buf + row_off + (uint32_t)cc * 128u) =
                    make_uint4(*reinterpret_cast<const uint32_t*>(&acc[0]), *reinterpret_cast<const uint32_t*>(&acc[1]),
                               *reinterpret_cast<const uint32_t*>(&acc[2]), *reinterpret_cast<const uint32_t*>(&acc[3]));
            }
        } else {
            // rows beyond N (or nothing to contribute): zero rows
#pragma unroll
            for (int bi = 0; bi < NB; ++bi)
                *reinterpret_cast<uint4*>(buf + row_off + (uint32_t)(bsel * NB + bi) * 128u) = make_uint4(0, 0, 0, 0);
        }
    };

    auto dequant_half = [&](int hb, int wt) { dequant_half_to(hb, sW + wt * W_BYTES + hb * W_HALF_BYTES); };

    // MMAs of one half step (64 k = 4 slices per token tile), issued by one thread; completion arrives on barrier hb.
    // (Single-CTA schedules; the pair form issues its own in the ring loop below.)
    auto issue_mma = [&](int step, int stage, int hb) {
        if (tid != (WS ? kMmaThreads : 0)) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const uint64_t da = desc_swizzle128(x_addr + stage * X_STAGE_BYTES + tt * kXTileBytes + hb * (kTileM * 128) + kk * 32);
                const uint64_t db = desc_noswizzle(w_addr + hb * W_HALF_BYTES + kk * 256);
                const uint32_t accumulate = (step != step0 || hb != 0 || kk != 0) ? 1u : 0u;
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                             :: "r"(tmem_d + (uint32_t)(tt * NW)), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u)
                             : "memory");
            }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                     :: "r"(bar_addr + 8u * hb) : "memory");
    };
    auto publish = [&]() {     // generic-proxy writes of this thread -> visible to the tensor core, then CTA barrier
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    };

    if constexpr (TT == 1) {
        // One token tile: the MMAs of a step are short next to its dequantisation, so the whole weight tile is
        // double-buffered and a step has a single CTA barrier: dequantise tile s into buffer s % 2 (last read by the
        // MMAs of step s - 2, long finished), publish, issue the MMAs of step s, go on with step s + 1.  Three
        // activation stages, so the copy for step s + 1 never waits for the MMAs of step s - 1 either.
        auto issue_step = [&](int step, int stage, int wt) {
            if (tid != 0) return;
            if (a.flags & kFlagTestNoMma) return;      // test only: nothing is issued, nothing completes, the waits run out
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int kk = 0; kk < kStepK / 16; ++kk) {
                const uint64_t da = desc_swizzle128(x_addr + stage * X_STAGE_BYTES + (kk >> 2) * (kTileM * 128) + (kk & 3) * 32);
                const uint64_t db = desc_noswizzle(w_addr + wt * W_BYTES + (kk >> 2) * W_HALF_BYTES + (kk & 3) * 256);
                const uint32_t accumulate = (step != step0 || kk != 0) ? 1u : 0u;
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                             :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         :: "r"(bar_addr + 8u * wt) : "memory");
        };
        if (step0 < step1) copy_x(step0, 0);
        asm volatile("cp.async.commit_group;" ::: "memory");
        for (int step = step0; step < step1; ++step) {
            const int i = step - step0, wt = i & 1;
            if (i >= 2) wait_mma(wt, (uint32_t)(((i >> 1) - 1) & 1));      // MMAs of step s - 2: buffer and stage are free
            if (step + 1 < step1) copy_x(step + 1, (i + 1) % 3);
            asm volatile("cp.async.commit_group;" ::: "memory");
            unrotate();
            decode_params(step);
            dequant_half(0, wt);
            dequant_half(1, wt);
            if (step + 1 < step1) load_weights(step + 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");          // this step's activation tile has landed
            publish();
            issue_step(step, i % 3, wt);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        const int n = step1 - step0;                                       // the last one or two steps' MMAs
        if (n >= 2) wait_mma((n - 2) & 1, (uint32_t)((((n - 2) >> 1)) & 1));
        if (n >= 1) wait_mma((n - 1) & 1, (uint32_t)((((n - 1) >> 1)) & 1));
    } else if constexpr (WS) {
        // Producer warps: dequantise a half, make it (and the activation stage) visible to the tensor core, arrive on the
        // half's "ready" barrier; before overwriting a half they wait for the MMAs that read it (the "done" barriers).
        // Issuer warp: wait for "ready", issue the half's MMAs, commit them to "done".
        auto arrive_ready = [&](int bar) {
            if constexpr (CG == 2) {
                // Each lane makes its own shared-memory writes visible to the tensor core, the warp converges, lane 0
                // arrives (release) on the leader's barrier.  The data stay in this CTA's shared memory, where the
                // tensor core reads them; only the arrival crosses to the peer.  (A cluster-scope release here was
                // measured 30 % slower for the whole kernel.)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {     // the leader's barrier, through the cluster window
                    uint32_t remote;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(bar_addr + 8u * bar), "r"(0u));
                    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" :: "r"(remote) : "memory");
                }
            } else {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0)
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar_addr + 8u * bar) : "memory");
            }
        };
        if constexpr (CG == 2) {
            // CTA pair: half steps i = 0, 1, ... run through rings of four slots (activation half tiles of 2 x 128
            // tokens x 64 k, and this CTA's 128 weight rows x 64 k); slot i mod 4 has a "ready" barrier (16 producer warps
            // of the pair, on the leader) and a "done" barrier (the half's MMAs, committed to both CTAs).  The producers run
            // up to two halves ahead of the MMAs' completion, which hides the hand-over latency through the cluster.
            constexpr int XH_BYTES = TT * kTileM * 128;          // activation slot
            constexpr int WH_BYTES = W_HALF_BYTES;               // weight slot
            const int n_half = 2 * (step1 - step0);
            auto copy_x_half = [&](int step, int kb, int slot) {
                const int j = tid & 7, r0 = tid >> 3;
                const uint32_t dst0 = x_addr + (uint32_t)slot * XH_BYTES + (uint32_t)r0 * 128u + (uint32_t)((j ^ (r0 & 7)) * 16);
                const int k = step * kStepK + kb * 64;
                const uint32_t live = (k < a.K) ? x_live : 0u;
                const int koff = (k < a.K) ? k : 0;
#pragma unroll
                for (int tt = 0; tt < TT; ++tt) {
#pragma unroll
                    for (int p = 0; p < NPASS; ++p) {
                        const uint32_t dst = dst0 + (uint32_t)(tt * (kTileM * 128) + p * RPP * 128);
                        const uint32_t nbytes = ((live >> (tt * NPASS + p)) & 1u) ? 16u : 0u;
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                                     :: "r"(dst), "l"(x_src[tt * NPASS + p] + koff), "r"(nbytes) : "memory");
                    }
                }
            };
            if (warp < kMmaThreads / 32) {
                if (n_half > 0) copy_x_half(step0, 0, 0);
                asm volatile("cp.async.commit_group;" ::: "memory");
                if (n_half > 1) copy_x_half(step0, 1, 1);
                asm volatile("cp.async.commit_group;" ::: "memory");
                // one half step; hb is a compile-time constant so that the plane words are picked statically
                auto half_iter = [&](int i, auto hb_c) {
                    constexpr int hb = decltype(hb_c)::value;
                    const int step = step0 + (i >> 1), slot = i & 3;
                    if (hb == 0) {
                        unrotate();
                        decode_params(step);
                    }
                    // the slot's previous half (i - 4) was waited for two iterations ago
                    dequant_half_to(hb, sW + slot * WH_BYTES);
                    if (hb == 1 && step + 1 < step1) load_weights(step + 1);
                    asm volatile("cp.async.wait_group 1;" ::: "memory");          // the activations of half i have landed
                    arrive_ready(4 + slot);
                    if (i >= 2) wait_mma((i - 2) & 3, (uint32_t)(((i - 2) >> 2) & 1));    // slot of half i + 2 is free
                    if (i + 2 < n_half) copy_x_half(step0 + ((i + 2) >> 1), hb, (i + 2) & 3);
                    asm volatile("cp.async.commit_group;" ::: "memory");
                };
                for (int i = 0; i < n_half; i += 2) {
                    half_iter(i, IntC<0>{});
                    half_iter(i + 1, IntC<1>{});
                }
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                if (n_half > 0) wait_mma((n_half - 1) & 3, (uint32_t)(((n_half - 1) >> 2) & 1));   // commits complete in order
            } else if (cta_rank == 0 && lane == 0) {
                for (int i = 0; i < n_half; ++i) {
                    const int slot = i & 3;
                    wait_ready(4 + slot, (uint32_t)((i >> 2) & 1));
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                    for (int tt = 0; tt < TT; ++tt) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            const uint64_t da = desc_swizzle128(x_addr + slot * XH_BYTES + tt * (kTileM * 128) + kk * 32);
                            const uint64_t db = desc_noswizzle(w_addr + slot * WH_BYTES + kk * 256);
                            const uint32_t accumulate = (i != 0 || kk != 0) ? 1u : 0u;
                            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                         "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
                                         :: "r"(tmem_d + (uint32_t)(tt * NW)), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u)
                                         : "memory");
                        }
                    }
                    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                                 :: "r"(bar_addr + 8u * slot), "h"((unsigned short)3) : "memory");
                }
            }
        } else {
            uint32_t phase = 0;                                   // every barrier completes once per step
            if (warp < kMmaThreads / 32) {
                if (step0 < step1) copy_x(step0, 0);
                asm volatile("cp.async.commit_group;" ::: "memory");
                for (int step = step0; step < step1; ++step) {
                    const int stage = (step - step0) & 1;
                    if (step > step0) wait_mma(0, phase ^ 1u);
                    unrotate();
                    decode_params(step);
                    dequant_half(0, 0);
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    arrive_ready(2);
                    if (step > step0) wait_mma(1, phase ^ 1u);
                    if (step + 1 < step1) copy_x(step + 1, stage ^ 1);
                    asm volatile("cp.async.commit_group;" ::: "memory");
                    dequant_half(1, 0);
                    if (step + 1 < step1) load_weights(step + 1);
                    arrive_ready(3);
                    phase ^= 1u;
                }
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                if (step1 > step0) {
                    wait_mma(0, phase ^ 1u);
                    wait_mma(1, phase ^ 1u);
                }
            } else {
                for (int step = step0; step < step1; ++step) {
                    const int stage = (step - step0) & 1;
                    wait_ready(2, phase);
                    issue_mma(step, stage, 0);
                    wait_ready(3, phase);
                    issue_mma(step, stage, 1);
                    phase ^= 1u;
                }
            }
        }
    } else {
        if (step0 < step1) copy_x(step0, 0);
        asm volatile("cp.async.commit_group;" ::: "memory");

        // Steady state: the tensor core works on one half of the weight tile while the threads dequantise the other.
        uint32_t phase = 0;                                   // both barriers complete once per step
        for (int step = step0; step < step1; ++step) {
            const int stage = (step - step0) & 1;
            if (step > step0) wait_mma(0, phase ^ 1u);        // half 0 of the previous step has been read
            unrotate();
            decode_params(step);
            dequant_half(0, 0);
            asm volatile("cp.async.wait_group 0;" ::: "memory");          // this step's activation tile has landed
            publish();
            issue_mma(step, stage, 0);

            if (step > step0) wait_mma(1, phase ^ 1u);        // half 1 and the other activation stage have been read
            if (step + 1 < step1) copy_x(step + 1, stage ^ 1);
            asm volatile("cp.async.commit_group;" ::: "memory");
            dequant_half(1, 0);
            if (step + 1 < step1) load_weights(step + 1);
            publish();
            issue_mma(step, stage, 1);
            phase ^= 1u;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (step1 > step0) {                                  // the last step's MMAs
            wait_mma(0, phase ^ 1u);
            wait_mma(1, phase ^ 1u);
        }
    }
    ok = __syncthreads_and(ok ? 1 : 0) != 0;

    // ---- epilogue: TMEM (lane = token, column = weight row) -> registers -> Y or partials ---------------
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok && step1 > step0 && warp < kMmaThreads / 32) {
        constexpr int CP = kMmaThreads / 128;                            // warps per TMEM lane group: column parts
        const int lane_grp = warp & 3, col_half = warp >> 2;            // TMEM lanes 32*lane_grp.., one part of the columns
        const size_t n_pad = (size_t)a.n_rb * kTileRows;
        const bool y_vec_ok = !(a.flags & (ELUTQ_FLAG_OUT_F32 | ELUTQ_FLAG_ACCUMULATE)) && (a.N % 8 == 0) &&
                              ((reinterpret_cast<uintptr_t>(a.Y) & 15) == 0);
#pragma unroll 1
        for (int tt = 0; tt < TT; ++tt) {
            const int m = m0 + tt * kTileM + lane_grp * 32 + lane;
#pragma unroll 1
            for (int c0 = col_half * (NW / CP); c0 < (col_half + 1) * (NW / CP); c0 += 32) {
                uint32_t r[32];
                const uint32_t taddr = tmem_d + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(tt * NW + c0);
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                             "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                             "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                             : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                               "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                               "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                               "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                             : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (m < a.M) store_row32(a, m, n_tile * NW + c0, r, splits, split, n_pad, y_vec_ok);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if constexpr (CG == 2) {
        cluster_barrier();           // nobody frees tensor memory or leaves while the pair may still use it
        if (warp == 0)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"((uint32_t)(TT * NW)) : "memory");
    } else {
        __syncthreads();
        if (warp == 0)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"((uint32_t)(TT * NW)) : "memory");
    }
}

template <int Q, int NW, int TT, bool WS = false, int CG = 1>
int launch_mma_cfg(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    constexpr int kSmem = (TT == 1 ? 3 : 2) * TT * kXTileBytes + (TT == 1 ? 2 : 1) * NW * kStepK * 2 + 128;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(hlq_mma_kernel<Q, NW, TT, WS, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return (int)e;
        configured[dev] = true;
    }
    const int n_tiles = (a.N + NW - 1) / NW, m_tiles = (a.M + TT * kTileM - 1) / (TT * kTileM);
    const long long tiles = (long long)n_tiles * m_tiles;
    const int max_splits = 2 * a.n_kc < 16 ? 2 * a.n_kc : 16;   // the partial buffer holds 2 * n_kc slices
    const bool pdl = true;

    auto launch = [&](int n_tile0, int n_count, int splits) -> cudaError_t {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = CG == 2 ? dim3((unsigned)m_tiles, (unsigned)n_count, (unsigned)splits)
                              : dim3((unsigned)n_count, (unsigned)m_tiles, (unsigned)splits);
        cfg.blockDim = dim3(kMmaThreads + (WS ? 32 : 0));
        cfg.dynamicSmemBytes = kSmem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl ? 1 : 0;
        if (CG == 2) {               // CTA pairs along the token dimension (the caller made sure m_tiles is even)
            attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
            attr[cfg.numAttrs].val.clusterDim.x = 2;
            attr[cfg.numAttrs].val.clusterDim.y = 1;
            attr[cfg.numAttrs].val.clusterDim.z = 1;
            cfg.numAttrs += 1;
        }
        cudaError_t e = cudaLaunchKernelEx(&cfg, hlq_mma_kernel<Q, NW, TT, WS, CG>, a, splits, n_tile0);
        count_launch(1);
        return e;
    };

    // Fewer tiles than SMs: K split while the tile count leaves SMs idle (partials cost M*N*4 bytes per split).
    if (tiles <= num_sms) {
        int splits = 1;
        while (splits * 2 <= max_splits && tiles * splits * 2 <= (long long)num_sms) splits *= 2;
        {   // a split that is no power of two (uneven step counts per CTA) only where it adds 30 % more CTAs or more
            // (measured: 8B qkv, 24 weight tiles: 6 instead of 4 splits -5 % at M = 32, 3 instead of 2 -7 % at M = 512;
            // o, 16 tiles: 9 instead of 8 splits +5 %)
            long long any = (long long)num_sms / tiles;
            if (any > max_splits) any = max_splits;
            if (any > 4 * a.n_kc) any = 4 * a.n_kc;
            if (any * 10 >= (long long)splits * 13) splits = (int)any;
        }
        if (splits > max_splits) splits = max_splits;
        cudaError_t e = launch(0, n_tiles, splits);
        if (e != cudaSuccess || splits == 1) return (int)e;
        return launch_finalize(a, splits, pdl, stream);
    }

    // More tiles than SMs: whole rounds of whole tiles, then the column stripe that would make a thin last round
    // is launched on its own with a K split that fills the GPU (reduced by the finalize kernel over those columns).
    const long long full = tiles / num_sms * num_sms;               // tiles in whole rounds
    int n_main = (int)(full / m_tiles);                             // whole columns of tiles within them
    if (n_main > n_tiles) n_main = n_tiles;
    const long long tail_tiles = (long long)(n_tiles - n_main) * m_tiles;
    int tail_splits = tail_tiles > 0 ? (int)(num_sms / tail_tiles) : 1;
    if (tail_splits > max_splits) tail_splits = max_splits;
    if (tail_splits > 4 * a.n_kc) tail_splits = 4 * a.n_kc;
    // worth it when the tail round shrinks by more than the extra launch and its partial-sum traffic cost
    const bool use_tail = tail_tiles > 0 && tail_splits >= 2 && n_main > 0 &&
                          (tail_tiles + num_sms - 1) / num_sms == 1;
    if (!use_tail) return (int)launch(0, n_tiles, 1);
    cudaError_t e = launch(0, n_main, 1);
    if (e != cudaSuccess) return (int)e;
    e = launch(n_main, n_tiles - n_main, tail_splits);
    if (e != cudaSuccess) return (int)e;
    const int col0 = n_main * NW;
    return launch_finalize(a, tail_splits, pdl, stream, col0, a.N - col0);
}

template <int Q>
int launch_mma_q(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    // Two token tiles per CTA once M exceeds one tile; 256 weight rows per CTA unless even the largest K split
    // would leave most SMs without work.
    const bool two = a.M > kTileM;
    const long long m_tiles = two ? (a.M + 2 * kTileM - 1) / (2 * kTileM) : (a.M + kTileM - 1) / kTileM;
    const long long tiles256 = (long long)((a.N + 255) / 256) * m_tiles;
    const int max_splits = 2 * a.n_kc < 16 ? 2 * a.n_kc : 16;
    bool narrow = tiles256 * max_splits * 2 <= num_sms;
    // measured: the warp-specialised form is 3-5 % faster (no CTA-wide barrier in the step, the issuing thread dequantises nothing)
    // measured: a CTA pair per weight tile (each CTA dequantises half of it) is 8-22 % faster again; it needs an even
    // number of 256-token tiles
    if (two && !narrow && m_tiles % 2 == 0) return launch_mma_cfg<Q, 256, 2, true, 2>(a, num_sms, stream);
    if (two && !narrow) return launch_mma_cfg<Q, 256, 2, true>(a, num_sms, stream);
    if (two) return narrow ? launch_mma_cfg<Q, 128, 2>(a, num_sms, stream) : launch_mma_cfg<Q, 256, 2>(a, num_sms, stream);
    return narrow ? launch_mma_cfg<Q, 128, 1>(a, num_sms, stream) : launch_mma_cfg<Q, 256, 1>(a, num_sms, stream);
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
