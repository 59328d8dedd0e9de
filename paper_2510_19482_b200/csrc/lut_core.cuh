// Device code shared by the M = 1 decode kernels (lut_gemv.cu: one call per launch; lut_chain.cu: a list of
// calls per launch): tile geometry, the weight-item register buffer, the table build (Appendix B: all partial
// sums of a slice are precomputed) and the look-up / accumulate step with per-plane scales and the offset term
// (Eq. 3 evaluated per group).
#pragma once

#include "common.cuh"

namespace elutq {

constexpr int kGemvThreads = 1024;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kTableBytes = 256 * 256;           // 256 entries x 64 columns x 4 bytes
constexpr int kModeFused = 0;      // 256-entry 0/1 tables (default)
constexpr int kModePlainG4 = 1;    // two 16-entry g = 4 tables per byte
constexpr int kModeMirror = 2;     // Appendix D mirror storage: 128-entry +-1 tables, sign applied on look-up

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

// vp = tile + lane*16 (plane vectors), pp = tile + PLANE_BYTES + lane*4 (parameter words);
// every load is base + compile-time offset.
template <int Q, int G>
__device__ __forceinline__ void load_item(Item<Q, G>& it, const uint8_t* vp, const uint8_t* pp, bool planes) {
    using C = Cfg<Q, G>;
    if (planes) static_for<0, C::NV>([&](auto i) { it.v[i] = ldg_stream_v4<i * 512>(vp); });
    static_for<0, C::NPW>([&](auto i) { it.p[i] = ldg_stream_u32<i * 128>(pp); });
}

// Builds the 64 fused tables of chunk kc and the chunk's group sums with 1024 threads.
// lane -> column pair (2*lane, 2*lane+1); warp -> high nibble hi = warp & 15 and low-nibble half
// lh = warp >> 4 (entries lo = 8*lh .. 8*lh+7).  Both columns are computed with packed fp32x2
// adds and stored with one 64-bit store per entry pair (conflict-free: 256 contiguous bytes per warp).
// X_L2: read X past the (incoherent) L1, for a kernel that outlives the producer of X.
template <int G, int MODE, bool X_L2 = false>
__device__ __forceinline__ void build_tables(uint8_t* smem, const __half* __restrict__ X, int kc, int K, int tid) {
    constexpr int W = G / 8;
    float* gsum = reinterpret_cast<float*>(smem + kTableBytes);
    const int lane = tid & 31, warp = tid >> 5;
    const int hi = warp & 15, lh = warp >> 4;
    const int k0 = kc * kChunkK + lane * 16;          // 16 activations = two byte-columns
    float2 x[8];                                       // x[i] = (x_i of column 2*lane, x_i of column 2*lane+1)
    if (k0 < K) {                                      // K is a multiple of 32, so both columns are in range together
        const uint4 r0 = X_L2 ? __ldcg(reinterpret_cast<const uint4*>(X + k0)) : *reinterpret_cast<const uint4*>(X + k0);
        const uint4 r1 = X_L2 ? __ldcg(reinterpret_cast<const uint4*>(X + k0 + 8)) : *reinterpret_cast<const uint4*>(X + k0 + 8);
        const uint32_t a[4] = {r0.x, r0.y, r0.z, r0.w}, b[4] = {r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&a[i]));
            const float2 fb = __half22float2(*reinterpret_cast<const __half2*>(&b[i]));
            x[2 * i] = make_float2(fa.x, fb.x);
            x[2 * i + 1] = make_float2(fa.y, fb.y);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = make_float2(0.f, 0.f);
    }
    // A[t] = sum of x_0..x_2 selected by the bits of t, plus x_3 for the upper half of the low nibble
    float2 A[8];
    A[0] = lh ? x[3] : make_float2(0.f, 0.f);
    A[1] = fadd2(A[0], x[0]);
    A[2] = fadd2(A[0], x[1]);
    A[3] = fadd2(A[1], x[1]);
    A[4] = fadd2(A[0], x[2]);
    A[5] = fadd2(A[1], x[2]);
    A[6] = fadd2(A[2], x[2]);
    A[7] = fadd2(A[3], x[2]);
    float2 Bv = make_float2(0.f, 0.f);                 // high-nibble partial sum (hi is warp-uniform)
#pragma unroll
    for (int b = 0; b < 4; ++b)
        if ((hi >> b) & 1) Bv = fadd2(Bv, x[4 + b]);
    float2* row = reinterpret_cast<float2*>(smem) + (size_t)(hi * 16 + lh * 8) * 32 + lane;
    float2 e7 = make_float2(0.f, 0.f);
    // mirror mode (Appendix D): entries are sums of +-x_i (+ where the index bit is set), i.e.
    // 2 * (0/1 sum) - (sum of all 8 activations); only indices with bit 7 clear (hi < 8) are stored
    float2 negsx = make_float2(0.f, 0.f);
    if (MODE == kModeMirror) {
#pragma unroll
        for (int i = 0; i < 8; ++i) negsx = fadd2(negsx, make_float2(-x[i].x, -x[i].y));
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float2 e;
        if (MODE == kModePlainG4) {
            // unfused variant: entry p holds A[lo] in rows with hi == 0 and B[hi] in rows with lo == 0
            const float2 zero = make_float2(0.f, 0.f);
            e = (hi == 0) ? A[t] : ((lh == 0 && t == 0) ? Bv : zero);
        } else {
            e = fadd2(A[t], Bv);
            if (MODE == kModeMirror) e = fadd2(fadd2(e, e), negsx);
        }
        if (MODE != kModeMirror || hi < 8) row[t * 32] = e;
        if (t == 7) e7 = fadd2(A[t], Bv);
    }
    if (warp == 31) {                                  // hi = 15, lo = 15: entry 255 = sum of the column's 8 activations
        float total = (MODE == kModeMirror) ? -(negsx.x + negsx.y) : e7.x + e7.y;
#pragma unroll
        for (int off = W / 4; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
        if ((lane % (W / 2)) == 0) gsum[lane / (W / 2)] = total;
    }
}

// Sum of n partial sums p[0], p[stride], ... in ascending order (the order fixes the rounding, so the
// result is bit-reproducible); loads are issued up to 32 at a time so that a reduction costs one or two
// L2 round trips instead of one per chunk.
__device__ __forceinline__ float sum_chunks(const float* p, size_t stride, int n) {
    float sum = 0.f;
    int c = 0;
    for (; c + 32 <= n; c += 32) {
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __ldcg(p + (size_t)(c + i) * stride);
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += v[i];
    }
    for (; c + 16 <= n; c += 16) {
        float v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __ldcg(p + (size_t)(c + i) * stride);
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += v[i];
    }
    if (c + 8 <= n) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __ldcg(p + (size_t)(c + i) * stride);
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += v[i];
        c += 8;
    }
    if (c + 4 <= n) {
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = __ldcg(p + (size_t)(c + i) * stride);
#pragma unroll
        for (int i = 0; i < 4; ++i) sum += v[i];
        c += 4;
    }
    for (; c < n; ++c) sum += __ldcg(p + (size_t)c * stride);
    return sum;
}

// Byte offset (< 128) of the lane's column inside a 256-byte table row, per step, four steps
// per register: the byte-permute in item_sum picks byte (i & 3) of colp[i >> 2] as address byte 0,
// the weight byte as address byte 1, and zero (sign-replicated msb of a byte < 128) above.
// Four steps share a phase (W >= 4), so the four bytes are computed at once:
// tau = W*((a+v) % NSG) + (r + ii0 + b) % W for b = 0..3.
template <int G>
__device__ __forceinline__ void make_colp(uint32_t (&colp)[4], int h, int l) {
    constexpr int W = G / 8, NSG = 128 / G;
#pragma unroll
    for (int w4 = 0; w4 < 4; ++w4) {
        const int v = (4 * w4) / W, ii0 = (4 * w4) % W;
        const uint32_t base = 16u * h + W * (((l / W) + v) % NSG);
        const uint32_t t = (((uint32_t)(l % W) + ii0) * 0x01010101u + 0x03020100u) & ((W - 1) * 0x01010101u);
        uint32_t vcol = (t + base * 0x01010101u) << 2;
        asm volatile("" : "+r"(vcol));   // keep the value in a register: recomputing it per item costs far more
        colp[w4] = vcol;
    }
}

// The lane's group activation sums S (all-ones table entries, reduced per group by build_tables).
template <int G>
__device__ __forceinline__ void load_group_sums(float (&S)[2 * (128 / G)], const float* gsum, int h, int l, bool used) {
    constexpr int W = G / 8, NSG = 128 / G;
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int v = 0; v < NSG; ++v)
            S[u * NSG + v] = used ? gsum[NSG * (h + 2 * u) + (l / W + v) % NSG] : 0.f;
}

// One item: look-ups, scales, offset term, half-warp combine; returns the row's partial sum over the chunk
// (valid in both half-warps).  With HAS_NEXT the registers of every consumed vector are refilled with the
// next item's data (plane vectors at nvp, parameter words at npp), so that the next item's loads are in
// flight while this one is processed, without a second buffer.
template <int Q, int G, int MODE, bool HAS_NEXT>
__device__ __forceinline__ float item_sum(Item<Q, G>& buf, const uint8_t* smem, const uint32_t (&colp)[4],
                                          const float (&S)[2 * (128 / G)], const uint8_t* nvp, const uint8_t* npp,
                                          bool use_planes, bool use_offset) {
    using C = Cfg<Q, G>;
    // Parameters: converted up front (mirror mode rewrites them) or kept as the packed fp16 words and
    // converted where used, which holds half as many registers through the look-up loop.
    constexpr bool LAZY = (MODE != kModeMirror) && Q >= 3;
    float prm[LAZY ? 1 : C::GL * (Q + 1)];
    uint32_t praw[LAZY ? C::NPW : 1];
    if constexpr (LAZY) {
#pragma unroll
        for (int i = 0; i < C::NPW; ++i) praw[i] = buf.p[i];
    } else {
#pragma unroll
        for (int i = 0; i < C::NPW; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&buf.p[i]));
            prm[2 * i] = f.x;
            prm[2 * i + 1] = f.y;
        }
    }
    auto param = [&](int idx) -> float {          // idx is a constant after unrolling
        if constexpr (LAZY) {
            const __half2 h2 = *reinterpret_cast<const __half2*>(&praw[idx >> 1]);
            return (idx & 1) ? __high2float(h2) : __low2float(h2);
        } else {
            return prm[idx];
        }
    };
    if (HAS_NEXT) static_for<0, C::NPW>([&](auto i) { buf.p[i] = ldg_stream_u32<i * 128>(npp); });
    if (MODE == kModeMirror) {
        // s^ = s / 2 and z^ = z + (1/2) sum_j s_j, formed in fp32 (exact halving, one rounding for z^)
#pragma unroll
        for (int gi = 0; gi < C::GL; ++gi) {
            float half_sum = 0.f;
#pragma unroll
            for (int j = 0; j < Q; ++j) {
                prm[gi * (Q + 1) + j] *= 0.5f;
                half_sum += prm[gi * (Q + 1) + j];
            }
            // the group-sum term carries z (unless the offset is skipped) and, when the planes are
            // used, the (1/2) sum_j s_j that the +-1 rewrite moves out of the look-ups
            prm[gi * (Q + 1) + Q] = (use_offset ? prm[gi * (Q + 1) + Q] : 0.f) + (use_planes ? half_sum : 0.f);
        }
    }
    float y = 0.f;
    if (use_planes) {
        static_for<0, 2 * Q>([&](auto uj) {
            constexpr int u = uj / Q, j = uj % Q;
            const uint32_t wd[4] = {buf.v[uj].x, buf.v[uj].y, buf.v[uj].z, buf.v[uj].w};
#pragma unroll
            for (int v = 0; v < C::NSG; ++v) {
                float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                for (int ii = 0; ii < C::W; ii += 2) {
                    float e[2];
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const int i = v * C::W + ii + t;
                        // address = (weight byte << 8) | lane column
                        const uint32_t off = prmt(wd[i >> 2], colp[i >> 2], 0xCC04 + 0x11 * (i & 3));
                        if (MODE == kModeFused) {
                            e[t] = *reinterpret_cast<const float*>(smem + off + u * 128);
                        } else if (MODE == kModeMirror) {
                            // index bit 7 set: read the complemented index and negate (the +-1 table is antisymmetric)
                            const uint32_t m = prmt(wd[i >> 2], colp[i >> 2], 0xCC8C + 0x10 * (i & 3));   // 0xFF00 or 0
                            const float tv = *reinterpret_cast<const float*>(smem + (off ^ m) + u * 128);
                            e[t] = __uint_as_float(__float_as_uint(tv) ^ ((m << 16) & 0x80000000u));
                        } else {
                            e[t] = *reinterpret_cast<const float*>(smem + (off & 0x0fffu) + u * 128)     // low nibble table
                                 + *reinterpret_cast<const float*>(smem + (off & 0xf0ffu) + u * 128);    // high nibble table
                        }
                    }
                    acc = fadd2(acc, make_float2(e[0], e[1]));
                }
                y = fmaf(param((u * C::NSG + v) * (Q + 1) + j), acc.x + acc.y, y);
            }
            // the vector is dead now: refill its registers with the next item's data
            if (HAS_NEXT) buf.v[uj] = ldg_stream_v4<uj * 512>(nvp);
        });
    }
#pragma unroll
    for (int gi = 0; gi < C::GL; ++gi) y = fmaf(param(gi * (Q + 1) + Q), S[gi], y);
    y += __shfl_xor_sync(0xffffffffu, y, 16);
    return y;
}

// ---- Items of different bit-widths through one register buffer (G = 128, fused tables), for a kernel that serves a
// list of calls of mixed q: the buffer is sized for q = 4, and one straight-line body per q works on it (the caller
// switches on the job's q).  A tile holds, per lane, 2 q plane vectors (vector (u, j) = plane j of the lane's half u,
// 512 bytes apart, half 1 after the q vectors of half 0) and q + 1 parameter words (fp16 pairs: s_0 .. s_{q-1}, z of
// half 0, then the same of half 1).  The look-ups and the order of the additions are those of item_sum, so the results
// are bit-identical.  Whether a next item exists is a run-time predicate on the refill loads (no second body).
struct ItemRt {
    uint4 v[2][4];
    uint32_t p[5];
};

constexpr __host__ __device__ int tile_bytes_g128(int q) { return 1024 * q + 128 * (q + 1); }

// vp = tile + lane * 16
template <int QC>
__device__ __forceinline__ void load_item_rt(ItemRt& it, const uint8_t* vp, int lane) {
    static_for<0, 2 * QC>([&](auto i) { it.v[i / QC][i % QC] = ldg_stream_v4<i * 512>(vp); });
    const uint8_t* pp = vp + (QC * 1024 - lane * 12);
    static_for<0, QC + 1>([&](auto i) { it.p[i] = ldg_stream_u32<i * 128>(pp); });
}

// sum of the 16 table entries one plane vector selects (the lane's 16 byte-columns of half U)
template <int U>
__device__ __forceinline__ float plane_lookups(const uint4& vec, const uint8_t* tab, const uint32_t (&colp)[4]) {
    const uint32_t wd[4] = {vec.x, vec.y, vec.z, vec.w};
    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
    for (int ii = 0; ii < 16; ii += 2) {
        float e[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int i = ii + t;
            const uint32_t off = prmt(wd[i >> 2], colp[i >> 2], 0xCC04 + 0x11 * (i & 3));   // (weight byte << 8) | lane column
            e[t] = *reinterpret_cast<const float*>(tab + off + U * 128);
        }
        acc = fadd2(acc, make_float2(e[0], e[1]));
    }
    return acc.x + acc.y;
}

// One item of bit-width QC; where `next` is non-zero the registers are refilled, as they are consumed, with the item
// at nvp (= its tile + lane * 16), which has the same bit-width.
template <int QC>
__device__ __forceinline__ float item_sum_rt(ItemRt& buf, const uint8_t* tab, const uint32_t (&colp)[4], const float (&S)[2],
                                             const uint8_t* nvp, const uint32_t next, const int lane) {
    // the scales of half 1 start at fp16 number QC + 1: bring them (and the two offsets) to fixed positions
    uint32_t s0[2] = {buf.p[0], buf.p[1]}, s1[2] = {0u, 0u}, zz;
    if constexpr (QC == 1) {
        s1[0] = buf.p[1]; zz = prmt(buf.p[0], buf.p[1], 0x7632);
    } else if constexpr (QC == 2) {
        s1[0] = prmt(buf.p[1], buf.p[2], 0x5432); zz = prmt(buf.p[1], buf.p[2], 0x7610);
    } else if constexpr (QC == 3) {
        s1[0] = buf.p[2]; s1[1] = buf.p[3]; zz = prmt(buf.p[1], buf.p[3], 0x7632);
    } else {
        s1[0] = prmt(buf.p[2], buf.p[3], 0x5432); s1[1] = prmt(buf.p[3], buf.p[4], 0x5432);
        zz = prmt(buf.p[2], buf.p[4], 0x7610);
    }
    const uint8_t* npp = nvp + (QC * 1024 - lane * 12);
    static_for<0, QC + 1>([&](auto i) { ldg_stream_u32_if<i * 128>(buf.p[i], npp, next); });
    float y = 0.f;
    static_for<0, 2 * QC>([&](auto uj) {
        constexpr int u = uj / QC, j = uj % QC;
        const __half2 h2 = *reinterpret_cast<const __half2*>(u ? &s1[j >> 1] : &s0[j >> 1]);
        const float sc = (j & 1) ? __high2float(h2) : __low2float(h2);
        y = fmaf(sc, plane_lookups<u>(buf.v[u][j], tab, colp), y);
        ldg_stream_v4_if<uj * 512>(buf.v[u][j], nvp, next);       // the vector is dead now: the next item's takes its place
    });
    const __half2 z2 = *reinterpret_cast<const __half2*>(&zz);
    y = fmaf(__low2float(z2), S[0], y);
    y = fmaf(__high2float(z2), S[1], y);
    y += __shfl_xor_sync(0xffffffffu, y, 16);
    return y;
}

// Aligned partition of one M = 1 call over the SMs: groups of `cpc` consecutive K chunks x R row ranges, one
// CTA each.  Returns false when the flat cut of the item list is predicted to finish sooner.
bool plan_gemv_partition(int n_rb, int n_kc, int num_sms, bool allow_flat, int* cpc, int* ranges);

}  // namespace elutq
