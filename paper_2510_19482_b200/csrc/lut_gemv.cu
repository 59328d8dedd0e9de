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
#include <cstdlib>
#include <map>
#include <mutex>
#include <string>

#include "common.cuh"

namespace elutq {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kTableBytes = 256 * 256;           // 256 entries x 64 columns x 4 bytes
constexpr int kSmemBytes = kTableBytes + 128;    // + up to 16 group sums + the reduction flag
constexpr int kClusterPartBytes = 32 * 1024;     // cluster mode: per-CTA partial sums (up to 512 row blocks)
constexpr int kMaxCluster = 8;
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
template <int G, int MODE>
__device__ __forceinline__ void build_tables(uint8_t* smem, const __half* __restrict__ X, int kc, int K, int tid) {
    constexpr int W = G / 8;
    float* gsum = reinterpret_cast<float*>(smem + kTableBytes);
    const int lane = tid & 31, warp = tid >> 5;
    const int hi = warp & 15, lh = warp >> 4;
    const int k0 = kc * kChunkK + lane * 16;          // 16 activations = two byte-columns
    float2 x[8];                                       // x[i] = (x_i of column 2*lane, x_i of column 2*lane+1)
    if (k0 < K) {                                      // K is a multiple of 32, so both columns are in range together
        const uint4 r0 = *reinterpret_cast<const uint4*>(X + k0);
        const uint4 r1 = *reinterpret_cast<const uint4*>(X + k0 + 8);
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

// FAST = the common call shape fixed at compile time (both terms, aligned partition with one chunk per CTA, K split
// reduced by the finalize kernel): the flag tests, the segment arithmetic and the other reduction forms drop out
// of the item loop.
template <int Q, int G, int MODE, bool FAST = false>
__global__ void __launch_bounds__(kThreads, 1) lut_gemv_kernel(const GemmArgs a) {
    using C = Cfg<Q, G>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const float* gsum = reinterpret_cast<const float*>(smem + kTableBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = lane >> 4, l = lane & 15;
    const int bid = blockIdx.x;
    // Work of this CTA: `nseg` segments of consecutive items; segment s starts at first + s * (len + jump).
    //   aligned partition: one segment per chunk of the CTA's chunk group, all over the same row range
    //                      (so one table build per chunk and no CTA straddles a chunk boundary)
    //   flat partition:    one contiguous range of the kc-major item list (jump = 0), cut at chunk ends
    int first, last, jump = 0, range = 0, range_rb0 = 0, range_rb1 = 0;
    if (a.ranges > 0) {
        // cluster mode: the n_kc CTAs of a cluster are the chunks of one row range (rank = chunk)
        const int grp = a.cluster_reduce ? bid % a.n_kc : bid / a.ranges;
        range = a.cluster_reduce ? bid / a.n_kc : bid - grp * a.ranges;
        range_rb0 = range * a.rb_q + min(range, a.rb_r);
        range_rb1 = range_rb0 + a.rb_q + (range < a.rb_r ? 1 : 0);
        const int kc0 = grp * a.cpc;
        const int nseg = min(a.cpc, a.n_kc - kc0);
        first = kc0 * a.n_rb + range_rb0;
        last = (kc0 + nseg - 1) * a.n_rb + range_rb1;       // end of the last segment
        jump = a.n_rb - (range_rb1 - range_rb0);
    } else {
        first = bid * a.items_q + min(bid, a.items_r);
        last = first + a.items_q + (bid < a.items_r ? 1 : 0);
    }
    const bool use_planes = FAST || !(a.flags & ELUTQ_FLAG_OFFSET_ONLY);
    const bool use_offset = FAST || !(a.flags & ELUTQ_FLAG_SKIP_OFFSET);

    // Byte offset (< 128) of the lane's column inside a 256-byte table row, per step, four steps
    // per register: the byte-permute below picks byte (i & 3) of colp[i >> 2] as address byte 0,
    // the weight byte as address byte 1, and zero (sign-replicated msb of a byte < 128) above.
    // Four steps share a phase (W >= 4), so the four bytes are computed at once:
    // tau = W*((a+v) % NSG) + (r + ii0 + b) % W for b = 0..3.
    uint32_t colp[4];
#pragma unroll
    for (int w4 = 0; w4 < 4; ++w4) {
        const int v = (4 * w4) / C::W, ii0 = (4 * w4) % C::W;
        const uint32_t base = 16u * h + C::W * (((l / C::W) + v) % C::NSG);
        const uint32_t t = (((uint32_t)(l % C::W) + ii0) * 0x01010101u + 0x03020100u) & ((C::W - 1) * 0x01010101u);
        uint32_t vcol = (t + base * 0x01010101u) << 2;
        asm volatile("" : "+r"(vcol));   // keep the value in a register: recomputing it per item costs far more
        colp[w4] = vcol;
    }

    // One register buffer per warp: every plane vector (and the parameter words) is reloaded with
    // the next item's data right after its last use, so the loads of item i+1 are in flight while
    // item i is processed, without a second buffer.
    Item<Q, G> buf;
    const int stride = a.active_warps;
    const int seg_len0 = (a.ranges > 0) ? (range_rb1 - range_rb0) : (last - first);
    // first item of this warp: position `warp` in the concatenated segments
    int it = last, it_end = first + seg_len0;                // it_end: end of the segment `it` lies in
    if (warp < stride) {
        it = first + warp;
        while (it >= it_end && it_end < last) { it += jump; it_end += a.n_rb; }
        if (it >= it_end) it = last;
    }
    if (it < last)
        load_item<Q, G>(buf, a.tiles + (size_t)it * C::TILE_BYTES + lane * 16,
                        a.tiles + (size_t)it * C::TILE_BYTES + C::PLANE_BYTES + lane * 4, use_planes);

    // weights do not depend on the previous kernel in the stream; X, Y and the workspace do
    grid_launch_dependents();
    grid_dependency_wait();

    const int n_pad = a.n_rb * kTileRows;
    int seg = first;
    while (seg < last) {
        const int kc = seg / a.n_rb;
        const int seg_end = (a.ranges > 0) ? seg + seg_len0 : min(last, (kc + 1) * a.n_rb);
        __syncthreads();
        build_tables<G, MODE>(smem, a.X, kc, a.K, tid);
        __syncthreads();

        float S[C::GL];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int v = 0; v < C::NSG; ++v)
                S[u * C::NSG + v] = (use_offset || MODE == kModeMirror) ? gsum[C::NSG * (h + 2 * u) + (l / C::W + v) % C::NSG] : 0.f;

        float* cpart = reinterpret_cast<float*>(smem + kTableBytes + 128);   // cluster mode: this CTA's partial sums
        const uint8_t* nvp = nullptr;     // next item's plane vectors / parameter words for this lane
        const uint8_t* npp = nullptr;
        // One item: look-ups, scales, offset term, half-warp combine; with HAS_NEXT the registers of
        // every consumed vector are refilled with the next item's data.
        auto do_item = [&](auto has_next_c) {
            constexpr bool HAS_NEXT = decltype(has_next_c)::value != 0;
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

            const int row = (it - kc * a.n_rb) * kTileRows + l;
            if (!FAST && a.n_kc == 1) {
                if (h == 0 && row < a.N) store_out(a, (size_t)row, y);
            } else if (h == 0) {
                if (!FAST && a.cluster_reduce) cpart[row - range_rb0 * kTileRows] = y;
                else a.partials[(size_t)kc * n_pad + row] = y;
            }
        };

        while (it < seg_end) {
            // next item of this warp: `stride` positions further in the concatenated segments
            int nit = it + stride, nend = it_end;
            if (!FAST) while (nit >= nend && nend < last) { nit += jump; nend += a.n_rb; }
            const bool has_next = nit < nend && (FAST || !(a.flags & 0x80000000u));
            nvp = a.tiles + (size_t)nit * C::TILE_BYTES + lane * 16;
            npp = nvp + (C::PLANE_BYTES - lane * 12);
            if (has_next) do_item(IntC<1>{});
            else do_item(IntC<0>{});
            it = (nit < nend) ? nit : last;
            it_end = nend;
        }

        seg = (a.ranges > 0) ? seg + a.n_rb : seg_end;
    }

    if (!FAST && a.cluster_reduce && !(a.flags & 0x40000000u)) {
        // K-split reduction inside the cluster: every CTA holds the partial sums of its chunk for the
        // cluster's row range in shared memory; after the cluster barrier CTA c adds, for its share of the
        // rows, the n_kc partials in ascending chunk order (bit-reproducible) straight from its peers'
        // shared memory.  No workspace, no second kernel.
        const float* cpart = reinterpret_cast<const float*>(smem + kTableBytes + 128);
        cluster_barrier();
        const int rows = (range_rb1 - range_rb0) * kTileRows;
        const int rank = bid % a.n_kc;
        const int per = (rows + a.n_kc - 1) / a.n_kc;
        const int r_end = min(rows, (rank + 1) * per);
        for (int r = rank * per + tid; r < r_end; r += kThreads) {
            float sum = 0.f;
            for (int k = 0; k < a.n_kc; ++k) sum += ld_cluster_f32(cpart + r, (unsigned)k);
            const int row = range_rb0 * kTileRows + r;
            if (row < a.N) store_out(a, (size_t)row, sum);
        }
        cluster_barrier();          // nobody leaves while a peer may still read its shared memory
    } else if (!FAST && a.fused_reduce && a.n_kc > 1) {
        // In-kernel K-split reduction: each CTA publishes its partials and takes one ticket for its row
        // range; the CTA that draws the last ticket of the range adds the chunks in ascending order
        // (bit-reproducible) and writes Y.  The counter wraps to zero, ready for the next call.
        int* flag = reinterpret_cast<int*>(smem + kTableBytes + 64);
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned old = atomicInc(a.counters + range, (unsigned)(a.n_kc - 1));
            *flag = (old == (unsigned)(a.n_kc - 1)) ? 1 : 0;
        }
        __syncthreads();
        if (*flag) {
            __threadfence();
            const int row_end = min(range_rb1 * kTileRows, a.N);
            for (int row = range_rb0 * kTileRows + tid; row < row_end; row += kThreads) {
                const float* p = a.partials + row;
                store_out(a, (size_t)row, sum_chunks(p, (size_t)n_pad, a.n_kc));
            }
        }
    }
}

// K-split epilogue: Y[m][n] = sum over the K chunks of partials[chunk][m][n], chunks added in ascending
// order (bit-reproducible), then the output conversion.  One thread per output element.  Launched right
// behind the main kernel with programmatic dependent launch: the grid dependency wait is the only barrier.
__global__ void __launch_bounds__(256) lut_finalize_kernel(const GemmArgs a, const int n_chunks, const int col0, const int cols) {
    grid_launch_dependents();
    grid_dependency_wait();
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)a.M * cols) return;
    const int m = (int)(idx / cols), row = col0 + (int)(idx % cols);
    const size_t n_pad = (size_t)a.n_rb * kTileRows;
    store_out(a, (size_t)m * a.N + row, sum_chunks(a.partials + (size_t)m * n_pad + row, (size_t)a.M * n_pad, n_chunks));
}

// The same epilogue for many chunks and few outputs: P warps share 32 outputs, warp p sums the contiguous
// chunk range [p * per, (p + 1) * per) in ascending order, and the P sub-sums are added in ascending order
// of p: a fixed order again, so the result stays bit-reproducible (it differs in rounding from the
// single-thread order, which is why this form is only used above 8 chunks, where no other reduction
// path exists to be compared with).
__global__ void __launch_bounds__(256) lut_finalize_parts_kernel(const GemmArgs a, const int n_chunks, const int per,
                                                                 const int col0, const int cols) {
    __shared__ float sub[8][32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int lane = threadIdx.x & 31, part = threadIdx.x >> 5, parts = blockDim.x >> 5;
    const long long idx = (long long)blockIdx.x * 32 + lane;
    const bool live = idx < (long long)a.M * cols;
    const int m = live ? (int)(idx / cols) : 0, row = live ? col0 + (int)(idx % cols) : 0;
    const size_t n_pad = (size_t)a.n_rb * kTileRows;
    const int c0 = part * per, c1 = min(n_chunks, c0 + per);
    float v = 0.f;
    if (live && c0 < c1)
        v = sum_chunks(a.partials + ((size_t)c0 * a.M + m) * n_pad + row, (size_t)a.M * n_pad, c1 - c0);
    sub[part][lane] = v;
    __syncthreads();
    if (part == 0 && live) {
        float y = sub[0][lane];
        for (int p = 1; p < parts; ++p) y += sub[p][lane];
        store_out(a, (size_t)m * a.N + row, y);
    }
}

}  // namespace

// Debug switches read once from the environment (0 when unset): launch-shape experiments only.
int debug_env(const char* name) {
    static std::map<std::string, int> cache;
    static std::mutex mu;
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(name);
    if (it != cache.end()) return it->second;
    const char* v = getenv(name);
    const int val = v ? atoi(v) : 0;
    cache[name] = val;
    return val;
}

int launch_finalize(const GemmArgs& a, int n_chunks, bool pdl, cudaStream_t stream, int col0, int cols) {
    if (cols <= 0) { col0 = 0; cols = a.N; }
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const long long outputs = (long long)a.M * cols;
    // The reduction is latency-bound (n_chunks independent loads per output), so it wants all the
    // parallelism it can get: above 8 chunks, and while the outputs alone do not fill the GPU, several
    // warps share an output's chunks (measured on N = 8192, K = 28672: 8.2 us -> 2.1 us).
    int parts = 1;
    if (n_chunks > 8 && outputs < 65536 && debug_env("ELUTQ_DEBUG_FINALIZE_PARTS") >= 0) {
        parts = (n_chunks + 7) / 8;
        if (parts > 8) parts = 8;
        if (debug_env("ELUTQ_DEBUG_FINALIZE_PARTS") > 0) parts = debug_env("ELUTQ_DEBUG_FINALIZE_PARTS");
        if (parts > 8) parts = 8;
    }
    cudaError_t e;
    if (parts > 1) {
        const int per = (n_chunks + parts - 1) / parts;
        cfg.gridDim = dim3((unsigned)((outputs + 31) / 32));
        cfg.blockDim = dim3(32 * parts);
        e = cudaLaunchKernelEx(&cfg, lut_finalize_parts_kernel, a, n_chunks, per, col0, cols);
    } else {
        // one thread per output element
        cfg.gridDim = dim3((unsigned)((outputs + 255) / 256));
        cfg.blockDim = dim3(256);
        e = cudaLaunchKernelEx(&cfg, lut_finalize_kernel, a, n_chunks, col0, cols);
    }
    count_launch(1);
    return (int)e;
}

namespace {

template <int Q, int G, int MODE>
int launch_one(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(lut_gemv_kernel<Q, G, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kSmemBytes + kClusterPartBytes);
        if (e != cudaSuccess) return (int)e;
        configured[dev] = true;
    }
    const long long total = (long long)a.n_kc * a.n_rb;
    if (total >= (1LL << 31) - kWarps) return (int)cudaErrorInvalidValue;
    long long grid = total < num_sms ? total : num_sms;   // one 1024-thread CTA per SM
    if (debug_env("ELUTQ_DEBUG_GRID") > 0) grid = debug_env("ELUTQ_DEBUG_GRID");
    if (grid > total) grid = total;
    if (grid < 1) grid = 1;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    GemmArgs b = a;
    b.items_q = (int)(total / grid);
    b.items_r = (int)(total % grid);
    // Aligned partition: groups of `cpc` consecutive chunks x R row ranges, one CTA each.  Pick the cpc
    // that keeps the SMs busiest (work / (SMs * largest CTA share)); fall back to the flat partition
    // of the item list when no choice reaches 80 %.
    b.ranges = 0; b.rb_q = 0; b.rb_r = 0; b.fused_reduce = 0; b.cpc = 1; b.cluster_reduce = 0;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = debug_env("ELUTQ_DEBUG_NO_PDL") > 0 ? 0 : 1;
    bool use_cluster = false;
    if (a.n_kc >= 2 && a.n_kc <= kMaxCluster && (a.flags & ELUTQ_FLAG_CLUSTER_REDUCE)) {
        // Up to 8 chunks: one cluster per row range, one CTA per chunk, reduction through distributed shared memory.
        int R = (num_sms - 20) / a.n_kc;
        if (R < 1) R = 1;
        if (R > a.n_rb) R = a.n_rb;
        if (debug_env("ELUTQ_DEBUG_R") > 0 && debug_env("ELUTQ_DEBUG_R") < R) R = debug_env("ELUTQ_DEBUG_R");
        if ((a.n_rb + R - 1) / R * kTileRows * (int)sizeof(float) <= kClusterPartBytes) {
            cfg.dynamicSmemBytes = kSmemBytes + kClusterPartBytes;
            cfg.gridDim = dim3((unsigned)(R * a.n_kc));
            attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
            attr[cfg.numAttrs].val.clusterDim.x = (unsigned)a.n_kc;
            attr[cfg.numAttrs].val.clusterDim.y = 1;
            attr[cfg.numAttrs].val.clusterDim.z = 1;
            cfg.numAttrs += 1;
            int max_clusters = 0;
            cudaError_t ce = cudaOccupancyMaxActiveClusters(&max_clusters, lut_gemv_kernel<Q, G, MODE>, &cfg);
            if (ce == cudaSuccess && max_clusters >= 1) {
                if (R > max_clusters) R = max_clusters;      // one wave of clusters
                use_cluster = true;
                b.cluster_reduce = 1;
                b.ranges = R;
                b.rb_q = a.n_rb / R;
                b.rb_r = a.n_rb % R;
                grid = (long long)R * a.n_kc;
                cfg.gridDim = dim3((unsigned)grid);
            } else {
                (void)cudaGetLastError();
                cfg.numAttrs -= 1;
                cfg.dynamicSmemBytes = kSmemBytes;
                cfg.gridDim = dim3((unsigned)grid);
            }
        }
    }
    if (!use_cluster && a.n_kc > 1 && debug_env("ELUTQ_DEBUG_FLAT") == 0) {
        // Cost model in item times: the kernel lasts as long as its largest CTA, i.e. that CTA's items
        // plus ~16 item times per table build (measured: an extra build costs far more than the
        // imbalance it could remove).  Minimise that makespan over the aligned choices and the flat one.
        const double kBuild = 16.0;
        const long long flat_grid = total < num_sms ? total : num_sms;
        const long long flat_items = (total + flat_grid - 1) / flat_grid;
        double best = (double)flat_items + kBuild * (double)((flat_items + a.n_rb - 1) / a.n_rb + 1);   // flat partition
        int best_cpc = 0, best_R = 0;
        const int force_cpc = debug_env("ELUTQ_DEBUG_CPC"), force_R = debug_env("ELUTQ_DEBUG_R");
        for (int cpc = 1; cpc <= 8 && cpc <= a.n_kc; ++cpc) {
            if (force_cpc > 0 && cpc != force_cpc) continue;
            const int groups = (a.n_kc + cpc - 1) / cpc;
            int R = num_sms / groups;
            // Short kernels (< ~100 items per CTA) run faster in a stream of calls when about 20 SMs stay
            // free for the early-launched CTAs of the kernels that follow (measured: 128 CTAs beat 144 by
            // ~12 % on 20-25 MB layers); long kernels want every SM.
            const int R_spare = (num_sms - 20) / groups;
            if (R_spare >= 1 && (a.n_rb + R - 1) / R < 100) R = R_spare;
            if (R > a.n_rb) R = a.n_rb;
            if (force_R > 0 && force_R < R) R = force_R;
            if (R < 1) continue;
            const double span = (double)cpc * ((double)((a.n_rb + R - 1) / R) + kBuild);
            if (span < best - 1e-9 || force_cpc > 0) { best = span; best_cpc = cpc; best_R = R; }
        }
        if (best_cpc > 0) {
            b.cpc = best_cpc;
            b.ranges = best_R;
            b.rb_q = a.n_rb / best_R;
            b.rb_r = a.n_rb % best_R;
            grid = (long long)best_R * ((a.n_kc + best_cpc - 1) / best_cpc);
            cfg.gridDim = dim3((unsigned)grid);
            b.fused_reduce = (best_cpc == 1 && a.counters != nullptr && debug_env("ELUTQ_DEBUG_FUSED") > 0) ? 1 : 0;
        }
    }
    {   // even rounds: with R = ceil(items/32) rounds, ceil(items/R) warps take items
        const int items_max = b.items_q + (b.items_r ? 1 : 0);
        const int rounds = (items_max + kWarps - 1) / kWarps;
        b.active_warps = kWarps;   // measured: evening out the rounds (ceil(items/rounds) warps) gains nothing
        (void)rounds;
        if (debug_env("ELUTQ_DEBUG_WARPS") > 0) b.active_warps = debug_env("ELUTQ_DEBUG_WARPS");
        if (b.active_warps > kWarps) b.active_warps = kWarps;
        if (b.active_warps < 1) b.active_warps = 1;
    }
    if (debug_env("ELUTQ_DEBUG_NOLOAD") > 0) b.flags |= 0x80000000u;
    if (debug_env("ELUTQ_DEBUG_SKIP_CLUSTER_REDUCE") > 0) b.flags |= 0x40000000u;   // timing experiment only   // timing experiment: skip reloads (results invalid)
    const bool fast = MODE == kModeFused && !use_cluster && b.ranges > 0 && b.cpc == 1 && a.n_kc > 1 && !b.fused_reduce &&
                      !(b.flags & (ELUTQ_FLAG_SKIP_OFFSET | ELUTQ_FLAG_OFFSET_ONLY | 0xC0000000u)) && debug_env("ELUTQ_DEBUG_NO_FAST") == 0;
    cudaError_t e;
    if constexpr (MODE == kModeFused) {
        if (fast) {
            static bool configured_fast[64] = {};
            if (dev >= 0 && dev < 64 && !configured_fast[dev]) {
                e = cudaFuncSetAttribute(lut_gemv_kernel<Q, G, MODE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
                if (e != cudaSuccess) return (int)e;
                configured_fast[dev] = true;
            }
            e = cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, G, MODE, true>, b);
        } else {
            e = cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, G, MODE, false>, b);
        }
    } else {
        e = cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, G, MODE, false>, b);
    }
    count_launch(1);
    if (e != cudaSuccess || a.n_kc == 1 || b.fused_reduce || b.cluster_reduce) return (int)e;
    if (debug_env("ELUTQ_DEBUG_SKIP_FINALIZE") > 0) return (int)e;   // timing experiment only (Y is not written)
    return launch_finalize(b, a.n_kc, debug_env("ELUTQ_DEBUG_NO_PDL") == 0, stream);
}

template <int Q>
int launch_q(const GemmArgs& a, int G, int num_sms, cudaStream_t stream) {
    switch (G) {
        case 32: return launch_one<Q, 32, kModeFused>(a, num_sms, stream);
        case 64: return launch_one<Q, 64, kModeFused>(a, num_sms, stream);
        case 128:
            if (a.flags & ELUTQ_FLAG_PLAIN_G4) return launch_one<Q, 128, kModePlainG4>(a, num_sms, stream);
            if (a.flags & ELUTQ_FLAG_MIRROR) return launch_one<Q, 128, kModeMirror>(a, num_sms, stream);
            return launch_one<Q, 128, kModeFused>(a, num_sms, stream);
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
