// 2 <= M < ELUTQ_TENSOR_MIN_M (or any M > 1 on request): batched look-up GEMM over the same packed layout.
//
// MB activation rows are processed per pass: a table entry holds the partial sums of all MB rows for one
// (byte value, column), so one weight byte costs one byte-permute, one shared-memory load and the adds of MB
// rows.  fp32 tables: MB = 2 or 4 (8- or 16-byte entries, packed fp32x2 adds).  Quantised tables of Appendix D
// as labelled variants: fp16 entries (MB = 4 or 8, converted and added in fp32) and int8 entries (MB = 8, one
// scale per row and group, integer adds in 16-bit lanes).  Tables of one pass cover half a tile (256 input
// columns = super-groups 2u and 2u+1 of a chunk): 256 entries x 32 columns.
//
// Work list: (row batch mb, half chunk kc2 = 2*kc + u, row block rb), flattened in that order.  A CTA (one
// 1024-thread CTA per SM) owns a row range of one (mb, kc2) segment and builds its tables once (aligned
// partition), or, when that would idle more than a tenth of the SMs, an equal contiguous cut of the whole list
// (tables are rebuilt when the cut crosses a segment boundary).  Partial sums go to partials[kc2][m][n]; the
// finalize kernel adds the 2*n_kc half chunks in ascending order.  With fp32 tables the shared-memory look-up
// rate (one 4-byte entry per lane per cycle per SM), not HBM, bounds this path: time grows with M.
#include "common.cuh"

namespace elutq {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kHalfK = 256;                        // input columns covered by one table set

// TQ selects the table entry format (table quantisation of Appendix D): 0 = fp32 (MB floats per entry);
// 1 = fp16 (first form: MB halves per entry, one 8- or 16-byte load serves 4 or 8 activation rows);
// 2 = int8 (second form, lossy: MB = 8 biased bytes per entry, one scale per activation row and 128-column group).
template <int Q, int G, int MB, int TQ = 0>
struct BCfg {
    static constexpr int W = G / 8;
    static constexpr int NSG = 128 / G;
    static constexpr int NPW = 2 * NSG * (Q + 1) / 2;          // parameter words per lane (both halves)
    static constexpr int PLANE_BYTES = 1024 * Q;
    static constexpr int TILE_BYTES = PLANE_BYTES + 128 * NPW;
    static constexpr int ENTRY_BYTES = (TQ == 0 ? 4 : TQ == 1 ? 2 : 1) * MB;
    static constexpr int TABLE_BYTES = 256 * 32 * ENTRY_BYTES; // 64 KiB (8-byte entries) or 128 KiB (16-byte entries)
    // + group sums [256/G][MB] (+ for int8 the row scales [2][MB]) + slack
    static constexpr int SMEM_BYTES = TABLE_BYTES + (256 / G) * MB * 4 + (TQ == 2 ? 2 * MB * 4 : 0) + 64;
};

// Pieces shared by the three table builders below.  A thread owns byte-column `lane` of the half chunk (8 consecutive
// activations) for a pair of activation rows, held as float2 (row m, row m + 1) per activation.

// x[i] = (x_i of row m, x_i of row m + 1) for the 8 activations from column k0 on; rows >= M and columns >= K are zeros.
__device__ __forceinline__ void load_row_pair(float2 (&x)[8], const __half* __restrict__ X, int M, int K, int m, int k0) {
    float xa[8], xb[8];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float* dst = r ? xb : xa;
        if (m + r < M && k0 < K) {
            const uint4 raw = *reinterpret_cast<const uint4*>(X + (size_t)(m + r) * K + k0);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
                dst[2 * i] = f.x;
                dst[2 * i + 1] = f.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = 0.f;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = make_float2(xa[i], xb[i]);
}

// The entries of the thread's 8 table rows (high nibble hi, low nibble 8*lh + t) are A[t] + Bv: A[t] = the sum of
// x_0..x_2 selected by the bits of t (plus x_3 for the upper half of the low nibble), Bv = the sum of x_4..x_7
// selected by the bits of hi.
__device__ __forceinline__ void half_table_sums(float2 (&A)[8], float2& Bv, const float2 (&x)[8], int hi, int lh) {
    A[0] = lh ? x[3] : make_float2(0.f, 0.f);
    A[1] = fadd2(A[0], x[0]);
    A[2] = fadd2(A[0], x[1]);
    A[3] = fadd2(A[1], x[1]);
    A[4] = fadd2(A[0], x[2]);
    A[5] = fadd2(A[1], x[2]);
    A[6] = fadd2(A[2], x[2]);
    A[7] = fadd2(A[3], x[2]);
    Bv = make_float2(0.f, 0.f);
#pragma unroll
    for (int b = 0; b < 4; ++b)
        if ((hi >> b) & 1) Bv = fadd2(Bv, x[4 + b]);
}

// Entry 255 (warp 31) is the column's activation sum: reduced over the W columns of a quantisation group, it gives
// the group sums of the offset term for the two rows of the pair, gsum[group][row], row = `row` and `row` + 1 of MB.
template <int W, int MB>
__device__ __forceinline__ void store_group_sums(float* gsum, const float2 e255, int lane, int row) {
    float sx = e255.x, sy = e255.y;
#pragma unroll
    for (int off = W / 2; off >= 1; off >>= 1) {
        sx += __shfl_xor_sync(0xffffffffu, sx, off);
        sy += __shfl_xor_sync(0xffffffffu, sy, off);
    }
    if ((lane % W) == 0) {
        gsum[(lane / W) * MB + row] = sx;
        gsum[(lane / W) * MB + row + 1] = sy;
    }
}

// Tables of half chunk kc2 for rows m0 .. m0+MB-1: lane -> column c (8 activations of every row),
// warp -> high nibble hi = warp & 15 and low-nibble half lh = warp >> 4.  Rows are paired in the
// packed adds.  Rows >= M and columns >= K contribute zeros.
template <int G, int MB>
__device__ __forceinline__ void build_tables_mb(uint8_t* smem, int table_bytes, const __half* __restrict__ X,
                                                int M, int K, int m0, int kc2, int tid) {
    constexpr int W = G / 8;
    constexpr int NP = MB / 2;                          // row pairs
    float* gsum = reinterpret_cast<float*>(smem + table_bytes);   // [256/G groups][MB]
    const int lane = tid & 31, warp = tid >> 5;
    const int hi = warp & 15, lh = warp >> 4;
    const int k0 = kc2 * kHalfK + lane * 8;
    uint8_t* rowp = smem + (size_t)(hi * 16 + lh * 8) * 32 * (4 * MB) + lane * (4 * MB);
    float2 A[NP][8], Bv[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        float2 x[8];
        load_row_pair(x, X, M, K, m0 + 2 * p, k0);
        half_table_sums(A[p], Bv[p], x, hi, lh);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float2 e[NP];
#pragma unroll
        for (int p = 0; p < NP; ++p) e[p] = fadd2(A[p][t], Bv[p]);
        uint8_t* dst = rowp + (size_t)t * 32 * (4 * MB);
        if (MB == 2) *reinterpret_cast<float2*>(dst) = e[0];
        else *reinterpret_cast<float4*>(dst) = make_float4(e[0].x, e[0].y, e[NP - 1].x, e[NP - 1].y);
        if (t == 7 && warp == 31) {
#pragma unroll
            for (int p = 0; p < NP; ++p) store_group_sums<W, MB>(gsum, e[p], lane, 2 * p);
        }
    }
}

// Half-precision tables for rows m0 .. m0+MB-1 (MB = 4 or 8): same decomposition as build_tables_mb, four rows
// at a time; every entry is formed in fp32 and rounded once to fp16.  The activation sums for the offset term
// stay in fp32.
template <int G, int MB>
__device__ __forceinline__ void build_tables_half(uint8_t* smem, int table_bytes, const __half* __restrict__ X,
                                                  int M, int K, int m0, int kc2, int tid) {
    constexpr int W = G / 8;
    constexpr int EB = 2 * MB;                          // entry bytes
    float* gsum = reinterpret_cast<float*>(smem + table_bytes);   // [256/G groups][MB]
    const int lane = tid & 31, warp = tid >> 5;
    const int hi = warp & 15, lh = warp >> 4;
    const int k0 = kc2 * kHalfK + lane * 8;
    uint8_t* rowp = smem + (size_t)(hi * 16 + lh * 8) * 32 * EB + lane * EB;
#pragma unroll 1
    for (int quad = 0; quad < MB / 4; ++quad) {
        float2 A[2][8], Bv[2];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            float2 x[8];
            load_row_pair(x, X, M, K, m0 + 4 * quad + 2 * p, k0);
            half_table_sums(A[p], Bv[p], x, hi, lh);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const float2 ea = fadd2(A[0][t], Bv[0]), eb = fadd2(A[1][t], Bv[1]);
            const __half2 ha = __floats2half2_rn(ea.x, ea.y), hb = __floats2half2_rn(eb.x, eb.y);
            *reinterpret_cast<uint2*>(rowp + (size_t)t * 32 * EB + quad * 8) =
                make_uint2(*reinterpret_cast<const uint32_t*>(&ha), *reinterpret_cast<const uint32_t*>(&hb));
            if (t == 7 && warp == 31) {
                store_group_sums<W, MB>(gsum, ea, lane, 4 * quad);
                store_group_sums<W, MB>(gsum, eb, lane, 4 * quad + 2);
            }
        }
    }
}

// int8 tables for rows m0 .. m0+7 at G = 128 (the half chunk holds two groups of 16 byte-columns): per row and group
// one scale = (largest possible |entry| of the group, i.e. max over its columns of sum_i |x_i|) / 127; an entry is
// round-to-nearest(entry / scale) + 128, one byte per row.  Group sums (offset term) stay in fp32.
__device__ __forceinline__ void build_tables_i8(uint8_t* smem, int table_bytes, const __half* __restrict__ X,
                                                int M, int K, int m0, int kc2, int tid) {
    constexpr int MB = 8, W = 16;
    float* gsum = reinterpret_cast<float*>(smem + table_bytes);   // [2 groups][MB]
    float* rscale = gsum + 2 * MB;                                // [2 groups][MB]
    const int lane = tid & 31, warp = tid >> 5;
    const int hi = warp & 15, lh = warp >> 4;
    const int k0 = kc2 * kHalfK + lane * 8;
    uint8_t* rowp = smem + (size_t)(hi * 16 + lh * 8) * 32 * MB + lane * MB;
#pragma unroll 1
    for (int quad = 0; quad < 2; ++quad) {
        float2 A[2][8], Bv[2], inv[2];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            float2 x[8];
            load_row_pair(x, X, M, K, m0 + 4 * quad + 2 * p, k0);
            // largest |entry| this column can produce, then the group's maximum over its 16 columns
            float ax = 0.f, ay = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) { ax += fabsf(x[i].x); ay += fabsf(x[i].y); }
#pragma unroll
            for (int off = W / 2; off >= 1; off >>= 1) {
                ax = fmaxf(ax, __shfl_xor_sync(0xffffffffu, ax, off));
                ay = fmaxf(ay, __shfl_xor_sync(0xffffffffu, ay, off));
            }
            inv[p] = make_float2(ax > 0.f ? 127.f / ax : 0.f, ay > 0.f ? 127.f / ay : 0.f);
            if (warp == 31 && (lane % W) == 0) {
                rscale[(lane / W) * MB + 4 * quad + 2 * p] = ax / 127.f;
                rscale[(lane / W) * MB + 4 * quad + 2 * p + 1] = ay / 127.f;
            }
            half_table_sums(A[p], Bv[p], x, hi, lh);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const float2 ea = fadd2(A[0][t], Bv[0]), eb = fadd2(A[1][t], Bv[1]);
            const uint32_t c0 = (uint32_t)(__float2int_rn(ea.x * inv[0].x) + 128), c1 = (uint32_t)(__float2int_rn(ea.y * inv[0].y) + 128);
            const uint32_t c2 = (uint32_t)(__float2int_rn(eb.x * inv[1].x) + 128), c3 = (uint32_t)(__float2int_rn(eb.y * inv[1].y) + 128);
            *reinterpret_cast<uint32_t*>(rowp + (size_t)t * 32 * MB + quad * 4) = c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
            if (t == 7 && warp == 31) {
                store_group_sums<W, MB>(gsum, ea, lane, 4 * quad);
                store_group_sums<W, MB>(gsum, eb, lane, 4 * quad + 2);
            }
        }
    }
}

template <int Q, int G, int MB, int TQ>
__global__ void __launch_bounds__(kThreads, 1) lut_gemm_kernel(const GemmArgs a) {
    using C = BCfg<Q, G, MB, TQ>;
    constexpr bool TH = (TQ == 1);
    extern __shared__ __align__(1024) uint8_t smem[];
    const float* gsum = reinterpret_cast<const float*>(smem + C::TABLE_BYTES);

    if (!blob_header_matches(a.tiles, Q, G, a.N, a.K, a.counters)) return;   // before any tile is read
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = lane >> 4, l = lane & 15;
    const int bid = blockIdx.x;
    // CTA b owns a contiguous range of the item list: either an even cut of the whole list, or (aligned partition,
    // ranges > 0) one of `ranges` row ranges of a single (row batch, half chunk) segment, so that it builds its
    // tables exactly once.
    int first, last;
    if (a.ranges > 0) {
        const int seg = bid / a.ranges, r = bid - seg * a.ranges;
        first = seg * a.n_rb + r * a.rb_q + min(r, a.rb_r);
        last = first + a.rb_q + (r < a.rb_r ? 1 : 0);
    } else {
        first = bid * a.items_q + min(bid, a.items_r);
        last = first + a.items_q + (bid < a.items_r ? 1 : 0);
    }
    const bool use_planes = !(a.flags & ELUTQ_FLAG_OFFSET_ONLY);
    const bool use_offset = !(a.flags & ELUTQ_FLAG_SKIP_OFFSET);
    const int n_kc2 = 2 * a.n_kc;
    const int per_mb = n_kc2 * a.n_rb;                 // items per row batch
    const size_t n_pad = (size_t)a.n_rb * kTileRows;

    // Lane column byte offsets inside a table row (column * 8 bytes; the address is doubled for 16-byte entries),
    // three steps per register, the fourth byte stays zero and supplies the upper address bytes.
    uint32_t colp[6];
#pragma unroll
    for (int w3 = 0; w3 < 6; ++w3) {
        uint32_t v = 0;
#pragma unroll
        for (int b = 0; b < 3; ++b) {
            const int i = 3 * w3 + b;
            if (i < 16) v |= (8u * (16 * h + tau_of(l, i, C::W, C::NSG))) << (8 * b);
        }
        asm volatile("" : "+r"(v));
        colp[w3] = v;
    }

    grid_launch_dependents();
    grid_dependency_wait();

    int seg = first;
    while (seg < last) {
        const int mb = seg / per_mb;
        const int rem = seg - mb * per_mb;
        const int kc2 = rem / a.n_rb;
        const int seg_end = min(last, mb * per_mb + (kc2 + 1) * a.n_rb);
        const int m0 = mb * MB;
        const int u = kc2 & 1;
        __syncthreads();
        if constexpr (TQ == 2) build_tables_i8(smem, C::TABLE_BYTES, a.X, a.M, a.K, m0, kc2, tid);
        else if constexpr (TQ == 1) build_tables_half<G, MB>(smem, C::TABLE_BYTES, a.X, a.M, a.K, m0, kc2, tid);
        else build_tables_mb<G, MB>(smem, C::TABLE_BYTES, a.X, a.M, a.K, m0, kc2, tid);
        __syncthreads();

        // group sums of this lane's groups in this half: group (NSG*h + (a+v) % NSG) of the half
        float S[C::NSG][MB];
#pragma unroll
        for (int v = 0; v < C::NSG; ++v)
#pragma unroll
            for (int m = 0; m < MB; ++m)
                S[v][m] = use_offset ? gsum[(C::NSG * h + (l / C::W + v) % C::NSG) * MB + m] : 0.f;

        for (int it = seg + warp; it < seg_end; it += kWarps) {
            const int rb = it - mb * per_mb - kc2 * a.n_rb;
            const uint8_t* tile = a.tiles + ((size_t)(kc2 >> 1) * a.n_rb + rb) * C::TILE_BYTES;
            uint4 vec[Q];
            uint32_t pw[C::NPW];
            if (use_planes) static_for<0, Q>([&](auto j) { vec[j] = ldg_stream_v4<0>(tile + ((u * Q + j) * 32 + lane) * 16); });
            static_for<0, C::NPW>([&](auto i) { pw[i] = ldg_stream_u32<0>(tile + C::PLANE_BYTES + (i * 32 + lane) * 4); });
            float prm_all[2 * C::NPW];
#pragma unroll
            for (int i = 0; i < C::NPW; ++i) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&pw[i]));
                prm_all[2 * i] = f.x;
                prm_all[2 * i + 1] = f.y;
            }
            float prm[C::NSG * (Q + 1)];               // this half's records (static indexing keeps it in registers)
#pragma unroll
            for (int i = 0; i < C::NSG * (Q + 1); ++i) prm[i] = u ? prm_all[C::NSG * (Q + 1) + i] : prm_all[i];
            float y[MB];
#pragma unroll
            for (int m = 0; m < MB; ++m) y[m] = 0.f;
            if (use_planes) {
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const uint32_t wd[4] = {vec[j].x, vec[j].y, vec[j].z, vec[j].w};
#pragma unroll
                    for (int v = 0; v < C::NSG; ++v) {
                        if constexpr (TQ == 2) {
                            // int8 entries: rows (0,2) / (1,3) / (4,6) / (5,7) accumulate as pairs of 16-bit lanes
                            // (16 look-ups of at most 255 each cannot carry), then each row is un-biased, converted
                            // and scaled by (row scale of the group) x (plane scale)
                            uint32_t ai[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                            for (int ii = 0; ii < C::W; ++ii) {
                                const uint32_t off = prmt(wd[ii >> 2], colp[ii / 3], 0x7704 + 0x10 * (ii & 3) + (ii % 3));
                                const uint2 e = *reinterpret_cast<const uint2*>(smem + off);
                                ai[0] += e.x & 0x00ff00ffu;
                                ai[1] += (e.x >> 8) & 0x00ff00ffu;
                                ai[2] += e.y & 0x00ff00ffu;
                                ai[3] += (e.y >> 8) & 0x00ff00ffu;
                            }
                            const float s = prm[v * (Q + 1) + j];
                            const float* rs = reinterpret_cast<const float*>(smem + C::TABLE_BYTES) + 2 * MB + h * MB;
#pragma unroll
                            for (int m = 0; m < MB; ++m) {
                                const uint32_t word = ai[(m >> 2) * 2 + (m & 1)];
                                const int code_sum = (int)((m & 2) ? (word >> 16) : (word & 0xffffu)) - C::W * 128;
                                y[m] = fmaf(s * rs[m], (float)code_sum, y[m]);
                            }
                            continue;
                        }
                        float2 acc[MB / 2];
#pragma unroll
                        for (int p = 0; p < MB / 2; ++p) acc[p] = make_float2(0.f, 0.f);
#pragma unroll
                        for (int ii = 0; ii < C::W; ++ii) {
                            const int i = v * C::W + ii;
                            // address byte 0 = lane column, byte 1 = weight byte, bytes 2..3 = 0
                            const uint32_t off = prmt(wd[i >> 2], colp[i / 3], 0x7704 + 0x10 * (i & 3) + (i % 3));
                            if (TH) {
                                uint32_t hw[MB / 2];
                                if constexpr (MB == 4) {
                                    const uint2 e = *reinterpret_cast<const uint2*>(smem + off);
                                    hw[0] = e.x; hw[1] = e.y;
                                } else if constexpr (MB == 8) {
                                    const uint4 e = *reinterpret_cast<const uint4*>(smem + 2 * off);
                                    hw[0] = e.x; hw[1] = e.y; hw[2] = e.z; hw[3] = e.w;
                                }
#pragma unroll
                                for (int p = 0; p < MB / 2; ++p)
                                    acc[p] = fadd2(acc[p], __half22float2(*reinterpret_cast<const __half2*>(&hw[p])));
                            } else if (MB == 2) {
                                const float2 e = *reinterpret_cast<const float2*>(smem + off);
                                acc[0] = fadd2(acc[0], e);
                            } else {
                                const float4 e = *reinterpret_cast<const float4*>(smem + 2 * off);
                                acc[0] = fadd2(acc[0], make_float2(e.x, e.y));
                                acc[MB / 2 - 1] = fadd2(acc[MB / 2 - 1], make_float2(e.z, e.w));
                            }
                        }
                        const float s = prm[v * (Q + 1) + j];
#pragma unroll
                        for (int p = 0; p < MB / 2; ++p) {
                            y[2 * p] = fmaf(s, acc[p].x, y[2 * p]);
                            y[2 * p + 1] = fmaf(s, acc[p].y, y[2 * p + 1]);
                        }
                    }
                }
            }
#pragma unroll
            for (int v = 0; v < C::NSG; ++v) {
                const float z = prm[v * (Q + 1) + Q];
#pragma unroll
                for (int m = 0; m < MB; ++m) y[m] = fmaf(z, S[v][m], y[m]);
            }
#pragma unroll
            for (int m = 0; m < MB; ++m) y[m] += __shfl_xor_sync(0xffffffffu, y[m], 16);
            if (h == 0) {
                const int row = rb * kTileRows + l;
#pragma unroll
                for (int m = 0; m < MB; ++m)
                    if (m0 + m < a.M) a.partials[((size_t)kc2 * a.M + (m0 + m)) * n_pad + row] = y[m];
            }
        }
        seg = seg_end;
    }
}

template <int Q, int G, int MB, int TQ = 0>
int launch_mb(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    using C = BCfg<Q, G, MB, TQ>;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(lut_gemm_kernel<Q, G, MB, TQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e != cudaSuccess) return (int)e;
        configured[dev] = true;
    }
    const int n_mb = (a.M + MB - 1) / MB;
    const long long total = (long long)n_mb * 2 * a.n_kc * a.n_rb;
    if (total >= (1LL << 31) - kWarps) return (int)cudaErrorInvalidValue;
    long long grid = (total + kWarps - 1) / kWarps;
    if (grid > num_sms) grid = num_sms;
    if (grid < 1) grid = 1;
    GemmArgs b = a;
    b.items_q = (int)(total / grid);
    b.items_r = (int)(total % grid);
    b.active_warps = kWarps;
    b.ranges = 0; b.rb_q = 0; b.rb_r = 0; b.cpc = 1; b.cluster_reduce = 0;
    // Aligned partition when every (row batch, half chunk) segment can have its own CTAs: a CTA that straddles two
    // segments builds two table sets, which costs more than the slightly uneven ranges.
    const long long n_seg = (long long)n_mb * 2 * a.n_kc;
    if (n_seg <= num_sms) {
        int R = (int)(num_sms / n_seg);
        if (R > a.n_rb) R = a.n_rb;
        if (R >= 1 && n_seg * R * 10 >= (long long)num_sms * 9) {      // only while it still uses >= 90 % of the SMs
            b.ranges = R;
            b.rb_q = a.n_rb / R;
            b.rb_r = a.n_rb % R;
            grid = n_seg * R;
        }
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, lut_gemm_kernel<Q, G, MB, TQ>, b);
    count_launch(1);
    if (e != cudaSuccess) return (int)e;
    return launch_finalize(b, 2 * a.n_kc, cfg.numAttrs != 0, stream);
}

template <int Q, int G>
int launch_qg(const GemmArgs& a, int num_sms, cudaStream_t stream) {
    if (a.flags & ELUTQ_FLAG_TABLE_I8) {
        if constexpr (G == 128) return launch_mb<Q, G, 8, 2>(a, num_sms, stream);
        else return (int)cudaErrorNotSupported;
    }
    if (a.flags & ELUTQ_FLAG_TABLE_F16) {
        if constexpr (G == 128)
            return a.M <= 4 ? launch_mb<Q, G, 4, 1>(a, num_sms, stream) : launch_mb<Q, G, 8, 1>(a, num_sms, stream);
        else
            return (int)cudaErrorNotSupported;
    }
    return a.M == 2 ? launch_mb<Q, G, 2>(a, num_sms, stream) : launch_mb<Q, G, 4>(a, num_sms, stream);
}

template <int Q>
int launch_q(const GemmArgs& a, int G, int num_sms, cudaStream_t stream) {
    switch (G) {
        case 32: return launch_qg<Q, 32>(a, num_sms, stream);
        case 64: return launch_qg<Q, 64>(a, num_sms, stream);
        case 128: return launch_qg<Q, 128>(a, num_sms, stream);
        default: return (int)cudaErrorInvalidValue;
    }
}

}  // namespace

int launch_lut_gemm(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream) {
    if (a.flags & (ELUTQ_FLAG_PLAIN_G4 | ELUTQ_FLAG_CLUSTER_REDUCE | ELUTQ_FLAG_MIRROR)) return (int)cudaErrorNotSupported;   // decode-kernel variants only
    switch (q) {
        case 1: return launch_q<1>(a, G, num_sms, stream);
        case 2: return launch_q<2>(a, G, num_sms, stream);
        case 3: return launch_q<3>(a, G, num_sms, stream);
        case 4: return launch_q<4>(a, G, num_sms, stream);
        default: return (int)cudaErrorInvalidValue;
    }
}

}  // namespace elutq
