// M = 1 decode kernel: bit-serial LUT GEMV over HLQ weights (Appendix B procedure, Eq. 3 parameters).
//
// Work decomposition
//   item  = one tile of the packed layout: 16 output rows x 512 input columns (all q planes,
//           their scales and offsets), processed by one warp.
//   CTA   = 32 warps; owns one K chunk over a row range (aligned partition; a contiguous range of the kc-major item
//           list where that balances better), so it needs the activation tables of one K chunk at a time.
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
// K split: one partial sum per K chunk goes to the workspace; a finalize kernel, launched right behind with programmatic
// dependent launch, adds the chunks in ascending order (bit-reproducible) and writes Y.  ELUTQ_FLAG_CLUSTER_REDUCE keeps
// the partial sums in shared memory instead and reduces them across a thread-block cluster.  (The chained entry of
// lut_chain.cu reduces inside its own kernel.)
#include "lut_core.cuh"

namespace elutq {

namespace {

constexpr int kThreads = kGemvThreads;
constexpr int kWarps = kGemvWarps;
constexpr int kSmemBytes = kTableBytes + 128;    // + up to 16 group sums + the reduction flag
constexpr int kClusterPartBytes = 32 * 1024;     // cluster mode: per-CTA partial sums (up to 512 row blocks)
constexpr int kMaxCluster = 8;

// FAST = the common call shape fixed at compile time (both terms, aligned partition with one chunk per CTA, K split
// reduced by the finalize kernel): the flag tests, the segment arithmetic and the other reduction forms drop out
// of the item loop.
template <int Q, int G, int MODE, bool FAST = false>
__global__ void __launch_bounds__(kThreads, 1) lut_gemv_kernel(const GemmArgs a) {
    using C = Cfg<Q, G>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const float* gsum = reinterpret_cast<const float*>(smem + kTableBytes);

    if (!blob_header_matches(a.tiles, Q, G, a.N, a.K, a.counters)) return;   // before any tile is read
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

    uint32_t colp[4];
    make_colp<G>(colp, h, l);

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
        load_group_sums<G>(S, gsum, h, l, use_offset || MODE == kModeMirror);

        float* cpart = reinterpret_cast<float*>(smem + kTableBytes + 128);   // cluster mode: this CTA's partial sums
        const uint8_t* nvp = nullptr;     // next item's plane vectors / parameter words for this lane
        const uint8_t* npp = nullptr;
        auto do_item = [&](auto has_next_c) {
            constexpr bool HAS_NEXT = decltype(has_next_c)::value != 0;
            const float y = item_sum<Q, G, MODE, HAS_NEXT>(buf, smem, colp, S, nvp, npp, use_planes, use_offset);
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
            const bool has_next = nit < nend;
            nvp = a.tiles + (size_t)nit * C::TILE_BYTES + lane * 16;
            npp = nvp + (C::PLANE_BYTES - lane * 12);
            if (has_next) do_item(IntC<1>{});
            else do_item(IntC<0>{});
            it = (nit < nend) ? nit : last;
            it_end = nend;
        }

        seg = (a.ranges > 0) ? seg + a.n_rb : seg_end;
    }

    if (!FAST && a.cluster_reduce) {
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
    }
}

// K-split epilogue: Y[m][n] = sum over the K chunks of partials[chunk][m][n], chunks added in ascending
// order (bit-reproducible), then the output conversion.  One thread per output element.  Launched right
// behind the main kernel with programmatic dependent launch: the grid dependency wait is the only barrier.
__global__ void __launch_bounds__(256) lut_finalize_kernel(const GemmArgs a, const int n_chunks, const int col0, const int cols) {
    grid_launch_dependents();
    grid_dependency_wait();
    if (a.counters != nullptr && __ldcg(a.counters) != 0u) return;   // the main kernel refused the blob: no partial sums, no Y
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
    if (a.counters != nullptr && __ldcg(a.counters) != 0u) return;   // the main kernel refused the blob: no partial sums, no Y
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


bool plan_gemv_partition(int n_rb, int n_kc, int num_sms, bool allow_flat, int* cpc_out, int* ranges_out) {
    // Cost model in item times: the kernel lasts as long as its largest CTA, i.e. that CTA's items
    // plus ~16 item times per table build (measured: an extra build costs far more than the
    // imbalance it could remove).  Minimise that makespan over the aligned choices and the flat one.
    const double kBuild = 16.0;
    const long long total = (long long)n_kc * n_rb;
    const long long flat_grid = total < num_sms ? total : num_sms;
    const long long flat_items = (total + flat_grid - 1) / flat_grid;
    double best = allow_flat ? (double)flat_items + kBuild * (double)((flat_items + n_rb - 1) / n_rb + 1) : 1e300;
    int best_cpc = 0, best_R = 0;
    for (int cpc = 1; cpc <= 8 && cpc <= n_kc; ++cpc) {
        const int groups = (n_kc + cpc - 1) / cpc;
        int R = num_sms / groups;
        // Short kernels (< ~100 items per CTA) run faster in a stream of calls when about 20 SMs stay
        // free for the early-launched CTAs of the kernels that follow (measured: 128 CTAs beat 144 by
        // ~12 % on 20-25 MB layers); long kernels want every SM.
        const int R_spare = (num_sms - 20) / groups;
        if (allow_flat && R_spare >= 1 && (n_rb + R - 1) / R < 100) R = R_spare;
        if (R > n_rb) R = n_rb;
        if (R < 1) continue;
        const double span = (double)cpc * ((double)((n_rb + R - 1) / R) + kBuild);
        if (span < best - 1e-9) { best = span; best_cpc = cpc; best_R = R; }
    }
    if (best_cpc == 0 && !allow_flat) {
        // more chunk groups than SMs even at 8 chunks per CTA: the fewest chunks per CTA that fit one wave
        best_cpc = (n_kc + num_sms - 1) / num_sms;
        best_R = 1;
    }
    *cpc_out = best_cpc;
    *ranges_out = best_R;
    return best_cpc > 0;
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
    if (n_chunks > 8 && outputs < 65536) {
        parts = (n_chunks + 7) / 8;
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
    if (grid < 1) grid = 1;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    GemmArgs b = a;
    b.items_q = (int)(total / grid);
    b.items_r = (int)(total % grid);
    b.ranges = 0; b.rb_q = 0; b.rb_r = 0; b.cpc = 1; b.cluster_reduce = 0;
    b.active_warps = kWarps;   // measured: evening out the rounds (ceil(items / rounds) warps) gains nothing
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    bool use_cluster = false;
    if (a.n_kc >= 2 && a.n_kc <= kMaxCluster && (a.flags & ELUTQ_FLAG_CLUSTER_REDUCE)) {
        // Up to 8 chunks: one cluster per row range, one CTA per chunk, reduction through distributed shared memory.
        int R = (num_sms - 20) / a.n_kc;
        if (R < 1) R = 1;
        if (R > a.n_rb) R = a.n_rb;
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
    if (!use_cluster && a.n_kc > 1) {
        int cpc = 0, R = 0;
        if (plan_gemv_partition(a.n_rb, a.n_kc, num_sms, true, &cpc, &R)) {
            b.cpc = cpc;
            b.ranges = R;
            b.rb_q = a.n_rb / R;
            b.rb_r = a.n_rb % R;
            grid = (long long)R * ((a.n_kc + cpc - 1) / cpc);
            cfg.gridDim = dim3((unsigned)grid);
        }
    }
    const bool fast = MODE == kModeFused && !use_cluster && b.ranges > 0 && b.cpc == 1 && a.n_kc > 1 &&
                      !(b.flags & (ELUTQ_FLAG_SKIP_OFFSET | ELUTQ_FLAG_OFFSET_ONLY));
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
    if (e != cudaSuccess || a.n_kc == 1 || b.cluster_reduce) return (int)e;
    return launch_finalize(b, a.n_kc, true, stream);
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
