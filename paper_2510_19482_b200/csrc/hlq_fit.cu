// Algorithm 1 on the GPU: alternating bit-pattern selection and least squares, one warp per weight group.
//
// The step before the hot path: it turns unquantised fp16 weights into the (B, s, z) that elutq_pack
// consumes.  Groups are independent, so a warp owns one group of G weights (G / 32 per lane) and keeps
// everything in registers:
//
//   initialisation   Delta = (max - min) / (2^q - 1), s = [Delta, 2 Delta, ...], z = min   (warp min / max)
//   selection        every lane evaluates the 2^q candidate values for its weights, first minimum wins
//   normal equations the matrix [B 1]^T [B 1] holds bit counts: ballots + popcounts, exact integers; the
//                    right-hand side sums weights in units of 2^-24 (every fp16 value is such an integer)
//                    in 64-bit integers, so the result does not depend on the reduction order
//   singular?        decided exactly by fraction-free elimination on the integer matrix; a singular system
//                    (a plane constant over the group, two equal planes) keeps the previous parameters
//   solve            elimination without pivoting and back substitution in fp64, one rounding per operation
//                    (explicit round-to-nearest intrinsics, no fused multiply-add), done redundantly by
//                    every lane
//
// All arithmetic that decides a bit is fp64 in a fixed order, so the selected planes and the fp16
// parameters are reproducible bit for bit.
#include "common.cuh"

namespace elutq {

namespace {

constexpr int kFitWarps = 8;      // warps (groups) per CTA

__device__ __forceinline__ long long warp_sum_ll(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <int Q, int EPL>
__global__ void __launch_bounds__(kFitWarps * 32) hlq_fit_kernel(const __half* __restrict__ W, int N, int K, int t_max,
                                                                 uint8_t* __restrict__ planes, __half* __restrict__ scales,
                                                                 __half* __restrict__ offsets, double* __restrict__ trace) {
    constexpr int G = 32 * EPL, NC = 1 << Q, NV = Q + 1;
    const int lane = threadIdx.x & 31;
    const long long n_groups = (long long)N * (K / G);
    const long long grp = (long long)blockIdx.x * kFitWarps + (threadIdx.x >> 5);
    if (grp >= n_groups) return;
    const int n = (int)(grp / (K / G)), kg = (int)(grp % (K / G));
    const size_t base = (size_t)n * K + (size_t)kg * G;

    double w[EPL];
    long long wfix[EPL];
    double wmax, wmin;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        w[e] = (double)__half2float(W[base + lane + 32 * e]);
        wfix[e] = (long long)(w[e] * 16777216.0);          // exact: fp16 values are multiples of 2^-24
    }
    wmax = w[0];
    wmin = w[0];
#pragma unroll
    for (int e = 1; e < EPL; ++e) {
        wmax = fmax(wmax, w[e]);
        wmin = fmin(wmin, w[e]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        wmax = fmax(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
        wmin = fmin(wmin, __shfl_xor_sync(0xffffffffu, wmin, o));
    }

    double s[Q], z = wmin;
    const double delta = __ddiv_rn(__dsub_rn(wmax, wmin), (double)(NC - 1));
#pragma unroll
    for (int j = 0; j < Q; ++j) s[j] = delta * (double)(1 << j);      // exact scaling

    int code[EPL];
    auto select = [&]() {
        double V[NC];
#pragma unroll
        for (int k = 0; k < NC; ++k) {
            double v = 0.0;
#pragma unroll
            for (int j = 0; j < Q; ++j)
                if ((k >> j) & 1) v = __dadd_rn(v, s[j]);
            V[k] = v;
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const double shifted = __dsub_rn(w[e], z);
            int best = 0;
            double bd = fabs(__dsub_rn(shifted, V[0]));
#pragma unroll
            for (int k = 1; k < NC; ++k) {
                const double d = fabs(__dsub_rn(shifted, V[k]));
                if (d < bd) { bd = d; best = k; }
            }
            code[e] = best;
        }
    };
    auto group_sse = [&]() {
        double acc = 0.0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            double rec = z;
#pragma unroll
            for (int j = 0; j < Q; ++j)
                if ((code[e] >> j) & 1) rec = __dadd_rn(rec, s[j]);
            const double d = __dsub_rn(w[e], rec);
            acc = __dadd_rn(acc, __dmul_rn(d, d));
        }
        return warp_sum_d(acc);
    };

    if (trace != nullptr) {
        select();
        const double e0 = group_sse();
        if (lane == 0) trace[grp] = e0;
    }

    for (int t = 1; t <= t_max; ++t) {
        select();

        // ---- normal equations: bit counts (exact) and fixed-point weight sums (exact) -----------------
        long long A[NV][NV];
        {
            unsigned mask[Q][EPL];
#pragma unroll
            for (int j = 0; j < Q; ++j)
#pragma unroll
                for (int e = 0; e < EPL; ++e) mask[j][e] = __ballot_sync(0xffffffffu, (code[e] >> j) & 1);
#pragma unroll
            for (int i = 0; i < Q; ++i) {
#pragma unroll
                for (int j = i; j < Q; ++j) {
                    int c = 0;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) c += __popc(mask[i][e] & mask[j][e]);
                    A[i][j] = c;
                    A[j][i] = c;
                }
                int c = 0;
#pragma unroll
                for (int e = 0; e < EPL; ++e) c += __popc(mask[i][e]);
                A[i][Q] = c;
                A[Q][i] = c;
            }
            A[Q][Q] = G;
        }
        double r[NV];
        {
            long long all = 0;
#pragma unroll
            for (int e = 0; e < EPL; ++e) all += wfix[e];
            r[Q] = __ll2double_rn(warp_sum_ll(all)) / 16777216.0;
#pragma unroll
            for (int j = 0; j < Q; ++j) {
                long long part = 0;
#pragma unroll
                for (int e = 0; e < EPL; ++e) part += ((code[e] >> j) & 1) ? wfix[e] : 0;
                r[j] = __ll2double_rn(warp_sum_ll(part)) / 16777216.0;
            }
        }

        // ---- exact singularity test: fraction-free elimination, a zero pivot means a singular system -----
        bool singular = false;
        {
            long long m[NV][NV];
#pragma unroll
            for (int i = 0; i < NV; ++i)
#pragma unroll
                for (int j = 0; j < NV; ++j) m[i][j] = A[i][j];
            // The divisions are exact and the quotients (minors of a Gram matrix of 0/1 vectors of length <= 128)
            // stay below 128^5 < 2^36, so rounding numerator * (1 / prev) in fp64 (relative error < 2^-50)
            // returns the exact integer; the numerators stay below 2^57.
            double inv_prev = 1.0;
#pragma unroll
            for (int c = 0; c < NV; ++c) {
                singular = singular || (m[c][c] == 0);
                const long long piv = singular ? 1 : m[c][c];
#pragma unroll
                for (int i = c + 1; i < NV; ++i)
#pragma unroll
                    for (int j = c + 1; j < NV; ++j)
                        m[i][j] = __double2ll_rn(__ll2double_rn(m[i][j] * piv - m[i][c] * m[c][j]) * inv_prev);
                inv_prev = 1.0 / (double)piv;
            }
        }

        // ---- solve (fp64, elimination without pivoting, one rounding per operation) ------------------------
        if (!singular) {
            double a[NV][NV], b[NV], x[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                b[i] = r[i];
#pragma unroll
                for (int j = 0; j < NV; ++j) a[i][j] = (double)A[i][j];
            }
#pragma unroll
            for (int c = 0; c < NV; ++c) {
#pragma unroll
                for (int i = c + 1; i < NV; ++i) {
                    const double f = __ddiv_rn(a[i][c], a[c][c]);
#pragma unroll
                    for (int j = c + 1; j < NV; ++j) a[i][j] = __dsub_rn(a[i][j], __dmul_rn(f, a[c][j]));
                    b[i] = __dsub_rn(b[i], __dmul_rn(f, b[c]));
                }
            }
#pragma unroll
            for (int i = NV - 1; i >= 0; --i) {
                double acc = b[i];
#pragma unroll
                for (int j = i + 1; j < NV; ++j) acc = __dsub_rn(acc, __dmul_rn(a[i][j], x[j]));
                x[i] = __ddiv_rn(acc, a[i][i]);
            }
#pragma unroll
            for (int j = 0; j < Q; ++j) s[j] = x[j];
            z = x[Q];
        }
        if (trace != nullptr) {
            const double et = group_sse();
            if (lane == 0) trace[(size_t)t * n_groups + grp] = et;
        }
    }

    // ---- results: one byte per bit (the input format of elutq_pack), fp16 parameters ----------------------
#pragma unroll
    for (int j = 0; j < Q; ++j)
#pragma unroll
        for (int e = 0; e < EPL; ++e) planes[(size_t)j * N * K + base + lane + 32 * e] = (uint8_t)((code[e] >> j) & 1);
    if (lane < Q) {
        double v = s[0];
#pragma unroll
        for (int j = 1; j < Q; ++j) v = (lane == j) ? s[j] : v;
        scales[(size_t)grp * Q + lane] = __double2half(v);
    }
    if (lane == Q) offsets[grp] = __double2half(z);
}

template <int Q>
int launch_fit_q(const __half* W, int G, int N, int K, int t_max, uint8_t* planes, __half* scales, __half* offsets,
                 double* trace, cudaStream_t stream) {
    const long long n_groups = (long long)N * (K / G);
    const unsigned grid = (unsigned)((n_groups + kFitWarps - 1) / kFitWarps);
    switch (G) {
        case 32: hlq_fit_kernel<Q, 1><<<grid, kFitWarps * 32, 0, stream>>>(W, N, K, t_max, planes, scales, offsets, trace); break;
        case 64: hlq_fit_kernel<Q, 2><<<grid, kFitWarps * 32, 0, stream>>>(W, N, K, t_max, planes, scales, offsets, trace); break;
        case 128: hlq_fit_kernel<Q, 4><<<grid, kFitWarps * 32, 0, stream>>>(W, N, K, t_max, planes, scales, offsets, trace); break;
        default: return (int)cudaErrorInvalidValue;
    }
    count_launch(1);
    return (int)cudaGetLastError();
}

}  // namespace

}  // namespace elutq

using namespace elutq;

extern "C" int elutq_hlq_fit(const void* W, int q, int G, int N, int K, int t_max, uint8_t* planes, void* scales,
                             void* offsets, double* err_trace, void* stream) {
    if (!W || !planes || !scales || !offsets) return ELUTQ_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0 || t_max < 1 || t_max > 1000) return ELUTQ_ERR_INVALID_ARG;
    if (q < 1 || q > 4 || (G != 32 && G != 64 && G != 128) || K % G != 0) return ELUTQ_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(W) & 1) || (reinterpret_cast<uintptr_t>(scales) & 1) ||
        (reinterpret_cast<uintptr_t>(offsets) & 1) || (reinterpret_cast<uintptr_t>(err_trace) & 7))
        return ELUTQ_ERR_ALIGN;
    const __half* w = reinterpret_cast<const __half*>(W);
    __half* s = reinterpret_cast<__half*>(scales);
    __half* z = reinterpret_cast<__half*>(offsets);
    cudaStream_t st = (cudaStream_t)stream;
    int ce;
    switch (q) {
        case 1: ce = launch_fit_q<1>(w, G, N, K, t_max, planes, s, z, err_trace, st); break;
        case 2: ce = launch_fit_q<2>(w, G, N, K, t_max, planes, s, z, err_trace, st); break;
        case 3: ce = launch_fit_q<3>(w, G, N, K, t_max, planes, s, z, err_trace, st); break;
        default: ce = launch_fit_q<4>(w, G, N, K, t_max, planes, s, z, err_trace, st); break;
    }
    if (ce != 0) {
        note_cuda_error(ce);
        return ELUTQ_ERR_CUDA;
    }
    return ELUTQ_OK;
}
