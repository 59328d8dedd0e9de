// M > 1: small-batch / prefill LUT GEMM.
#include "common.cuh"

namespace elutq {

int launch_lut_gemm(const GemmArgs& a, int q, int G, int num_sms, cudaStream_t stream) {
    // Row-at-a-time: every activation row runs the decode kernel (correct for any M).
    const size_t ybytes = (a.flags & ELUTQ_FLAG_OUT_F32) ? sizeof(float) : sizeof(__half);
    for (int m = 0; m < a.M; ++m) {
        GemmArgs r = a;
        r.M = 1;
        r.X = a.X + (size_t)m * a.K;
        r.Y = reinterpret_cast<uint8_t*>(a.Y) + (size_t)m * a.N * ybytes;
        int e = launch_lut_gemv(r, q, G, num_sms, stream);
        if (e != 0) return e;
    }
    return 0;
}

}  // namespace elutq
