"""GPU parity of the tensor-core (dequantise-and-contract) path for batches of 9 rows or more.

Tolerance: the path rebuilds W_hat in fp16 in the BCQ form (z^ = z + (1/2) sum_j s_j formed in fp32 and rounded
once; per plane the sign bit of the packed -s_j/2 is flipped by an integer operation and one packed fp16 add
accumulates it, each add rounding at 2^-11 relative), multiplies exactly and accumulates in fp32.  The weight
rounding errors are independent across k, so the relative Frobenius error of Y is about 2^-12..2^-11
(2.5e-4 .. 5e-4) before the output rounding; the bar is the benchmark's 1e-3.  Every element is also held to
the worst-case bound of gpu_util.assert_elementwise.
"""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_elementwise, gemm_f16, gemm_f32, pack_layer, x_dev  # noqa: E402

TOL = 1e-3

# (q, N, K, M): one tile, ragged N / M / K tails, every q, several token tiles, a K split
CASES = [(2, 300, 1024, 9), (2, 512, 1024, 16), (3, 300, 1536, 40), (2, 256, 512, 64), (2, 200, 1024, 100), (3, 1000, 1536, 128), (4, 384, 2560, 300),
         (1, 130, 640, 65), (2, 4096, 4096, 128), (3, 512, 4096, 700),
         (2, 4096, 512, 2560),      # 160 tiles: whole rounds plus a K-split tail stripe
         # an even number of 256-token tiles and enough weight tiles: the shapes a CTA pair would take
         (2, 4096, 1024, 512), (3, 4000, 1024, 500), (4, 8192, 1024, 300), (1, 4096, 1536, 1024),
         (2, 8192, 640, 512), (3, 20000, 128, 512)]      # the same with K ending inside a 512-column chunk / a single K step


@pytest.mark.parametrize("q,N,K,M", CASES)
def test_tensor_core_path_matches_oracle(q, N, K, M):
    G = 128
    layer = workloads.hlq_layer(30, f"mma/{q}/{N}/{K}", q, G, N, K, signed_scales=(q == 3))
    X = synth.activations(30, f"mma/x/{M}/{K}", M, K, outliers=(q == 2))
    packed = pack_layer(layer)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    y32 = gemm_f32(X, packed, N, K)
    assert elutq.elutq_device_status() == 0
    assert np.all(np.isfinite(y32))
    assert hlq.rel_fro_error(y32, ref) <= TOL
    worst_row = max(hlq.rel_fro_error(y32[m], ref[m]) for m in range(M))
    assert worst_row <= 2 * TOL
    A = hlq.magnitude_bound(X, layer.scales, layer.offsets, G)
    assert_elementwise(y32, ref, A, q, K, True, False, "tensor-core path, fp32 out")
    y16 = gemm_f16(X, packed, N, K)
    assert hlq.rel_fro_error(y16, ref) <= TOL
    assert_elementwise(y16, ref, A, q, K, True, True, "tensor-core path, fp16 out")
    # the look-up-table kernels on the same batch agree with it within the same bar
    ylut = gemm_f32(X, packed, N, K, elutq.FLAG_LUT_ONLY)
    assert hlq.rel_fro_error(ylut, ref) <= 5e-6
    assert_elementwise(ylut, ref, A, q, K, False, False, "look-up kernels, fp32 out")
    assert hlq.rel_fro_error(y32, ylut) <= TOL


@pytest.mark.parametrize("N,K,M", [(300, 1024, 96), (4096, 1024, 512)])     # one token tile; CTA pairs
def test_tensor_core_path_terms_and_accumulate(N, K, M):
    q, G = 2, 128
    layer = workloads.hlq_layer(31, f"mma/flags/{N}", q, G, N, K)
    X = synth.activations(31, f"mma/flags/x/{M}", M, K)
    packed = pack_layer(layer)
    ys = gemm_f32(X, packed, N, K, elutq.FLAG_SKIP_OFFSET)
    yb = gemm_f32(X, packed, N, K, elutq.FLAG_OFFSET_ONLY)
    yf = gemm_f32(X, packed, N, K)
    assert hlq.rel_fro_error(ys, hlq.scale_term(X, layer.planes, layer.scales, G)) <= TOL
    assert hlq.rel_fro_error(yb, hlq.offset_term(X, layer.offsets, G)) <= TOL
    assert hlq.rel_fro_error(yf, hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)) <= TOL
    Y = torch.full((M, N), 1.5, dtype=torch.float32, device="cuda")
    elutq.elutq_lut_gemm_f32(x_dev(X), packed, Y, M, N, K, elutq.FLAG_ACCUMULATE)
    torch.cuda.synchronize()
    np.testing.assert_allclose(Y.cpu().numpy(), yf + 1.5, rtol=0, atol=1e-5 * np.abs(yf).max())
    assert elutq.elutq_device_status() == 0


@pytest.mark.parametrize("q,N,K,M", [(3, 512, 2048, 128), (2, 4096, 2048, 512), (4, 8192, 1024, 1000)])
def test_tensor_core_path_is_bit_reproducible(q, N, K, M):
    """One token tile, and the shapes that run as CTA pairs (hand-over through barriers across two SMs): repeated
    calls give identical bits, so no half of a weight or activation tile is read before it is complete."""
    G = 128
    layer = workloads.hlq_layer(32, f"mma/repro/{q}/{N}", q, G, N, K)
    X = synth.activations(32, f"mma/repro/x/{M}/{K}", M, K)
    packed = pack_layer(layer)
    a = gemm_f16(X, packed, N, K)
    for _ in range(5):
        b = gemm_f16(X, packed, N, K)
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    assert elutq.elutq_device_status() == 0


def test_a_wait_for_mma_completion_that_runs_out_is_reported_and_the_stream_stays_usable():
    # The test entry launches the one-token-tile kernel with its issuing thread told to issue nothing and the poll
    # limit at 4096: every thread's wait for the MMAs of two steps ago runs out, the kernel stops waiting, joins its
    # barriers, frees its tensor memory and returns; the status word says so.  The next ordinary call on the same
    # stream is correct.
    q, G, N, K, M = 2, 128, 512, 2048, 64
    layer = workloads.hlq_layer(33, "mma/expiry", q, G, N, K)
    X = synth.activations(33, "mma/expiry/x", M, K)
    packed = pack_layer(layer)
    elutq.elutq_release_scratch()
    Y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    elutq.elutq_test_wait_expiry(x_dev(X), packed, Y, M, N, K, 4096)
    assert elutq.elutq_device_status() == 0x7C05
    elutq.elutq_release_scratch()
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    y = gemm_f32(X, packed, N, K)
    assert elutq.elutq_device_status() == 0
    assert hlq.rel_fro_error(y, ref) <= TOL
