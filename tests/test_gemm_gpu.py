"""GPU parity of the batched (M > 1) path against the fp64 oracle, through the C ABI."""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_elementwise, gemm_f16, gemm_f32, pack_layer, x_dev  # noqa: E402

TOL_F32 = 5e-6
TOL_F16 = 1e-3

# (q, G, N, K, M): row batches of 2 and 4 with ragged remainders, every q and G, ragged N and K tails,
# a single-chunk K, and the sweep's largest small batch with outlier activations
CASES = [(2, 128, 200, 1024, 5), (3, 128, 333, 1536, 2), (4, 64, 50, 1088, 4), (1, 32, 17, 96, 3),
         (2, 128, 64, 512, 7), (3, 64, 1000, 4096, 16), (2, 128, 1000, 4096, 32), (4, 128, 48, 2560, 9)]


@pytest.mark.parametrize("q,G,N,K,M", CASES)
def test_batched_gemm_matches_oracle(q, G, N, K, M):
    layer = workloads.hlq_layer(20, f"gemm/{q}/{G}/{N}/{K}", q, G, N, K, signed_scales=(q % 2 == 0))
    X = synth.activations(20, f"gemm/x/{M}/{K}", M, K, outliers=True)
    packed = pack_layer(layer)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    y32 = gemm_f32(X, packed, N, K, elutq.FLAG_LUT_ONLY)           # the look-up kernels at every M
    assert np.all(np.isfinite(y32))
    assert hlq.rel_fro_error(y32, ref) <= TOL_F32
    for m in range(M):                                   # every activation row on its own, too
        assert hlq.rel_fro_error(y32[m], ref[m]) <= 2 * TOL_F32
    A = hlq.magnitude_bound(X, layer.scales, layer.offsets, G)
    assert_elementwise(y32, ref, A, q, K, False, False, "batched look-up kernel, fp32 out")
    y16 = gemm_f16(X, packed, N, K)                                # default path
    assert hlq.rel_fro_error(y16, ref) <= TOL_F16
    tensor_path = elutq.elutq_takes_tensor_path(M, N, K, G)
    assert_elementwise(y16, ref, A, q, K, tensor_path, True, "default path, fp16 out")
    if not tensor_path:                                  # on the look-up kernels by default: the same kernels
        assert np.array_equal(y16.view(np.uint16), y32.astype(np.float16).view(np.uint16))


def test_batched_rows_equal_single_row_calls_up_to_rounding():
    q, G, N, K, M = 2, 128, 333, 1536, 6
    layer = workloads.hlq_layer(21, "gemm/rows", q, G, N, K)
    X = synth.activations(21, "gemm/rows/x", M, K)
    packed = pack_layer(layer)
    yb = gemm_f32(X, packed, N, K, elutq.FLAG_LUT_ONLY)            # (a narrow layer at M = 6 would take the tensor cores by default)
    for m in range(M):
        y1 = gemm_f32(X[m:m + 1], packed, N, K)
        np.testing.assert_allclose(yb[m], y1[0], rtol=0, atol=4e-6 * np.abs(y1).max())


def test_batched_offset_scale_and_accumulate_flags():
    q, G, N, K, M = 3, 64, 100, 1088, 4
    layer = workloads.hlq_layer(22, "gemm/flags", q, G, N, K)
    X = synth.activations(22, "gemm/flags/x", M, K)
    packed = pack_layer(layer)
    ys = gemm_f32(X, packed, N, K, elutq.FLAG_SKIP_OFFSET)
    yb = gemm_f32(X, packed, N, K, elutq.FLAG_OFFSET_ONLY)
    yf = gemm_f32(X, packed, N, K)
    assert hlq.rel_fro_error(ys, hlq.scale_term(X, layer.planes, layer.scales, G)) <= TOL_F32
    assert hlq.rel_fro_error(yb, hlq.offset_term(X, layer.offsets, G)) <= TOL_F32
    np.testing.assert_allclose(ys + yb, yf, rtol=0, atol=4e-6 * np.abs(yf).max())
    Y = torch.full((M, N), 2.0, dtype=torch.float32, device="cuda")
    elutq.elutq_lut_gemm_f32(x_dev(X), packed, Y, M, N, K, elutq.FLAG_ACCUMULATE)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(Y.cpu().numpy(), yf + np.float32(2.0))
    Yb = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm_bias(x_dev(X), packed, Yb, M, N, K)
    torch.cuda.synchronize()
    assert hlq.rel_fro_error(Yb.cpu().numpy(), hlq.offset_term(X, layer.offsets, G)) <= TOL_F16


def test_prefill_sized_batch_on_a_layer_sized_matrix():
    # M = 128 rows on the 8B attention-output shape (config 4a's smallest), compared in full
    q, G, N, K, M = 2, 128, 4096, 4096, 128
    layer = workloads.hlq_layer(0, f"o/q{q}/G{G}/{N}x{K}", q, G, N, K)
    X = synth.activations(23, "prefill/x", M, K)
    packed = pack_layer(layer)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    A = hlq.magnitude_bound(X, layer.scales, layer.offsets, G)
    y16 = gemm_f16(X, packed, N, K)                                  # default path for M >= 9: tensor cores
    assert hlq.rel_fro_error(y16, ref) <= TOL_F16
    assert_elementwise(y16, ref, A, q, K, True, True, "tensor-core path, fp16 out")
    y32 = gemm_f32(X, packed, N, K, elutq.FLAG_LUT_ONLY)           # look-up-table kernels
    assert hlq.rel_fro_error(y32, ref) <= TOL_F32
    assert_elementwise(y32, ref, A, q, K, False, False, "look-up kernels, fp32 out")


def test_workspace_entry_and_reproducibility_for_batches():
    q, G, N, K, M = 2, 128, 500, 2048, 8
    layer = workloads.hlq_layer(24, "gemm/ws", q, G, N, K)
    X = synth.activations(24, "gemm/ws/x", M, K)
    packed = pack_layer(layer)
    a = gemm_f16(X, packed, N, K)
    b = gemm_f16(X, packed, N, K)
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    ws = torch.empty(elutq.elutq_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    elutq.elutq_workspace_init(ws)
    Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm_ws(x_dev(X), packed, Y, M, N, K, 0, ws)
    torch.cuda.synchronize()
    assert np.array_equal(Y.cpu().numpy().view(np.uint16), a.view(np.uint16))
