"""Seeded sweep over odd shapes through every dispatch path (decode, batched look-up, tensor cores) against the
fp64 oracle: ragged N, K that is not a multiple of 512, M on both sides of each threshold, every q and G."""
import numpy as np
import pytest

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_elementwise, gemm_f16, gemm_f32, pack_layer  # noqa: E402


def _cases():
    rng = np.random.default_rng(20251019)
    out = []
    for i in range(48):
        q = int(rng.integers(1, 5))
        G = int(rng.choice([32, 64, 128]))
        K = G * int(rng.integers(1, 2048 // G + 1))
        N = int(rng.choice([1, 7, 16, 17, 100, 255, 256, 257, 300, 513, 777]))
        M = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 10, 15, 16, 17, 31, 33, 64, 127, 128, 129, 200, 257]))
        out.append((i, q, G, N, K, M))
    return out


@pytest.mark.parametrize("i,q,G,N,K,M", _cases())
def test_random_shape(i, q, G, N, K, M):
    layer = workloads.hlq_layer(50 + i, f"rand/{i}", q, G, N, K, signed_scales=(i % 3 == 0))
    X = synth.activations(50 + i, f"rand/x/{i}", M, K, outliers=(i % 4 == 0))
    packed = pack_layer(layer)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    tensor_path = elutq.elutq_takes_tensor_path(M, N, K, G)
    y32 = gemm_f32(X, packed, N, K)
    assert np.all(np.isfinite(y32))
    assert hlq.rel_fro_error(y32, ref) <= (1e-3 if tensor_path else 5e-6)
    A = hlq.magnitude_bound(X, layer.scales, layer.offsets, G)
    assert_elementwise(y32, ref, A, q, K, tensor_path, False, "default path, fp32 out")
    y16 = gemm_f16(X, packed, N, K)
    assert hlq.rel_fro_error(y16, ref) <= 1e-3
    assert_elementwise(y16, ref, A, q, K, tensor_path, True, "default path, fp16 out")
    if tensor_path:
        ylut = gemm_f32(X, packed, N, K, elutq.FLAG_LUT_ONLY)
        assert hlq.rel_fro_error(ylut, ref) <= 5e-6
        assert_elementwise(ylut, ref, A, q, K, False, False, "look-up kernels, fp32 out")
    assert elutq.elutq_device_status() == 0


def _prefill_cases():
    rng = np.random.default_rng(20251020)
    out = []
    for i in range(20):
        q = int(rng.integers(1, 5))
        K = 128 * int(rng.integers(1, 25))
        N = int(rng.choice([2048, 3000, 4096, 5000, 8192]))
        M = int(rng.choice([257, 300, 512, 513, 700, 1000, 1024, 1500, 2048]))
        out.append((i, q, N, K, M))
    return out


@pytest.mark.parametrize("i,q,N,K,M", _prefill_cases())
def test_random_prefill_shape(i, q, N, K, M):
    """Prefill-sized batches at G = 128: several token tiles per weight tile (CTA pairs when their number is even),
    K splits, tail stripes, ragged N / M / K."""
    G = 128
    layer = workloads.hlq_layer(80 + i, f"randp/{i}", q, G, N, K, signed_scales=(i % 3 == 0))
    X = synth.activations(80 + i, f"randp/x/{i}", M, K, outliers=(i % 4 == 0))
    packed = pack_layer(layer)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
    y16 = gemm_f16(X, packed, N, K)
    assert np.all(np.isfinite(y16))
    assert hlq.rel_fro_error(y16, ref) <= 1e-3
    assert max(hlq.rel_fro_error(y16[m], ref[m]) for m in range(M)) <= 2e-3
    assert_elementwise(y16, ref, hlq.magnitude_bound(X, layer.scales, layer.offsets, G), q, K, True, True,
                       "tensor-core path, fp16 out")
    assert elutq.elutq_device_status() == 0
