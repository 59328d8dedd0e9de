"""GPU parity of elutq_hlq_fit (Algorithm 1) against the fp64 oracle: planes and fp16 parameters bit for bit."""
import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import fit as ofit
from oracle import hlq
from tests.gpu_util import gemm_f32, to_dev

pytestmark = pytest.mark.gpu


def _fit_gpu(W, q, G, t_max=10, trace=False):
    Wd = to_dev(W.view(np.int16)).view(torch.float16)
    out = elutq.elutq_hlq_fit(Wd, q, G, t_max, trace)
    torch.cuda.synchronize()
    planes = out[0].cpu().numpy()
    scales = out[1].cpu().view(torch.int16).numpy().view(np.float16)
    offsets = out[2].cpu().view(torch.int16).numpy().view(np.float16)
    if trace:
        return planes, scales, offsets, out[3].cpu().numpy()
    return planes, scales, offsets


def _same_bits(a, b):
    return np.array_equal(np.ascontiguousarray(a).view(np.uint16), np.ascontiguousarray(b).view(np.uint16))


@pytest.mark.parametrize("q", [1, 2, 3, 4])
@pytest.mark.parametrize("G", [32, 64, 128])
def test_fit_matches_oracle_bit_for_bit(q, G):
    N, K = 37, 1024                       # 37 rows: the last CTA of 8 groups is ragged for every G
    W = workloads.dense_weights(23, f"fit{q}{G}", N, K)
    p_ref, s_ref, z_ref, tr_ref = ofit.fit(W, q, G, 10, trace=True)
    p, s, z, tr = _fit_gpu(W, q, G, 10, trace=True)
    assert np.array_equal(p, p_ref)
    assert _same_bits(s, s_ref) and _same_bits(z, z_ref)
    assert np.allclose(tr, tr_ref, rtol=1e-10, atol=1e-20)
    assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-12) + 1e-18)


@pytest.mark.parametrize("t_max", [1, 3])
def test_fit_short_runs(t_max):
    W = workloads.dense_weights(29, "fit-short", 16, 512)
    p_ref, s_ref, z_ref = ofit.fit(W, 3, 128, t_max)
    p, s, z = _fit_gpu(W, 3, 128, t_max)
    assert np.array_equal(p, p_ref) and _same_bits(s, s_ref) and _same_bits(z, z_ref)


def test_fit_degenerate_groups():
    """Constant groups (singular from the first round), two-valued groups (higher planes dependent), grid weights."""
    q, G = 3, 32
    rng = np.random.default_rng(4)
    W = workloads.dense_weights(31, "fit-deg", 8, 256)
    W[0, :32] = np.float16(0.0625)                                            # constant
    W[1, 32:64] = np.where(rng.integers(0, 2, 32) == 1, np.float16(0.5), np.float16(-0.25))   # two values
    c = rng.integers(0, 8, 32)
    c[:8] = np.arange(8)
    W[2, 64:96] = (-0.125 + 2.0 ** -6 * c).astype(np.float16)                 # exactly on a uniform grid
    p_ref, s_ref, z_ref = ofit.fit(W, q, G, 10)
    p, s, z = _fit_gpu(W, q, G, 10)
    assert np.array_equal(p, p_ref) and _same_bits(s, s_ref) and _same_bits(z, z_ref)
    rec = hlq.reconstruct(p, s, z, G)
    assert np.array_equal(rec[0, :32], W[0, :32].astype(np.float64))
    assert np.allclose(rec[1, 32:64], W[1, 32:64].astype(np.float64), atol=1e-3)
    assert np.allclose(rec[2, 64:96], W[2, 64:96].astype(np.float64), atol=2e-4)


def test_fit_then_pack_then_product():
    """The offline chain on the device: fit -> pack -> GEMV equals the oracle product of the oracle's fit."""
    q, G, N, K = 2, 128, 64, 1024
    W = workloads.dense_weights(37, "fit-chain", N, K)
    Wd = to_dev(W.view(np.int16)).view(torch.float16)
    planes, scales, offsets = elutq.elutq_hlq_fit(Wd, q, G)
    packed = elutq.elutq_pack(planes, scales, offsets, q, G, N, K)
    X = workloads.activations(37, "fit-chain", 1, K)
    Y = gemm_f32(X, packed, N, K)
    p_ref, s_ref, z_ref = ofit.fit(W, q, G)
    Y_ref = hlq.matmul(X, p_ref, s_ref, z_ref, G)
    assert hlq.rel_fro_error(Y, Y_ref) <= 5e-6
    # and the fitted layer approximates the dense product far better than its energy
    Y_dense = X.astype(np.float64) @ W.astype(np.float64).T
    assert hlq.rel_fro_error(Y_ref, Y_dense) < 0.5
