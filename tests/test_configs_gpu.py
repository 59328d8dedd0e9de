"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (C-ABI calls on a
stream, library-owned scratch): every shape of configs 0, 1 and 3 at M = 1, and the small-batch sweep's
extremes on one 8B shape, and four calls of the prefill configuration.  The 8B shapes at M = 1 are compared in full against the fp64 oracle; the 70B shapes on
a seeded sample of output rows (first and last tiles plus random rows), which the oracle computes row by row.
"""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import gemm_f16, pack_layer  # noqa: E402

TOL_F16 = 1e-3


def _run(call, seed=0):
    layer = workloads.hlq_layer(seed, call.tag, call.q, call.G, call.N, call.K)
    X = synth.activations(seed, call.tag + "/x", call.M, call.K, outliers=call.outliers)
    packed = pack_layer(layer)
    return layer, X, gemm_f16(X, packed, call.N, call.K)


@pytest.mark.parametrize("call", workloads.config1_calls(), ids=lambda c: f"{c.name}-q{c.q}")
def test_config1_shapes_full_compare(call):
    layer, X, y = _run(call)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, call.G)
    assert np.all(np.isfinite(y))
    assert hlq.rel_fro_error(y, ref) <= TOL_F16
    # element-wise: one fp16 rounding of the exact value plus fp32 accumulation noise
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-3 * np.abs(ref).max() * 2.0 ** -6)


def test_config0_single_gemv():
    call = workloads.config0()[0]
    layer, X, y = _run(call)
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, call.G)
    assert hlq.rel_fro_error(y, ref) <= TOL_F16


@pytest.mark.parametrize("call", [c for c in workloads.config3_calls() if c.q == 2 or c.name in ("o", "down")],
                         ids=lambda c: f"{c.name}-q{c.q}")
def test_config3_shapes_sampled_rows(call):
    layer, X, y = _run(call)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([np.arange(32), np.arange(call.N - 32, call.N),
                                     rng.integers(0, call.N, 1024)]))
    ref = hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
    assert np.all(np.isfinite(y))
    assert hlq.rel_fro_error(y[:, rows], ref) <= TOL_F16


@pytest.mark.parametrize("M", [2, 32])
def test_config2_small_batch_extremes_on_gate_up(M):
    call = [c for c in workloads.config2_calls() if c.name == "gate_up" and c.q == 2 and c.M == M][0]
    layer, X, y = _run(call)
    rng = np.random.default_rng(6)
    rows = np.unique(np.concatenate([np.arange(16), np.arange(call.N - 16, call.N), rng.integers(0, call.N, 2048)]))
    ref = hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
    assert hlq.rel_fro_error(y[:, rows], ref) <= TOL_F16


@pytest.mark.parametrize("name,M", [("gate_up", 2048), ("down", 2048), ("qkv", 512), ("o", 128)])
def test_config4_prefill_shapes_sampled(name, M):
    """The prefill configuration at full size (tensor-core path; CTA pairs for M = 512 and 2048, whole rounds plus
    the K-split tail stripe on gate_up): sampled weight rows x sampled tokens against the oracle."""
    call = [c for c in workloads.config4_prefill_calls() if c.name == name and c.M == M][0]
    layer, X, y = _run(call)
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([np.arange(32), np.arange(call.N - 32, call.N), rng.integers(0, call.N, 1024)]))
    toks = np.unique(np.concatenate([np.arange(8), np.arange(call.M - 8, call.M), rng.integers(0, call.M, 112)]))
    ref = hlq.matmul(X[toks], layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
    got = y[np.ix_(toks, rows)]
    assert np.all(np.isfinite(y))
    assert hlq.rel_fro_error(got, ref) <= TOL_F16
    assert max(hlq.rel_fro_error(got[i], ref[i]) for i in range(len(toks))) <= 2 * TOL_F16
    assert elutq.elutq_device_status() == 0


def test_smoke_entry_runs():
    import __graft_entry__ as g
    g.smoke()
