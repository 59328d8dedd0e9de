"""Parity at the benchmark's full sizes, in the launch configurations bench.py times (C-ABI calls on a stream with
library-owned scratch, and the chained decode entry): every call of configs 0, 1, 2, 3 and 4a, the whole config-1 and config-3 steps as one plan each, and two layers of the
32-layer stack of config 4b with their own seeds.  The 8B shapes at M = 1 are compared in full against the fp64
oracle; the larger problems on a seeded sample of output rows (first and last tiles plus random rows) x all tokens,
which the oracle computes row by row.  Every comparison is a relative Frobenius error AND an element-wise bound.
"""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_elementwise, gemm_f16, pack_layer, x_dev  # noqa: E402

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


def _sample_rows(N, n_random, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([np.arange(min(32, N)), np.arange(max(0, N - 32), N), rng.integers(0, N, n_random)]))


@pytest.mark.parametrize("call", workloads.config3_calls(), ids=lambda c: f"{c.name}-q{c.q}")
def test_config3_shapes_sampled_rows(call):
    layer, X, y = _run(call)
    rows = _sample_rows(call.N, 1024, 5)
    ref = hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
    assert np.all(np.isfinite(y))
    assert hlq.rel_fro_error(y[:, rows], ref) <= TOL_F16
    A = hlq.magnitude_bound(X, layer.scales[rows], layer.offsets[rows], call.G)
    assert_elementwise(y[:, rows], ref, A, call.q, call.K, False, True, f"config 3 {call.name} q{call.q}")


_CFG2 = workloads.config2_calls()


@pytest.mark.parametrize("name,q", sorted({(c.name, c.q) for c in _CFG2}))
def test_config2_every_call_of_the_small_batch_sweep(name, q):
    """All six batch sizes of the sweep on one (layer, q): sampled weight rows x all tokens, norm and element-wise."""
    calls = [c for c in _CFG2 if c.name == name and c.q == q]
    c0 = calls[0]
    layer = workloads.hlq_layer(0, c0.tag, c0.q, c0.G, c0.N, c0.K)
    packed = pack_layer(layer)
    rows = _sample_rows(c0.N, 1024, 6)
    for call in calls:
        X = synth.activations(0, call.tag + f"/x{call.M}", call.M, call.K, outliers=True)
        y = gemm_f16(X, packed, call.N, call.K)
        ref = hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
        assert np.all(np.isfinite(y))
        assert hlq.rel_fro_error(y[:, rows], ref) <= TOL_F16, call
        A = hlq.magnitude_bound(X, layer.scales[rows], layer.offsets[rows], call.G)
        assert_elementwise(y[:, rows], ref, A, call.q, call.K, elutq.elutq_takes_tensor_path(call.M, call.N, call.K, call.G), True,
                           f"config 2 {name} q{q} M{call.M}")
    assert elutq.elutq_device_status() == 0


@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_config4_every_prefill_call(name):
    """The prefill configuration at full size (tensor-core path; CTA pairs for M = 512 and 2048, whole rounds plus
    the K-split tail stripe on gate_up): sampled weight rows x all tokens against the oracle, norm and element-wise."""
    calls = [c for c in workloads.config4_prefill_calls() if c.name == name]
    c0 = calls[0]
    layer = workloads.hlq_layer(0, c0.tag, c0.q, c0.G, c0.N, c0.K)
    packed = pack_layer(layer)
    rows = _sample_rows(c0.N, 512, 7)
    for call in calls:
        X = synth.activations(0, call.tag + f"/x{call.M}", call.M, call.K)
        y = gemm_f16(X, packed, call.N, call.K)
        ref = hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], call.G)
        got = y[:, rows]
        assert np.all(np.isfinite(y))
        assert hlq.rel_fro_error(got, ref) <= TOL_F16, call
        assert max(hlq.rel_fro_error(got[i], ref[i]) for i in range(call.M)) <= 2 * TOL_F16, call
        A = hlq.magnitude_bound(X, layer.scales[rows], layer.offsets[rows], call.G)
        assert_elementwise(got, ref, A, call.q, call.K, True, True, f"config 4a {name} M{call.M}")
    assert elutq.elutq_device_status() == 0


@pytest.mark.parametrize("layer_index", [0, 17])
def test_config4_stack_layers_with_their_own_seeds(layer_index):
    """Two layers of the 32-layer stack (four linears each, their own seeds), as separate calls and as one chain."""
    calls = [c for c in workloads.config4_stack_calls() if c.name.startswith(f"L{layer_index}.")]
    assert len(calls) == 4
    layers = [workloads.hlq_layer(0, c.tag, c.q, c.G, c.N, c.K) for c in calls]
    packed = [pack_layer(l) for l in layers]
    Xs = [synth.activations(0, c.tag + "/x", 1, c.K) for c in calls]
    xd = [x_dev(x) for x in Xs]
    Yc = [torch.zeros((1, c.N), dtype=torch.float16, device="cuda") for c in calls]
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Yc[i], c.N, c.K) for i, c in enumerate(calls)])
    elutq.elutq_chain_run(plan, 4)
    assert elutq.elutq_chain_status(plan) == 0
    for i, c in enumerate(calls):
        ref = hlq.matmul(Xs[i], layers[i].planes, layers[i].scales, layers[i].offsets, c.G)
        A = hlq.magnitude_bound(Xs[i], layers[i].scales, layers[i].offsets, c.G)
        ys = gemm_f16(Xs[i], packed[i], c.N, c.K)
        for y, how in ((ys, "separate call"), (Yc[i].cpu().numpy(), "chain")):
            assert hlq.rel_fro_error(y, ref) <= TOL_F16, (c.name, how)
            assert_elementwise(y, ref, A, c.q, c.K, False, True, f"{c.name} {how}")
    elutq.elutq_chain_forget(plan)


@pytest.mark.parametrize("q", [2, 3, 4])
def test_config1_step_through_the_chain_entry(q):
    """The benchmark's launch configuration: the four linears of one bit-width as one chain, compared in full."""
    calls = [c for c in workloads.config1_calls() if c.q == q]
    layers = [workloads.hlq_layer(0, c.tag, c.q, c.G, c.N, c.K) for c in calls]
    packed = [pack_layer(l) for l in layers]
    Xs = [synth.activations(0, c.tag + "/x", 1, c.K) for c in calls]
    xd = [x_dev(x) for x in Xs]
    Y = [torch.zeros((1, c.N), dtype=torch.float16, device="cuda") for c in calls]
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Y[i], c.N, c.K) for i, c in enumerate(calls)])
    for _ in range(3):
        elutq.elutq_chain_run(plan, len(calls))
    assert elutq.elutq_chain_status(plan) == 0
    for i, c in enumerate(calls):
        ref = hlq.matmul(Xs[i], layers[i].planes, layers[i].scales, layers[i].offsets, c.G)
        y = Y[i].cpu().numpy()
        assert hlq.rel_fro_error(y, ref) <= TOL_F16, c
        assert_elementwise(y, ref, hlq.magnitude_bound(Xs[i], layers[i].scales, layers[i].offsets, c.G), c.q, c.K, False, True, c.name)
    elutq.elutq_chain_forget(plan)


def test_config1_whole_step_as_one_plan():
    """The benchmark's headline launch configuration: all twelve calls (q = 2, 3, 4) in one plan, which elutq_chain_run
    runs as one launch; run three times (epochs), every output compared in full."""
    calls = workloads.config1_calls()
    layers = [workloads.hlq_layer(0, c.tag, c.q, c.G, c.N, c.K) for c in calls]
    packed = [pack_layer(l) for l in layers]
    Xs = [synth.activations(0, c.tag + "/x", 1, c.K) for c in calls]
    xd = [x_dev(x) for x in Xs]
    Y = [torch.zeros((1, c.N), dtype=torch.float16, device="cuda") for c in calls]
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Y[i], c.N, c.K) for i, c in enumerate(calls)])
    for _ in range(3):
        for y in Y:
            y.fill_(float("nan"))
        elutq.elutq_chain_run(plan, len(calls))
    assert elutq.elutq_chain_status(plan) == 0
    for i, c in enumerate(calls):
        ref = hlq.matmul(Xs[i], layers[i].planes, layers[i].scales, layers[i].offsets, c.G)
        y = Y[i].cpu().numpy()
        assert np.all(np.isfinite(y)), c
        assert hlq.rel_fro_error(y, ref) <= TOL_F16, c
        assert_elementwise(y, ref, hlq.magnitude_bound(Xs[i], layers[i].scales, layers[i].offsets, c.G), c.q, c.K, False, True,
                           f"{c.name} q{c.q} in the twelve-call plan")
    elutq.elutq_chain_forget(plan)


def test_config3_step_through_the_chain_entry():
    """The eight 70B calls as one plan (two launches): sampled rows against the oracle, every output finite."""
    calls = workloads.config3_calls()
    packed, xd, Y, refs = [], [], [], []
    for c in calls:
        layer = workloads.hlq_layer(0, c.tag, c.q, c.G, c.N, c.K)
        X = synth.activations(0, c.tag + "/x", 1, c.K)
        rows = _sample_rows(c.N, 512, 8)
        refs.append((rows, hlq.matmul(X, layer.planes[:, rows], layer.scales[rows], layer.offsets[rows], c.G),
                     hlq.magnitude_bound(X, layer.scales[rows], layer.offsets[rows], c.G)))
        packed.append(pack_layer(layer))
        xd.append(x_dev(X))
        Y.append(torch.full((1, c.N), float("nan"), dtype=torch.float16, device="cuda"))
        del layer
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Y[i], c.N, c.K) for i, c in enumerate(calls)])
    elutq.elutq_chain_run(plan, len(calls))
    assert elutq.elutq_chain_status(plan) == 0
    for i, c in enumerate(calls):
        rows, ref, A = refs[i]
        y = Y[i].cpu().numpy()
        assert np.all(np.isfinite(y)), c
        assert hlq.rel_fro_error(y[:, rows], ref) <= TOL_F16, c
        assert_elementwise(y[:, rows], ref, A, c.q, c.K, False, True, f"config 3 {c.name} q{c.q} in the chain")
    elutq.elutq_chain_forget(plan)


def test_smoke_entry_runs():
    import __graft_entry__ as g
    g.smoke()
