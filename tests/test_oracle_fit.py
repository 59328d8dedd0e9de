"""Pins for the Algorithm 1 oracle (oracle/fit.py): closed forms, invariants, brute force, library least squares."""
import itertools

import numpy as np
import pytest

import workloads
from oracle import fit as ofit
from oracle import hlq


def _w(seed, N, K, tag="fit"):
    return workloads.dense_weights(seed, tag, N, K)


def _sse_fp64(W, planes, scales, offsets, G):
    rec = hlq.reconstruct(planes, scales, offsets, G)
    return float(np.sum((W.astype(np.float64) - rec) ** 2))


@pytest.mark.parametrize("q", [1, 2, 3, 4])
def test_first_selection_is_uniform_rounding(q):
    """With the initial parameters (Algorithm 1, initialisation) the nearest candidate is the ordinary uniform
    round-to-nearest code clamp(round((w - min) / Delta)): a textbook closed form."""
    G = 64
    W = _w(3, 8, 256)
    w = W.astype(np.float64).reshape(-1, G)
    wmin, wmax = w.min(1), w.max(1)
    delta = (wmax - wmin) / ((1 << q) - 1)
    s = np.stack([delta * (1 << j) for j in range(q)], axis=1)
    codes = ofit.select_bits(w, s, wmin, q)
    t = (w - wmin[:, None]) / delta[:, None]
    expect = np.clip(np.floor(t + 0.5), 0, (1 << q) - 1).astype(np.int64)
    frac = np.abs(t - np.floor(t) - 0.5)
    safe = frac > 1e-9                               # away from exact midpoints
    assert safe.mean() > 0.999
    assert np.array_equal(codes[safe], expect[safe])


@pytest.mark.parametrize("q,G", [(2, 32), (3, 64), (4, 128)])
def test_grid_weights_are_a_fixed_point(q, G):
    """Weights that already lie on a uniform grid min + c * step (all codes present) are reproduced exactly:
    planes = binary digits of c, s_j = step * 2^j, z = min."""
    rng = np.random.default_rng(5)
    N, K = 6, 2 * G
    step = 2.0 ** -7
    c = rng.integers(0, 1 << q, size=(N, K))
    c.reshape(-1, G)[:, : (1 << q)] = np.arange(1 << q)   # every code occurs in every group
    W = (-0.25 + step * c).astype(np.float16)
    assert np.array_equal(W.astype(np.float64), -0.25 + step * c)
    planes, s, z = ofit.fit(W, q, G, t_max=3)
    assert np.array_equal(planes, hlq.split_bit_planes(c, q))
    assert np.allclose(z.astype(np.float64), -0.25, atol=1e-6)
    for j in range(q):
        assert np.allclose(s[:, :, j].astype(np.float64), step * (1 << j), rtol=1e-3)
    assert _sse_fp64(W, planes, s, z, G) < 1e-12


@pytest.mark.parametrize("q", [2, 3, 4])
def test_error_never_increases(q):
    """Both half-steps minimise the same objective (Eq. 7), so the per-group error is non-increasing in t."""
    W = _w(7, 16, 512)
    *_, tr = ofit.fit(W, q, 128, t_max=10, trace=True)
    assert tr.shape == (11, 16 * 4)
    assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-12) + 1e-18)
    assert tr[-1].sum() < 0.9 * tr[0].sum()           # and the fit clearly beats the uniform start


def test_least_squares_step_matches_library():
    """The elimination without pivoting agrees with numpy.linalg.lstsq on [B 1] for the selected bits."""
    q, G = 3, 64
    W = _w(11, 4, 256)
    w = W.astype(np.float64).reshape(-1, G)
    wmin, wmax = w.min(1), w.max(1)
    delta = (wmax - wmin) / ((1 << q) - 1)
    s0 = np.stack([delta * (1 << j) for j in range(q)], axis=1)
    codes = ofit.select_bits(w, s0, wmin, q)
    A, r = ofit.normal_equations(w, codes, q)
    assert not ofit.is_singular(A).any()
    x = ofit.solve_spd(A, r)
    for g in range(w.shape[0]):
        B1 = np.stack([((codes[g] >> j) & 1).astype(np.float64) for j in range(q)] + [np.ones(G)], axis=1)
        ref, *_ = np.linalg.lstsq(B1, w[g], rcond=None)
        assert np.allclose(x[g], ref, rtol=1e-9, atol=1e-12)
        assert np.array_equal(A[g], (B1.T @ B1).astype(np.int64))
        assert np.allclose(r[g], B1.T @ w[g], rtol=1e-12, atol=1e-15)


def test_one_bit_is_two_means():
    """q = 1: the least-squares step puts z on the mean of the zero class and z + s on the mean of the one class,
    and the selection step assigns to the nearer of the two: Lloyd's algorithm for two centres."""
    G = 64
    W = _w(13, 4, 256)
    w = W.astype(np.float64).reshape(-1, G)
    lo, hi = w.min(1), w.max(1)                        # initial centres: min and max (Delta = max - min)
    for _ in range(10):
        assign = np.abs(w - hi[:, None]) < np.abs(w - lo[:, None])
        lo = np.array([w[g][~assign[g]].mean() for g in range(w.shape[0])])
        hi = np.array([w[g][assign[g]].mean() for g in range(w.shape[0])])
    assign = None
    planes, s, z = ofit.fit(W, 1, G, t_max=10)
    assert np.allclose(z.astype(np.float64).ravel(), lo, rtol=2e-3, atol=1e-6)
    assert np.allclose((z.astype(np.float64) + s[:, :, 0].astype(np.float64)).ravel(), hi, rtol=2e-3, atol=1e-6)


def test_brute_force_tiny_group():
    """G = 6, q = 2: the alternating fit can not beat the global optimum over all 4^6 bit assignments (each with its
    own least-squares parameters), and it is no worse than its uniform start."""
    q, G = 2, 6
    W = _w(17, 5, 6)
    *_, tr = ofit.fit(W, q, G, t_max=10, trace=True)
    w = W.astype(np.float64)
    for g in range(5):
        best = np.inf
        for assign in itertools.product(range(4), repeat=G):
            a = np.array(assign)
            B1 = np.stack([(a & 1).astype(np.float64), ((a >> 1) & 1).astype(np.float64), np.ones(G)], axis=1)
            x, *_ = np.linalg.lstsq(B1, w[g], rcond=None)
            best = min(best, float(np.sum((w[g] - B1 @ x) ** 2)))
        assert tr[-1, g] >= best - 1e-15
        assert tr[-1, g] <= tr[0, g] + 1e-18


def test_constant_group_keeps_parameters():
    """max = min: Delta = 0, every candidate equals z, the code is 0 everywhere, the normal equations are singular
    and the parameters stay s = 0, z = min: the group is reproduced exactly."""
    W = np.full((2, 64), 0.125, dtype=np.float16)
    planes, s, z = ofit.fit(W, 2, 32, t_max=4)
    assert not planes.any()
    assert np.all(s == 0) and np.all(z == np.float16(0.125))


def test_singularity_test_is_exact():
    """Gram matrices of dependent columns (equal planes, a constant plane) are singular; independent ones are not."""
    G = 32
    rng = np.random.default_rng(2)
    b0 = rng.integers(0, 2, G)
    b1 = rng.integers(0, 2, G)
    codes_dep = (b0 | (b0 << 1))[None, :]              # plane 1 == plane 0
    codes_const = (b0 | (1 << 1))[None, :]             # plane 1 constant one == the ones column
    codes_ok = (b0 | (b1 << 1))[None, :]
    w = np.zeros((1, G))
    for codes, want in [(codes_dep, True), (codes_const, True), (codes_ok, False)]:
        A, _ = ofit.normal_equations(w, codes, 2)
        assert bool(ofit.is_singular(A)[0]) is want
        assert bool(abs(np.linalg.det(A[0].astype(np.float64))) < 1e-6) == want


def test_fit_output_feeds_the_product():
    """The fitted layer is a valid HLQ layer: reconstruction error (Eq. 7) well below the weights' energy and
    below round-to-nearest uniform quantisation with the same bit width."""
    q, G = 2, 128
    W = _w(19, 8, 512)
    planes, s, z = ofit.fit(W, q, G)
    w = W.astype(np.float64)
    err = _sse_fp64(W, planes, s, z, G)
    wg = w.reshape(-1, G)
    delta = (wg.max(1) - wg.min(1)) / 3
    rtn = wg.min(1)[:, None] + np.clip(np.floor((wg - wg.min(1)[:, None]) / delta[:, None] + 0.5), 0, 3) * delta[:, None]
    assert err < np.sum((wg - rtn) ** 2)
    assert err < 0.2 * np.sum(w ** 2)
