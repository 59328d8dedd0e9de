"""Pins for oracle.hlq: the definition of the HLQ product (Eq. 3 / Eq. 6, Algorithm 1 shapes).

Each test compares the oracle with something that is not the oracle: the
paper's worked example, exact rational brute force, the uniform closed form
through an integer matmul, or invariants of the definition.
"""

import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import hlq

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_example():
    vals = {}
    with open(os.path.join(GOLDEN, "bit_plane_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = [int(x) for x in v]
    return vals


def test_bit_plane_split_matches_paper_example():
    ex = _read_example()
    planes = hlq.split_bit_planes(np.array([ex["integers"]]), ex["bits"][0])
    assert planes.shape == (4, 1, 4)
    assert planes[0, 0].tolist() == ex["lowest_plane"]
    assert planes[3, 0].tolist() == ex["highest_plane"]


def test_example_reconstructs_integers_and_dot_product():
    # with s_j = 2^j and z = 0 the planes of the worked example must give back (9,7,6,3);
    # an all-ones activation then sums them: 25
    ex = _read_example()
    planes = hlq.split_bit_planes(np.array([ex["integers"]]), 4)
    s = np.array([[[1.0, 2.0, 4.0, 8.0]]])
    z = np.zeros((1, 1))
    w = hlq.reconstruct(planes, s, z, G=4)
    assert w.tolist() == [[9.0, 7.0, 6.0, 3.0]]
    y = hlq.matmul(np.ones((1, 4), np.float16), planes, s, z, G=4)
    assert y.tolist() == [[25.0]]


def _frac(x):
    return Fraction(float(x))


def _brute(X, planes, s, z, G):
    """Exact rational Y from the definition, independent of numpy arithmetic."""
    q, N, K = planes.shape
    M = len(X)
    out = [[Fraction(0)] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                w = _frac(z[n][k // G])
                for j in range(q):
                    if planes[j][n][k]:
                        w += _frac(s[n][k // G][j])
                acc += _frac(X[m][k]) * w
            out[m][n] = acc
    return out


@pytest.mark.parametrize("q,K", [(1, 4), (2, 4), (1, 8)])
def test_all_bit_patterns_against_exact_rationals(q, K):
    # every one of the 2^(qK) bit patterns of a single row, one group
    rng = np.random.default_rng(1)
    X = rng.standard_normal((2, K)).astype(np.float16)
    s = rng.standard_normal((1, 1, q)).astype(np.float16)
    z = rng.standard_normal((1, 1)).astype(np.float16)
    for bits in itertools.product((0, 1), repeat=q * K):
        planes = np.array(bits, dtype=np.uint8).reshape(q, 1, K)
        y = hlq.matmul(X, planes, s, z, G=K)
        ref = _brute(X, planes, s, z, K)
        for m in range(2):
            assert abs(Fraction(float(y[m, 0])) - ref[m][0]) <= abs(ref[m][0]) * Fraction(1, 10**12) + Fraction(1, 10**14)


@pytest.mark.parametrize("q,G,M,N,K", [(2, 8, 3, 5, 16), (3, 16, 2, 4, 32), (4, 8, 1, 3, 24)])
def test_random_tiny_against_exact_rationals_and_loops(q, G, M, N, K):
    rng = np.random.default_rng(q * 100 + K)
    X = rng.standard_normal((M, K)).astype(np.float16)
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    s = (rng.standard_normal((N, K // G, q)) * 0.02).astype(np.float16)   # signed scales
    z = (rng.standard_normal((N, K // G)) * 0.01).astype(np.float16)
    y = hlq.matmul(X, planes, s, z, G)
    ref = _brute(X, planes, s, z, G)
    loops = hlq.matmul_loops(X, planes, s, z, G)
    for m in range(M):
        for n in range(N):
            r = float(ref[m][n])
            assert y[m, n] == pytest.approx(r, rel=1e-12, abs=1e-15)
            assert loops[m, n] == pytest.approx(r, rel=1e-12, abs=1e-15)


@pytest.mark.parametrize("q", [1, 2, 3, 4])
def test_uniform_closed_form_equals_integer_dequantisation(q):
    # Algorithm 1 initialises s = [D, 2D, .., 2^(q-1) D], z = min: then W_hat = D * w_int + z,
    # i.e. ordinary asymmetric uniform dequantisation.  D is a power of two so fp16 holds D*2^j exactly.
    rng = np.random.default_rng(7 + q)
    M, N, K, G = 3, 12, 256, 64
    w_int = rng.integers(0, 1 << q, (N, K))
    delta = 2.0 ** rng.integers(-8, -3, (N, K // G))
    zmin = (rng.standard_normal((N, K // G)) * 0.05).astype(np.float16)
    planes = hlq.split_bit_planes(w_int, q)
    s = np.stack([delta * (1 << j) for j in range(q)], axis=2).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    y = hlq.matmul(X, planes, s, zmin, G)
    # independent path: integer codes -> dequantise -> library matmul
    w_deq = np.repeat(delta, G, axis=1) * w_int.astype(np.float64) + np.repeat(zmin.astype(np.float64), G, axis=1)
    ref = X.astype(np.float64) @ w_deq.T
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)


def test_scale_and_offset_terms_add_up_and_isolate():
    rng = np.random.default_rng(3)
    q, G, M, N, K = 3, 32, 4, 9, 128
    X = rng.standard_normal((M, K)).astype(np.float16)
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    s = np.abs(rng.standard_normal((N, K // G, q)) * 0.02).astype(np.float16)
    z = (rng.standard_normal((N, K // G)) * 0.01).astype(np.float16)
    y = hlq.matmul(X, planes, s, z, G)
    ys = hlq.scale_term(X, planes, s, G)
    yb = hlq.offset_term(X, z, G)
    np.testing.assert_allclose(ys + yb, y, rtol=1e-12, atol=1e-14)
    # all scales zero: only the offset term remains, and it is z[n,Gi] * sum of the group's x
    y0 = hlq.matmul(X, planes, np.zeros_like(s), z, G)
    np.testing.assert_allclose(y0, yb, rtol=1e-12, atol=1e-14)
    grp = X.astype(np.float64).reshape(M, K // G, G).sum(axis=2)
    np.testing.assert_allclose(yb, np.einsum("mg,ng->mn", grp, z.astype(np.float64)), rtol=1e-12, atol=1e-14)
    # all bits zero: scales cannot matter
    yz = hlq.matmul(X, np.zeros_like(planes), s, z, G)
    np.testing.assert_allclose(yz, yb, rtol=1e-12, atol=1e-14)


def test_one_hot_rows_select_single_parameters():
    # a single set bit in plane j at (n,k) with x = e_k must return exactly s[n, k//G, j] + z[n, k//G]
    q, G, N, K = 3, 4, 5, 12
    rng = np.random.default_rng(11)
    s = rng.standard_normal((N, K // G, q)).astype(np.float16)
    z = rng.standard_normal((N, K // G)).astype(np.float16)
    for j, n, k in [(0, 0, 0), (2, 4, 11), (1, 2, 5)]:
        planes = np.zeros((q, N, K), np.uint8)
        planes[j, n, k] = 1
        X = np.zeros((1, K), np.float16)
        X[0, k] = 1.0
        y = hlq.matmul(X, planes, s, z, G)
        expect = z[:, k // G].astype(np.float64)
        expect[n] += float(s[n, k // G, j])
        np.testing.assert_array_equal(y[0], expect)


def test_fp16_rounding_and_error_metric():
    y = np.array([[1.0 + 2.0 ** -12, 65504.0, 1e-9]])
    h = hlq.to_fp16(y)
    assert h.dtype == np.float16 and float(h[0, 0]) == 1.0 and float(h[0, 1]) == 65504.0
    assert hlq.rel_fro_error(np.array([3.0, 4.0]), np.array([3.0, 4.0])) == 0.0
    assert hlq.rel_fro_error(np.array([0.0, 0.0]), np.array([3.0, 4.0])) == pytest.approx(1.0)


def test_magnitude_bound_dominates_the_product_of_magnitudes_for_any_planes():
    # pin of oracle.hlq.magnitude_bound (the scale of the element-wise parity bounds): for random signed
    # parameters and ALL bit patterns of a tiny group, and for random planes of a larger layer, it is at least
    # |X| |W_hat|^T, and it is attained when every weight of a group sits at the group's extreme value
    rng = np.random.default_rng(11)
    q, G, N, K = 2, 2, 1, 4
    s = rng.normal(0, 0.02, (N, K // G, q)).astype(np.float16)
    z = rng.normal(0, 0.01, (N, K // G)).astype(np.float16)
    X = rng.normal(0, 1, (2, K)).astype(np.float16)
    A = hlq.magnitude_bound(X, s, z, G)
    worst = np.zeros_like(A)
    for code in range(1 << (q * N * K)):
        bits = np.array([(code >> i) & 1 for i in range(q * N * K)], dtype=np.uint8).reshape(q, N, K)
        W = hlq.reconstruct(bits, s, z, G)
        worst = np.maximum(worst, np.abs(np.asarray(X, dtype=np.float64)) @ np.abs(W).T)
    assert np.all(A >= worst - 1e-15)
    assert np.allclose(A, worst, rtol=1e-12)          # the maximum over all planes attains the bound
    q, G, N, K = 3, 32, 40, 256
    s = rng.normal(0, 0.02, (N, K // G, q)).astype(np.float16)
    z = rng.normal(0, 0.01, (N, K // G)).astype(np.float16)
    X = rng.normal(0, 1, (5, K)).astype(np.float16)
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    W = hlq.reconstruct(planes, s, z, G)
    assert np.all(hlq.magnitude_bound(X, s, z, G) >= np.abs(np.asarray(X, dtype=np.float64)) @ np.abs(W).T - 1e-12)
