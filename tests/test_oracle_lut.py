"""Pins for oracle.lut: the bit-serial LUT procedure (Appendix B) and mirror storage (Appendix D)."""

import numpy as np
import pytest

from oracle import hlq, lut


def test_table_size_recurrences_and_all_ones_entry():
    rng = np.random.default_rng(0)
    for g in (1, 2, 4, 8):
        x = rng.standard_normal(8 * g).astype(np.float16)
        T = lut.build_lut(x, g)
        assert T.shape == (8, 1 << g)                      # 2^g entries per slice; 16 for g = 4
        assert np.all(T[:, 0] == 0.0)
        xs = x.astype(np.float64).reshape(8, g)
        for i in range(g):                                  # LUT[p | 2^i] = LUT[p] + x_i for p without bit i
            for p in range(1 << g):
                if not (p >> i) & 1:
                    np.testing.assert_allclose(T[:, p | (1 << i)], T[:, p] + xs[:, i], rtol=0, atol=1e-12)
        np.testing.assert_allclose(T[:, -1], xs.sum(axis=1), rtol=0, atol=1e-12)


def test_indices_of_the_worked_example_are_little_endian():
    planes = hlq.split_bit_planes(np.array([[9, 7, 6, 3]]), 4)
    idx = lut.plane_indices(planes, 4)
    assert idx[:, 0, 0].tolist() == [11, 14, 6, 1]         # plane 0 = (1,1,0,1) -> 1+2+8; plane 1 = (0,1,1,1) -> 14; plane 3 = (1,0,0,0) -> 1
    y = lut.lut_matmul(np.ones((1, 4), np.float16), planes,
                       np.array([[[1.0, 2.0, 4.0, 8.0]]]), np.zeros((1, 1)), G=4, g=4)
    assert y.tolist() == [[25.0]]


@pytest.mark.parametrize("q,G,g", [(2, 128, 4), (3, 64, 4), (4, 32, 8), (2, 128, 8), (1, 16, 2)])
def test_lut_procedure_equals_definition(q, G, g):
    rng = np.random.default_rng(q + G + g)
    M, N, K = 3, 17, 2 * G
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, 3] *= 20.0
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    s = (rng.standard_normal((N, K // G, q)) * 0.02).astype(np.float16)
    z = (rng.standard_normal((N, K // G)) * 0.01).astype(np.float16)
    ref = hlq.matmul(X, planes, s, z, G)
    np.testing.assert_allclose(lut.lut_matmul(X, planes, s, z, G, g), ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lut.mirror_lut_matmul(X, planes, s, z, G, g), ref, rtol=1e-11, atol=1e-12)


def test_mirror_identity_and_antisymmetry():
    rng = np.random.default_rng(5)
    q, G, N, K = 3, 16, 6, 64
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    s = (rng.standard_normal((N, K // G, q)) * 0.02).astype(np.float16)
    z = (rng.standard_normal((N, K // G)) * 0.01).astype(np.float16)
    np.testing.assert_allclose(lut.reconstruct_mirror(planes, s, z, G),
                               hlq.reconstruct(planes, s, z, G), rtol=1e-13, atol=1e-15)
    g = 4
    x = rng.standard_normal(K).astype(np.float16)
    half = lut.build_mirror_half_lut(x, g)
    assert half.shape == (K // g, 8)                        # half of the 16 entries is stored
    xs = x.astype(np.float64).reshape(-1, g)
    t = np.arange(K // g)
    for p in range(16):
        signs = np.array([1.0 if (p >> i) & 1 else -1.0 for i in range(g)])
        direct = xs @ signs
        got = lut.mirror_lookup(half, t, np.full_like(t, p), g)
        np.testing.assert_allclose(got, direct, rtol=0, atol=1e-12)
        comp = lut.mirror_lookup(half, t, np.full_like(t, 15 - p), g)
        np.testing.assert_allclose(comp, -direct, rtol=0, atol=1e-12)   # table is antisymmetric
    # the extreme entries are -(x1+..+x4) and +(x1+..+x4)
    np.testing.assert_allclose(lut.mirror_lookup(half, t, np.zeros_like(t), g), -xs.sum(1), atol=1e-12)
    np.testing.assert_allclose(lut.mirror_lookup(half, t, np.full_like(t, 15), g), xs.sum(1), atol=1e-12)


def test_f16_tables_are_exact_when_entries_are_representable():
    """Small-integer activations: every table entry is an integer below 2048, exactly an fp16 value, so the
    fp16-table procedure must reproduce the definition (Eq. 3 / Eq. 6) exactly."""
    rng = np.random.default_rng(8)
    q, G, N, K, M = 2, 32, 12, 128, 3
    planes = rng.integers(0, 2, size=(q, N, K)).astype(np.uint8)
    scales = rng.integers(-4, 5, size=(N, K // G, q)).astype(np.float16)
    offsets = rng.integers(-3, 4, size=(N, K // G)).astype(np.float16)
    X = rng.integers(-50, 51, size=(M, K)).astype(np.float16)
    ref = hlq.matmul(X, planes, scales, offsets, G)
    assert np.array_equal(lut.table_f16_lut_matmul(X, planes, scales, offsets, G), ref)


def test_f16_tables_error_is_one_rounding_per_entry():
    """General activations: the deviation from the definition is bounded by 2^-11 of the looked-up magnitudes
    weighted by |s| (one fp16 rounding per entry), and is not zero."""
    rng = np.random.default_rng(9)
    q, G, N, K, M = 3, 64, 10, 256, 2
    planes = rng.integers(0, 2, size=(q, N, K)).astype(np.uint8)
    scales = np.abs(rng.normal(0, 0.02, size=(N, K // G, q))).astype(np.float16)
    offsets = rng.normal(0, 0.01, size=(N, K // G)).astype(np.float16)
    X = rng.normal(0, 1, size=(M, K)).astype(np.float16)
    ref = hlq.matmul(X, planes, scales, offsets, G)
    got = lut.table_f16_lut_matmul(X, planes, scales, offsets, G)
    # bound: sum over planes, groups and slices of |s| * 2^-11 * sum|x| of the slice
    absx = np.abs(X.astype(np.float64)).reshape(M, K // G, G).sum(axis=2)            # [M, groups]
    bound = 2.0 ** -11 * np.einsum("mg,ngj->mn", absx, np.abs(scales.astype(np.float64)))
    assert np.all(np.abs(got - ref) <= bound)
    assert np.any(got != ref)
    assert hlq.rel_fro_error(got, ref) < 1e-3


def test_i8_tables_are_exact_when_entries_sit_on_the_code_grid():
    """Activations that are multiples of 1/16 with one slice per group summing to 127/16 in magnitude: the scale is
    exactly 1/16, every table entry is an integer number of scales, so the int8-table procedure is lossless and
    must reproduce the definition exactly."""
    rng = np.random.default_rng(10)
    q, G, N, K, M = 2, 64, 9, 256, 2
    X = (rng.integers(-12, 13, size=(M, K)) / 16.0)
    for m in range(M):
        for gi in range(K // G):
            X[m, gi * G: gi * G + 8] = [1, -1, 1, 1, -1, 1, 1, 0.9375]        # sum |x| = 127/16, the group's maximum
    X = X.astype(np.float16)
    assert np.abs(X.astype(np.float64)).reshape(M, K // 8, 8).sum(axis=2).max() == 127 / 16
    planes = rng.integers(0, 2, size=(q, N, K)).astype(np.uint8)
    scales = rng.integers(-4, 5, size=(N, K // G, q)).astype(np.float16)
    offsets = rng.integers(-3, 4, size=(N, K // G)).astype(np.float16)
    ref = hlq.matmul(X, planes, scales, offsets, G)
    assert np.array_equal(lut.table_i8_lut_matmul(X, planes, scales, offsets, G), ref)


def test_i8_tables_error_is_half_a_code_per_lookup():
    """General activations: each looked-up value is off by at most scale / 2, so the deviation from the definition
    is bounded by sum |s| * (slices per group) * scale / 2; it is far larger than the fp16-table error."""
    rng = np.random.default_rng(11)
    q, G, N, K, M = 3, 128, 10, 512, 2
    planes = rng.integers(0, 2, size=(q, N, K)).astype(np.uint8)
    scales = np.abs(rng.normal(0, 0.02, size=(N, K // G, q))).astype(np.float16)
    offsets = rng.normal(0, 0.01, size=(N, K // G)).astype(np.float16)
    X = rng.normal(0, 1, size=(M, K)).astype(np.float16)
    ref = hlq.matmul(X, planes, scales, offsets, G)
    got = lut.table_i8_lut_matmul(X, planes, scales, offsets, G)
    amax = np.abs(X.astype(np.float64)).reshape(M, K // G, G // 8, 8).sum(axis=3).max(axis=2)   # [M, groups]
    bound = np.einsum("mg,ngj->mn", amax / 127.0 / 2.0 * (G // 8), np.abs(scales.astype(np.float64)))
    assert np.all(np.abs(got - ref) <= bound * (1 + 1e-12))
    e8 = hlq.rel_fro_error(got, ref)
    e16 = hlq.rel_fro_error(lut.table_f16_lut_matmul(X, planes, scales, offsets, G), ref)
    assert 1e-3 < e8 < 3e-2 and e8 > 5 * e16
