"""The seeded input generators: determinism, row-wise generation, distributions, config call lists."""

import numpy as np

import workloads
from workloads import synth


def test_generators_are_deterministic_and_row_addressable():
    a = synth.bit_planes(0, "t", 2, 40, 128)
    b = synth.bit_planes(0, "t", 2, 40, 128)
    np.testing.assert_array_equal(a, b)
    rows = np.array([3, 17, 39])
    np.testing.assert_array_equal(synth.bit_planes(0, "t", 2, 40, 128, rows=rows), a[:, rows])
    s = synth.scales(0, "t", 40, 4, 3)
    np.testing.assert_array_equal(synth.scales(0, "t", 40, 4, 3, rows=rows), s[rows])
    z = synth.offsets(0, "t", 40, 4)
    np.testing.assert_array_equal(synth.offsets(0, "t", 40, 4, rows=rows), z[rows])
    assert not np.array_equal(synth.bit_planes(1, "t", 2, 40, 128), a)
    assert not np.array_equal(synth.bit_planes(0, "u", 2, 40, 128), a)


def test_distributions_follow_the_recipe():
    p = synth.bit_planes(0, "d", 2, 256, 1024)
    assert set(np.unique(p)) == {0, 1} and abs(p.mean() - 0.5) < 0.005
    s = synth.scales(0, "d", 4096, 8, 2).astype(np.float64)
    assert s.dtype == np.float64 and s.min() >= 0 and abs(s.mean() - 0.02 * np.sqrt(2 / np.pi)) < 5e-4
    z = synth.offsets(0, "d", 4096, 8).astype(np.float64)
    assert abs(z.mean()) < 5e-4 and abs(z.std() - 0.01) < 5e-4
    x = synth.activations(0, "d", 4, 4096).astype(np.float64)
    assert abs(x.mean()) < 0.05 and abs(x.std() - 1.0) < 0.05
    assert synth.scales(0, "d", 64, 8, 2, signed=True).min() < 0


def test_outlier_columns():
    assert len(synth.outlier_columns(0, "o", 4096)) == 41
    assert len(synth.outlier_columns(0, "o", 14336)) == 144
    x = synth.activations(0, "o", 8, 4096, outliers=True).astype(np.float64)
    x0 = synth.activations(0, "o", 8, 4096).astype(np.float64)
    cols = synth.outlier_columns(0, "o", 4096)
    mask = np.zeros(4096, bool)
    mask[cols] = True
    np.testing.assert_array_equal(x[:, ~mask], x0[:, ~mask])
    assert np.abs(x[:, mask]).mean() > 10 * np.abs(x0[:, mask]).mean()


def test_config_call_lists():
    assert len(workloads.config1_calls()) == 12
    assert len(workloads.config2_calls()) == 48
    assert len(workloads.config3_calls()) == 8
    assert len(workloads.config4_prefill_calls()) == 12
    assert len(workloads.config4_stack_calls()) == 128
    c = workloads.config0()[0]
    assert workloads.algorithmic_bytes(c.M, c.N, c.K, c.q, c.G) == 4_997_120
    assert workloads.algorithmic_bytes(1, 28672, 4096, 2, 128) == 34_930_688
    assert workloads.algorithmic_bytes(1, 57344, 8192, 3, 128) == 205_651_968
    total = sum(workloads.algorithmic_bytes(c.M, c.N, c.K, c.q, c.G) for c in workloads.config4_stack_calls())
    assert total == 2_076_442_624
