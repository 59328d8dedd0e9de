"""Pins for oracle.layout: the reference packer of the device layout.

The paper fixes no device layout, so these pins are structural: the scatter map
is a bijection onto the blob body, packing round-trips, the rotation keeps the
16 lanes of a half-warp on 16 different columns at every step, and reading the
blob in the documented lane order reproduces the definition of Y.
"""

import numpy as np
import pytest

from oracle import hlq, layout


def _layer(rng, q, G, N, K, signed=True):
    planes = rng.integers(0, 2, (q, N, K)).astype(np.uint8)
    s = rng.standard_normal((N, K // G, q)) * 0.02
    s = (s if signed else np.abs(s)).astype(np.float16)
    z = (rng.standard_normal((N, K // G)) * 0.01).astype(np.float16)
    return planes, s, z


@pytest.mark.parametrize("q,G", [(1, 128), (2, 128), (3, 64), (4, 32)])
def test_scatter_map_is_a_bijection_onto_the_body(q, G):
    N, K = 32, 1024
    geo = layout.geometry(q, G, N, K)
    n = np.arange(N)[:, None]
    cg = np.arange(K // 8)[None, :]
    offs = [layout._plane_byte_offsets(geo, j, n, cg).ravel() for j in range(q)]
    gi = np.arange(K // G)[None, :]
    for comp in range(q + 1):
        o = layout._param_offsets(geo, n, gi, comp).ravel()
        offs += [o, o + 1]
    allo = np.concatenate(offs)
    assert allo.min() == layout.HEADER_BYTES
    assert allo.max() == geo["total"] - 1
    assert len(np.unique(allo)) == len(allo) == geo["total"] - layout.HEADER_BYTES


@pytest.mark.parametrize("G", [32, 64, 128])
def test_rotation_is_conflict_free_and_stays_in_one_group_per_phase(G):
    w, nsg = G // 8, 128 // G
    for i in range(16):
        v, ii = divmod(i, w)
        taus = []
        for l in range(16):
            a, r = divmod(l, w)
            tau = w * ((a + v) % nsg) + (r + ii) % w
            taus.append(tau)
            assert tau // w == (a + v) % nsg          # whole phase v stays in one quantisation group
        assert sorted(taus) == list(range(16))        # 16 lanes, 16 different columns


@pytest.mark.parametrize("q,G,N,K", [(2, 128, 48, 1024), (3, 64, 21, 640), (4, 32, 5, 96), (1, 128, 16, 512)])
def test_round_trip_and_header(q, G, N, K):
    rng = np.random.default_rng(q * 7 + N)
    planes, s, z = _layer(rng, q, G, N, K)
    blob = layout.pack_reference(planes, s, z, G)
    assert blob.dtype == np.uint8 and blob.size == layout.packed_bytes(q, G, N, K)
    hd = layout.parse_header(blob)
    assert (hd["q"], hd["G"], hd["N"], hd["K"]) == (q, G, N, K)
    p2, s2, z2 = layout.unpack_reference(blob)
    np.testing.assert_array_equal(p2, planes)
    np.testing.assert_array_equal(s2.view(np.uint16), s.view(np.uint16))
    np.testing.assert_array_equal(z2.view(np.uint16), z.view(np.uint16))


def test_single_bit_lands_where_the_documented_formula_says():
    # q=2, G=128, N=16, K=512: one tile.  Row 5, plane 1, k = 8*(16*3+2)+6: column 50 -> sigma 3 (h=1,u=1), tau 2;
    # lane 16+5, step i = (2-5) mod 16 = 13, vector u*q+j = 3, bit 6.
    q, G, N, K = 2, 128, 16, 512
    planes = np.zeros((q, N, K), np.uint8)
    planes[1, 5, 8 * 50 + 6] = 1
    blob = layout.pack_reference(planes, np.zeros((N, 4, q), np.float16), np.zeros((N, 4), np.float16), G)
    body = blob[layout.HEADER_BYTES:]
    (nz,) = np.nonzero(body)
    assert nz.tolist() == [(3 * 32 + 21) * 16 + 13]
    assert body[nz[0]] == 1 << 6


def test_parameter_record_order_g128():
    # lane (h, l) record = [s_0..s_{q-1}, z] of group h, then of group h+2
    q, G, N, K = 2, 128, 16, 512
    s = (np.arange(N * 4 * q).reshape(N, 4, q) + 1).astype(np.float16)
    z = -(np.arange(N * 4).reshape(N, 4) + 1).astype(np.float16)
    blob = layout.pack_reference(np.zeros((q, N, K), np.uint8), s, z, G)
    par = blob[layout.HEADER_BYTES + 32 * 32 * q:].view(np.float16).reshape(3, 32, 2)   # [word][lane][half]
    for lane in (0, 7, 16, 31):
        h, l = divmod(lane, 16)
        rec = par[:, lane, :].reshape(-1)
        expect = [s[l, h, 0], s[l, h, 1], z[l, h], s[l, h + 2, 0], s[l, h + 2, 1], z[l, h + 2]]
        assert rec.tolist() == [float(e) for e in expect]


@pytest.mark.parametrize("q,G,N,K", [(2, 128, 21, 640), (3, 64, 17, 512), (2, 32, 9, 160), (4, 128, 3, 1024)])
def test_consumer_walk_reproduces_the_definition(q, G, N, K):
    rng = np.random.default_rng(q + G + N + K)
    planes, s, z = _layer(rng, q, G, N, K)
    X = rng.standard_normal((2, K)).astype(np.float16)
    blob = layout.pack_reference(planes, s, z, G)
    np.testing.assert_allclose(layout.consumer_walk(blob, X), hlq.matmul(X, planes, s, z, G),
                               rtol=1e-11, atol=1e-12)


def test_index_map_is_the_little_endian_byte_of_each_column():
    rng = np.random.default_rng(2)
    planes = rng.integers(0, 2, (2, 3, 64)).astype(np.uint8)
    idx = layout.index_map(planes)
    assert idx.shape == (2, 3, 8) and idx.dtype == np.uint8
    for j, n, c in [(0, 0, 0), (1, 2, 7), (0, 1, 3)]:
        assert int(idx[j, n, c]) == sum(int(planes[j, n, 8 * c + b]) << b for b in range(8))
