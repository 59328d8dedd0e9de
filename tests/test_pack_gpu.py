"""GPU parity of elutq_pack / elutq_unpack: byte-exact against the oracle's reference packer."""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import layout

pytestmark = pytest.mark.gpu

from gpu_util import pack_layer, to_dev  # noqa: E402

CASES = [(2, 128, 4096, 4096), (3, 128, 333, 1536), (4, 128, 64, 2560), (2, 64, 50, 1088),
         (1, 32, 17, 96), (2, 128, 16, 512), (3, 64, 1000, 4096), (4, 32, 48, 1024), (2, 128, 1, 128)]


@pytest.mark.parametrize("q,G,N,K", CASES)
def test_pack_is_byte_exact_and_round_trips(q, G, N, K):
    layer = workloads.hlq_layer(3, f"pack/{q}/{G}/{N}/{K}", q, G, N, K, signed_scales=True)
    packed = pack_layer(layer)
    ref = layout.pack_reference(layer.planes, layer.scales, layer.offsets, G)
    got = packed.cpu().numpy()
    assert got.size == ref.size
    assert np.array_equal(got, ref), f"first differing byte at {int(np.argmax(got != ref))}"
    # inverse
    planes = torch.empty((q, N, K), dtype=torch.uint8, device="cuda")
    scales = torch.empty((N, K // G, q), dtype=torch.float16, device="cuda")
    offsets = torch.empty((N, K // G), dtype=torch.float16, device="cuda")
    elutq.elutq_unpack(packed, N, K, planes, scales, offsets)
    torch.cuda.synchronize()
    assert np.array_equal(planes.cpu().numpy(), layer.planes)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), layer.scales.view(np.uint16))
    assert np.array_equal(offsets.cpu().numpy().view(np.uint16), layer.offsets.view(np.uint16))


def test_nonzero_plane_bytes_count_as_one():
    # a weight bit is (value != 0): any non-zero byte is a set bit
    q, G, N, K = 2, 128, 16, 512
    layer = workloads.hlq_layer(5, "pack/nz", q, G, N, K)
    planes = layer.planes.copy()
    planes[planes != 0] = 0x80
    blob_a = pack_layer(layer).cpu().numpy()
    p = elutq.elutq_pack(to_dev(planes), to_dev(layer.scales.view(np.int16)).view(torch.float16),
                         to_dev(layer.offsets.view(np.int16)).view(torch.float16), q, G, N, K)
    torch.cuda.synchronize()
    assert np.array_equal(p.cpu().numpy(), blob_a)


def test_blob_is_position_independent_and_self_describing():
    q, G, N, K = 3, 64, 40, 1024
    layer = workloads.hlq_layer(6, "pack/move", q, G, N, K)
    packed = pack_layer(layer)
    moved = packed.clone()                       # a different address, unknown to the registry
    assert elutq.elutq_describe(moved, N, K) == (q, G)
    with pytest.raises(elutq.ElutqError) as ei:
        elutq.elutq_describe(moved, N + 1, K)    # wrong shape for this blob
    assert ei.value.status == -2
    junk = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(elutq.ElutqError) as ei:
        elutq.elutq_describe(junk, 16, 512)
    assert ei.value.status == -2
    elutq.elutq_forget(moved)


def test_pack_rejects_small_buffer_on_device_pointers():
    q, G, N, K = 2, 128, 32, 512
    layer = workloads.hlq_layer(7, "pack/small", q, G, N, K)
    small = torch.empty(elutq.elutq_packed_bytes(q, G, N, K) - 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(elutq.ElutqError) as ei:
        elutq.elutq_pack(to_dev(layer.planes), to_dev(layer.scales.view(np.int16)),
                         to_dev(layer.offsets.view(np.int16)), q, G, N, K, packed=small)
    assert ei.value.status == -4
