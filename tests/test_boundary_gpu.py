"""GPU tests of the boundary's safety rules: a stale blob description is caught on the device before any tile is read,
library-owned scratch is never freed under a captured graph, nothing is allocated during stream capture, and
unsupported flag / shape combinations are refused before any launch."""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import pack_layer, x_dev  # noqa: E402

TOL_F16 = 1e-3


@pytest.mark.parametrize("M", [1, 4, 16])
def test_a_stale_description_of_a_blob_is_caught_before_any_tile_is_read(M):
    # The library remembers the buffer as a 4-plane blob (it packed it).  A 2-plane blob of the same (N, K) is then
    # copied over the start of the same allocation - which stays as large as the 4-plane blob, so that even an
    # unguarded kernel would stay inside it.  The next call is launched for q = 4; every kernel compares the header
    # first: status 0x7C0B, Y untouched.  After elutq_describe the call is right.
    G, N, K = 128, 512, 1024
    big = workloads.hlq_layer(31, "stale/4", 4, G, N, K)
    small = workloads.hlq_layer(31, "stale/2", 2, G, N, K)
    buf = pack_layer(big)
    small_blob = pack_layer(small)
    buf[: small_blob.numel()].copy_(small_blob)
    X = synth.activations(31, f"stale/x{M}", M, K)
    xd = x_dev(X)
    Y = torch.full((M, N), 7.0, dtype=torch.float16, device="cuda")
    elutq.elutq_release_scratch()
    elutq.elutq_lut_gemm(xd, buf, Y, M, N, K)
    assert elutq.elutq_device_status() == 0x7C0B
    assert torch.all(Y == 7.0)
    elutq.elutq_release_scratch()                      # clears the status word
    assert elutq.elutq_describe(buf, N, K) == (2, G)
    elutq.elutq_lut_gemm(xd, buf, Y, M, N, K)
    assert elutq.elutq_device_status() == 0
    ref = hlq.matmul(X, small.planes, small.scales, small.offsets, G)
    assert hlq.rel_fro_error(Y.cpu().numpy(), ref) <= TOL_F16
    elutq.elutq_forget(buf)


def test_unpack_refuses_a_stale_description_too():
    G, N, K = 128, 64, 512
    big = workloads.hlq_layer(32, "stale-unpack/3", 3, G, N, K)
    small = workloads.hlq_layer(32, "stale-unpack/1", 1, G, N, K)
    buf = pack_layer(big)
    small_blob = pack_layer(small)
    buf[: small_blob.numel()].copy_(small_blob)
    planes = torch.full((3, N, K), 9, dtype=torch.uint8, device="cuda")
    scales = torch.zeros((N, K // G, 3), dtype=torch.float16, device="cuda")
    offsets = torch.zeros((N, K // G), dtype=torch.float16, device="cuda")
    elutq.elutq_unpack(buf, N, K, planes, scales, offsets)   # launched for q = 3 from the remembered description
    torch.cuda.synchronize()
    assert torch.all(planes == 9)                            # nothing was read, nothing written
    elutq.elutq_forget(buf)


def test_scratch_that_grows_is_replaced_not_freed_and_a_captured_graph_keeps_working():
    q, G = 2, 128
    small = workloads.hlq_layer(33, "grow/small", q, G, 256, 2048)
    large = workloads.hlq_layer(33, "grow/large", q, G, 40000, 4096)     # partial sums above the 1 MiB first allocation
    ps, pl = pack_layer(small), pack_layer(large)
    Xs, Xl = synth.activations(33, "grow/xs", 1, 2048), synth.activations(33, "grow/xl", 1, 4096)
    xs, xl = x_dev(Xs), x_dev(Xl)
    Ys = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    Yl = torch.zeros((1, 40000), dtype=torch.float16, device="cuda")
    elutq.elutq_release_scratch()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        elutq.elutq_lut_gemm(xs, ps, Ys, 1, 256, 2048)            # allocates the stream's scratch
        stream.synchronize()
        first, first_bytes = elutq.elutq_scratch_address(3)
        assert first is not None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            elutq.elutq_lut_gemm(xs, ps, Ys, 1, 256, 2048)
            # while capturing nothing is allocated: a shape that needs more scratch is refused
            with pytest.raises(elutq.ElutqError) as err:
                elutq.elutq_lut_gemm(xl, pl, Yl, 1, 40000, 4096)
            assert err.value.status == -4
        elutq.elutq_lut_gemm(xl, pl, Yl, 1, 40000, 4096)          # eager: the scratch grows
        stream.synchronize()
        second, second_bytes = elutq.elutq_scratch_address(3)
        assert second != first and second_bytes > first_bytes
        Ys.zero_()
        g.replay()                                                # still uses the first buffer: it must still be there
        stream.synchronize()
    ref_s = hlq.matmul(Xs, small.planes, small.scales, small.offsets, G)
    ref_l = hlq.matmul(Xl, large.planes, large.scales, large.offsets, G)
    assert hlq.rel_fro_error(Ys.cpu().numpy(), ref_s) <= TOL_F16
    assert hlq.rel_fro_error(Yl.cpu().numpy(), ref_l) <= TOL_F16
    assert elutq.elutq_device_status(stream) == 0
    del g
    elutq.elutq_release_scratch()


def test_reserve_makes_room_before_a_capture():
    q, G, N, K = 2, 128, 40000, 4096
    layer = workloads.hlq_layer(34, "reserve", q, G, N, K)
    packed = pack_layer(layer)
    X = synth.activations(34, "reserve/x", 1, K)
    xd = x_dev(X)
    Y = torch.zeros((1, N), dtype=torch.float16, device="cuda")
    elutq.elutq_release_scratch()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        elutq.elutq_reserve(1, N, K)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            elutq.elutq_lut_gemm(xd, packed, Y, 1, N, K)
        g.replay()
        stream.synchronize()
    assert hlq.rel_fro_error(Y.cpu().numpy(), hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)) <= TOL_F16
    del g
    elutq.elutq_release_scratch()


def test_pack_then_gemm_without_a_synchronisation_in_between():
    # the GEMM kernels request the first weights before they wait for the preceding work on the stream; after
    # elutq_pack on the same stream that is safe (the pack kernels complete before a dependent launch starts)
    q, G, N, K = 3, 128, 1000, 2048
    layer = workloads.hlq_layer(35, "nosync", q, G, N, K)
    planes = torch.from_numpy(layer.planes).cuda()
    scales = torch.from_numpy(layer.scales.view(np.int16)).cuda().view(torch.float16)
    offsets = torch.from_numpy(layer.offsets.view(np.int16)).cuda().view(torch.float16)
    X = synth.activations(35, "nosync/x", 1, K)
    xd = x_dev(X)
    outs = []
    for sync in (True, False):
        packed = torch.zeros(elutq.elutq_packed_bytes(q, G, N, K), dtype=torch.uint8, device="cuda")
        Y = torch.zeros((1, N), dtype=torch.float16, device="cuda")
        torch.cuda.synchronize()
        elutq.elutq_pack(planes, scales, offsets, q, G, N, K, packed=packed)
        if sync:
            torch.cuda.synchronize()
        elutq.elutq_lut_gemm(xd, packed, Y, 1, N, K)
        torch.cuda.synchronize()
        outs.append(Y.cpu().numpy().copy())
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    assert hlq.rel_fro_error(outs[1], hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)) <= TOL_F16


def test_unsupported_combinations_are_refused_with_their_own_code():
    q, G, N, K = 2, 128, 64, 1024
    layer = workloads.hlq_layer(36, "unsup", q, G, N, K)
    packed = pack_layer(layer)
    X = synth.activations(36, "unsup/x", 4, K)
    xd = x_dev(X)
    Y = torch.zeros((4, N), dtype=torch.float32, device="cuda")
    before = elutq.elutq_launch_count()
    for flag in (elutq.FLAG_PLAIN_G4, elutq.FLAG_MIRROR, elutq.FLAG_CLUSTER_REDUCE):
        with pytest.raises(elutq.ElutqError) as err:
            elutq.elutq_lut_gemm_f32(xd, packed, Y, 4, N, K, flag)       # decode-kernel variants at M > 1
        assert err.value.status == -5
    layer64 = workloads.hlq_layer(36, "unsup64", q, 64, N, K)
    p64 = pack_layer(layer64)
    before = elutq.elutq_launch_count()
    with pytest.raises(elutq.ElutqError) as err:
        elutq.elutq_lut_gemm_f32(xd, p64, Y, 4, N, K, elutq.FLAG_TABLE_F16)
    assert err.value.status == -5
    with pytest.raises(elutq.ElutqError) as err:
        elutq.elutq_chain_plan([(xd, packed, Y, N, K, elutq.FLAG_SKIP_OFFSET)])
    assert err.value.status == -5
    assert elutq.elutq_launch_count() == before
