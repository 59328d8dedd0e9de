"""elutq_lut_gemm_static: the entry point for callers that cannot allocate device memory.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  The entry point keeps its K-split scratch in a fixed array inside the library,
so it must give the same result as elutq_lut_gemm, call after call, with no set-up by the caller.
"""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

TOL_F16 = 1e-3


def test_static_entry_rejects_shapes_beyond_its_scratch_before_any_launch():
    # 16 chunks * 64 rows * 57344 output rows * 4 bytes is far above the 4 MiB built-in scratch
    L = elutq.lib()
    before = elutq.elutq_launch_count()
    assert L.elutq_lut_gemm_static(16, 16, 16, 64, 57344, 8192, None) == -4
    assert L.elutq_lut_gemm_static(None, 16, 16, 1, 64, 1024, None) == -1
    assert L.elutq_lut_gemm_static(8, 16, 16, 1, 64, 1024, None) == -3
    assert elutq.elutq_launch_count() == before


@pytest.mark.gpu
def test_static_entry_matches_the_allocating_entry_on_two_calls_in_a_row():
    from gpu_util import pack_layer, x_dev

    q, G, N, K = 3, 128, 1000, 4096            # 8-way K split, ragged row tail
    layer = workloads.hlq_layer(11, "static", q, G, N, K)
    packed = pack_layer(layer)
    ref64 = None
    for call in range(2):                       # second call reuses the array with the first call's leftovers in it
        X = synth.activations(11 + call, "static/x", 1, K)
        xd = x_dev(X)
        Y_ref = torch.empty((1, N), dtype=torch.float16, device="cuda")
        elutq.elutq_lut_gemm(xd, packed, Y_ref, 1, N, K)
        Y = torch.full((1, N), float("nan"), dtype=torch.float16, device="cuda")
        elutq.elutq_lut_gemm_static(xd, packed, Y, 1, N, K)
        torch.cuda.synchronize()
        got, want = Y.cpu().numpy(), Y_ref.cpu().numpy()
        assert np.all(np.isfinite(got))
        assert hlq.rel_fro_error(got, want) <= TOL_F16
        ref64 = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G)
        assert hlq.rel_fro_error(got, ref64) <= TOL_F16
    # a small batch goes through the same entry
    Xb = synth.activations(13, "static/xb", 3, K)
    Yb = torch.empty((3, N), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm_static(x_dev(Xb), packed, Yb, 3, N, K)
    torch.cuda.synchronize()
    assert hlq.rel_fro_error(Yb.cpu().numpy(), hlq.matmul(Xb, layer.planes, layer.scales, layer.offsets, G)) <= TOL_F16


@pytest.mark.gpu
def test_static_entry_at_the_edges_of_what_it_offers():
    """A single K chunk (no scratch at all), a batch of nine (which stays on the look-up kernels here), the largest
    shape the built-in scratch holds and the first one beyond it, and a small call right after a large one, when the
    array still holds the large call's partial sums."""
    from gpu_util import pack_layer, x_dev

    # K = 512: one chunk, nothing is split; and M = 9 on the same layer and on a split one
    for (q, N, K, M) in [(2, 300, 512, 1), (2, 300, 512, 9), (3, 500, 2048, 9)]:
        layer = workloads.hlq_layer(14, f"static/edge/{N}/{K}", q, 128, N, K)
        packed = pack_layer(layer)
        X = synth.activations(14, f"static/edge/x/{M}/{K}", M, K)
        Y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        elutq.elutq_lut_gemm_static(x_dev(X), packed, Y, M, N, K)
        torch.cuda.synchronize()
        assert hlq.rel_fro_error(Y.cpu().numpy(), hlq.matmul(X, layer.planes, layer.scales, layer.offsets, 128)) <= TOL_F16

    # exactly 4 MiB of partial sums: 8 chunks x 131072 rows x 4 bytes (inputs drawn on the device; the allocating
    # entry is the reference here), then one row block more: refused before any launch
    q, G, N, K = 1, 128, 131072, 4096
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    planes = torch.randint(0, 2, (q, N, K), dtype=torch.uint8, device="cuda", generator=gen)
    scales = (torch.randn((N, K // G, q), device="cuda", generator=gen) * 0.02).abs().to(torch.float16)
    offsets = (torch.randn((N, K // G), device="cuda", generator=gen) * 0.01).to(torch.float16)
    packed = elutq.elutq_pack(planes, scales, offsets, q, G, N, K)
    xd = torch.randn((1, K), device="cuda", generator=gen).to(torch.float16)
    Y_ref = torch.empty((1, N), dtype=torch.float16, device="cuda")
    Y = torch.full((1, N), float("nan"), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm(xd, packed, Y_ref, 1, N, K)
    elutq.elutq_lut_gemm_static(xd, packed, Y, 1, N, K)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y_ref)                 # the same kernels, the same order of the chunk sums
    before = elutq.elutq_launch_count()
    assert elutq.lib().elutq_lut_gemm_static(xd.data_ptr(), packed.data_ptr(), Y.data_ptr(), 1, N + 1, K, None) == -4
    assert elutq.elutq_launch_count() == before

    # a small shape right after: the array is full of the large call's partial sums
    layer = workloads.hlq_layer(15, "static/after", 2, 128, 100, 1024)
    small = pack_layer(layer)
    X = synth.activations(15, "static/after/x", 1, 1024)
    Ys = torch.full((1, 100), float("nan"), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm_static(x_dev(X), small, Ys, 1, 100, 1024)
    torch.cuda.synchronize()
    assert hlq.rel_fro_error(Ys.cpu().numpy(), hlq.matmul(X, layer.planes, layer.scales, layer.offsets, 128)) <= TOL_F16
