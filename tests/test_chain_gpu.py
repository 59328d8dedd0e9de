"""GPU parity of the chained decode entry (elutq_chain_plan / elutq_chain_run) against the fp64 oracle.

A chain runs a list of M = 1 calls in one persistent launch; every call must give what the oracle's
definition gives for it (same tolerances as the single-call decode tests: fp32 output <= 5e-6 relative
Frobenius error, fp16 output <= 1e-3), consecutive calls must be ordered like calls on a stream, launches of
one plan must be bit-reproducible, and the two device-side refusals (a hand-over wait that runs out, a blob
whose header no longer matches the plan) must end the launch with a status word instead of a hang or a stray
read.
"""

import numpy as np
import pytest
import torch

import paper_2510_19482_b200 as elutq
import workloads
from oracle import hlq
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import pack_layer, x_dev  # noqa: E402

TOL_F32 = 5e-6
TOL_F16 = 1e-3

# (q, G, N, K): every q, every G, ragged rows, one-chunk layers (no K split), many chunks, several chunks per CTA,
# chunk counts that give one, two and four finisher threads per output row (up to 8, 9-16, more chunks)
SHAPES = [(2, 128, 100, 1024), (3, 128, 333, 1536), (4, 128, 64, 2560), (2, 64, 50, 1088), (1, 32, 17, 96),
          (2, 128, 16, 512), (3, 64, 1000, 4096), (4, 32, 48, 1024), (1, 128, 1, 128), (2, 128, 5000, 4096),
          (2, 128, 40, 512 * 160), (3, 128, 100, 6144), (4, 64, 300, 512 * 20)]


def _elementwise_ok(y, ref, rel):
    scale = np.abs(ref).max() + 1e-30
    return np.all(np.abs(y - ref) <= rel * (np.abs(ref) + scale))


def _build(shapes, seed, tag):
    layers, Xs = [], []
    for i, (q, G, N, K) in enumerate(shapes):
        layers.append(workloads.hlq_layer(seed, f"{tag}/{i}", q, G, N, K, signed_scales=(i % 2 == 1)))
        Xs.append(synth.activations(seed, f"{tag}/x{i}", 1, K))
    return layers, Xs


def test_chain_of_mixed_calls_matches_oracle():
    layers, Xs = _build(SHAPES, 21, "chain-mixed")
    packed = [pack_layer(l) for l in layers]
    xd = [x_dev(x) for x in Xs]
    Y32 = [torch.full((1, l.N), float("nan"), dtype=torch.float32, device="cuda") for l in layers]
    Y16 = [torch.full((1, l.N), float("nan"), dtype=torch.float16, device="cuda") for l in layers]
    calls32 = [(xd[i], packed[i], Y32[i], l.N, l.K, elutq.FLAG_OUT_F32) for i, l in enumerate(layers)]
    calls16 = [(xd[i], packed[i], Y16[i], l.N, l.K, 0) for i, l in enumerate(layers)]
    plan32, plan16 = elutq.elutq_chain_plan(calls32), elutq.elutq_chain_plan(calls16)
    elutq.elutq_chain_run(plan32, len(calls32))
    elutq.elutq_chain_run(plan16, len(calls16))
    assert elutq.elutq_chain_status(plan32) == 0 and elutq.elutq_chain_status(plan16) == 0
    for i, l in enumerate(layers):
        ref = hlq.matmul(Xs[i], l.planes, l.scales, l.offsets, l.G)
        y32, y16 = Y32[i].cpu().numpy(), Y16[i].cpu().numpy()
        assert np.all(np.isfinite(y32)), SHAPES[i]
        assert hlq.rel_fro_error(y32, ref) <= TOL_F32, SHAPES[i]
        assert _elementwise_ok(y32, ref, 2e-5), SHAPES[i]
        assert hlq.rel_fro_error(y16, ref) <= TOL_F16, SHAPES[i]
        assert np.array_equal(y16.view(np.uint16), y32.astype(np.float16).view(np.uint16)), SHAPES[i]


def test_chain_equals_single_calls_bit_for_bit_up_to_eight_chunks():
    # up to 8 chunks both paths add the chunk sums one by one in ascending order
    shapes = [s for s in SHAPES if s[3] <= 4096]
    layers, Xs = _build(shapes, 22, "chain-bits")
    packed = [pack_layer(l) for l in layers]
    xd = [x_dev(x) for x in Xs]
    Yc = [torch.zeros((1, l.N), dtype=torch.float32, device="cuda") for l in layers]
    Ys = [torch.zeros((1, l.N), dtype=torch.float32, device="cuda") for l in layers]
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Yc[i], l.N, l.K, elutq.FLAG_OUT_F32) for i, l in enumerate(layers)])
    elutq.elutq_chain_run(plan, len(layers))
    for i, l in enumerate(layers):
        elutq.elutq_lut_gemm_f32(xd[i], packed[i], Ys[i], 1, l.N, l.K)
    torch.cuda.synchronize()
    for i in range(len(layers)):
        assert torch.equal(Yc[i], Ys[i]), shapes[i]


def test_chain_orders_calls_like_a_stream_and_repeats_bit_for_bit():
    # three layers whose outputs feed the next one: Y0 -> X1 -> ... (fp16 in between, as the entry writes it)
    q, G = 2, 128
    dims = [(1536, 2048), (1024, 1536), (700, 1024)]            # (N, K), K of a layer = N of the one before
    layers = [workloads.hlq_layer(23, f"chain-dep/{i}", q, G, n, k) for i, (n, k) in enumerate(dims)]
    packed = [pack_layer(l) for l in layers]
    X0 = synth.activations(23, "chain-dep/x", 1, dims[0][1])
    bufs = [x_dev(X0)] + [torch.zeros((1, n), dtype=torch.float16, device="cuda") for n, _ in dims]
    calls = [(bufs[i], packed[i], bufs[i + 1], n, k) for i, (n, k) in enumerate(dims)]
    plan = elutq.elutq_chain_plan(calls)
    # oracle: the same pipeline with the intermediate rounded to fp16
    x = X0
    for l in layers:
        y = hlq.matmul(x, l.planes, l.scales, l.offsets, G)
        x = y.astype(np.float16)
    outs = []
    for rep in range(4):
        for b in bufs[1:]:
            b.fill_(float("nan"))
        elutq.elutq_chain_run(plan, len(calls))
        assert elutq.elutq_chain_status(plan) == 0
        outs.append(bufs[-1].cpu().numpy().copy())
        assert np.all(np.isfinite(outs[-1]))
        assert hlq.rel_fro_error(outs[-1], y) <= TOL_F16
        assert np.array_equal(outs[-1].view(np.uint16), outs[0].view(np.uint16))


def test_chain_accumulate_flag_adds_into_y():
    q, G, N, K = 3, 128, 200, 1024
    layer = workloads.hlq_layer(24, "chain-acc", q, G, N, K)
    X = synth.activations(24, "chain-acc/x", 1, K)
    packed = pack_layer(layer)
    Y = torch.ones((1, N), dtype=torch.float32, device="cuda")
    plan = elutq.elutq_chain_plan([(x_dev(X), packed, Y, N, K, elutq.FLAG_OUT_F32 | elutq.FLAG_ACCUMULATE)])
    elutq.elutq_chain_run(plan, 1)
    torch.cuda.synchronize()
    ref = hlq.matmul(X, layer.planes, layer.scales, layer.offsets, G) + 1.0
    assert hlq.rel_fro_error(Y.cpu().numpy(), ref) <= TOL_F32


def test_chain_with_host_buffers_moves_one_arena_per_direction():
    # every call's X in one pinned host arena, every Y in another: one copy in, the launches, one copy out
    shapes = [(2, 128, 300, 1024), (3, 128, 128, 2048), (2, 64, 77, 512)]
    layers, Xs = _build(shapes, 27, "chain-host")
    packed = [pack_layer(l) for l in layers]
    x_off = np.cumsum([0] + [l.K for l in layers])                     # in fp16 elements; K is a multiple of 32
    y_off = np.cumsum([0] + [(l.N + 127) // 128 * 128 for l in layers])
    x_host = torch.empty(int(x_off[-1]), dtype=torch.float16).pin_memory()
    y_host = torch.full((int(y_off[-1]),), float("nan"), dtype=torch.float16).pin_memory()
    for i, X in enumerate(Xs):
        x_host[int(x_off[i]):int(x_off[i + 1])] = torch.from_numpy(X.view(np.int16)).view(torch.float16).reshape(-1)
    x_dev = torch.zeros_like(x_host, device="cuda")
    y_dev = torch.zeros_like(y_host, device="cuda")
    calls = [(x_dev[int(x_off[i]):], packed[i], y_dev[int(y_off[i]):], l.N, l.K) for i, l in enumerate(layers)]
    plan = elutq.elutq_chain_plan(calls)
    elutq.elutq_chain_run_host(plan, len(calls), x_dev, x_host, y_dev, y_host)
    assert elutq.elutq_chain_status(plan) == 0          # (synchronises the stream)
    for i, l in enumerate(layers):
        ref = hlq.matmul(Xs[i], l.planes, l.scales, l.offsets, l.G)
        y = y_host[int(y_off[i]):int(y_off[i]) + l.N].numpy().reshape(1, -1)
        assert hlq.rel_fro_error(y, ref) <= TOL_F16, shapes[i]
    # the same with the calls' Y in pinned host memory themselves: no copy out, bit-identical outputs
    y_host2 = torch.full((int(y_off[-1]),), float("nan"), dtype=torch.float16).pin_memory()
    plan2 = elutq.elutq_chain_plan([(x_dev[int(x_off[i]):], packed[i], y_host2[int(y_off[i]):], l.N, l.K) for i, l in enumerate(layers)])
    elutq.elutq_chain_run_host(plan2, len(calls), x_dev, x_host)
    assert elutq.elutq_chain_status(plan2) == 0
    for i, l in enumerate(layers):
        a, b = int(y_off[i]), int(y_off[i]) + l.N
        assert torch.equal(y_host2[a:b].view(torch.int16), y_host[a:b].view(torch.int16)), shapes[i]
    # Pinned activations are fetched by a kernel that reads them across the bus, pageable ones go through a copy: the
    # same bits either way, also when the run is repeated with other activations and between runs that fetch nothing
    x_alt = (x_host.float() * 0.5).half()
    for rep, xs in enumerate((x_alt, x_host)):
        for pinned in (True, False):
            src = xs.clone().pin_memory() if pinned else xs.clone()
            y_host2.fill_(float("nan"))
            elutq.elutq_chain_run_host(plan2, len(calls), x_dev, src)
            assert elutq.elutq_chain_status(plan2) == 0
            assert torch.equal(x_dev.cpu().view(torch.int16), xs.view(torch.int16))
            elutq.elutq_chain_run(plan2, len(calls))                 # X resident: nothing fetched, same outputs
            assert elutq.elutq_chain_status(plan2) == 0
            if rep == 1:
                for i, l in enumerate(layers):
                    a, b = int(y_off[i]), int(y_off[i]) + l.N
                    assert torch.equal(y_host2[a:b].view(torch.int16), y_host[a:b].view(torch.int16)), (shapes[i], pinned)
    elutq.elutq_chain_forget(plan)
    elutq.elutq_chain_forget(plan2)


def test_a_hand_over_wait_that_runs_out_ends_the_launch_with_a_status():
    # Call 1 reads what call 0 writes, so it waits for call 0's completion count.  Call 0 is planned with the
    # test-only flag that leaves out its completion signal and the poll limit is set to 4096: the wait runs out,
    # the launch returns, the status word says so, and a fresh plan of the same buffers runs correctly
    # afterwards.  Nothing faults and nothing waits without a limit.
    q, G = 2, 128
    dims = [(1024, 1024), (128, 1024)]                      # Y of call 0 is X of call 1
    layers = [workloads.hlq_layer(25, f"chain-exp/{i}", q, G, n, k) for i, (n, k) in enumerate(dims)]
    packed = [pack_layer(l) for l in layers]
    X0 = synth.activations(25, "chain-exp/x0", 1, dims[0][1])
    bufs = [x_dev(X0)] + [torch.zeros((1, n), dtype=torch.float16, device="cuda") for n, _ in dims]
    calls = [(bufs[0], packed[0], bufs[1], dims[0][0], dims[0][1], 0x40000000), (bufs[1], packed[1], bufs[2], dims[1][0], dims[1][1])]
    plan = elutq.elutq_chain_plan(calls)
    elutq.elutq_chain_run_opts(plan, 2, wait_limit=4096)
    assert elutq.elutq_chain_status(plan) == 0x7C05
    good = [(c[0], c[1], c[2], c[3], c[4]) for c in calls]
    elutq.elutq_chain_plan(good, plan=plan)
    elutq.elutq_chain_run(plan, 2)
    assert elutq.elutq_chain_status(plan) == 0
    y0 = hlq.matmul(X0, layers[0].planes, layers[0].scales, layers[0].offsets, G)
    y1 = hlq.matmul(y0.astype(np.float16), layers[1].planes, layers[1].scales, layers[1].offsets, G)
    assert hlq.rel_fro_error(bufs[1].cpu().numpy(), y0) <= TOL_F16
    assert hlq.rel_fro_error(bufs[2].cpu().numpy(), y1) <= TOL_F16


def test_a_blob_that_changed_under_the_plan_is_refused_before_any_tile_is_read():
    # The plan is written for a 4-plane blob; a 2-plane blob of the same (N, K) is then copied over the start of the
    # same allocation (which stays as large as the 4-plane blob, so that even an unguarded kernel would stay inside
    # it).  Every CTA compares the header with the plan first: status 0x7C0B, Y untouched.
    G, N, K = 128, 256, 1024
    big = workloads.hlq_layer(26, "chain-blob/4", 4, G, N, K)
    small = workloads.hlq_layer(26, "chain-blob/2", 2, G, N, K)
    buf = pack_layer(big)
    X = synth.activations(26, "chain-blob/x", 1, K)
    Y = torch.full((1, N), 7.0, dtype=torch.float16, device="cuda")
    plan = elutq.elutq_chain_plan([(x_dev(X), buf, Y, N, K)])
    small_blob = pack_layer(small)
    buf[: small_blob.numel()].copy_(small_blob)
    torch.cuda.synchronize()
    elutq.elutq_chain_run(plan, 1)
    assert elutq.elutq_chain_status(plan) == 0x7C0B
    assert torch.all(Y == 7.0)
    elutq.elutq_forget(buf)


def test_list_of_mixed_bit_widths_is_one_launch_and_equals_the_per_q_kernels_bit_for_bit():
    # G = 128 and q = 1 .. 4 in one list: one launch of the run-time-q instance.  Its look-ups and the order of its
    # additions are those of the per-q instances (which a list of one bit-width takes), so every output must equal,
    # bit for bit, what the same call gives as a chain of its own; small and large row counts, one chunk and many.
    shapes = [(2, 128, 300, 2048), (3, 128, 1000, 4096), (4, 128, 77, 1536), (1, 128, 4096, 512), (2, 128, 6144, 4096),
              (4, 128, 2048, 1024), (3, 128, 33, 7168), (2, 128, 16, 128)]
    layers, Xs = _build(shapes, 29, "chain-rtq")
    packed = [pack_layer(l) for l in layers]
    xd = [x_dev(x) for x in Xs]
    Y = [torch.full((1, l.N), float("nan"), dtype=torch.float32, device="cuda") for l in layers]
    Y1 = [torch.full((1, l.N), float("nan"), dtype=torch.float32, device="cuda") for l in layers]
    plan = elutq.elutq_chain_plan([(xd[i], packed[i], Y[i], l.N, l.K, elutq.FLAG_OUT_F32) for i, l in enumerate(layers)])
    torch.cuda.synchronize()
    n0 = elutq.elutq_launch_count()
    elutq.elutq_chain_run(plan, len(layers))
    assert elutq.elutq_launch_count() - n0 == 1
    assert elutq.elutq_chain_status(plan) == 0
    for i, l in enumerate(layers):
        single = elutq.elutq_chain_plan([(xd[i], packed[i], Y1[i], l.N, l.K, elutq.FLAG_OUT_F32)])
        elutq.elutq_chain_run(single, 1)
        assert elutq.elutq_chain_status(single) == 0
        elutq.elutq_chain_forget(single)
        ref = hlq.matmul(Xs[i], l.planes, l.scales, l.offsets, l.G)
        y = Y[i].cpu().numpy().astype(np.float64)
        assert hlq.rel_fro_error(y, ref) <= TOL_F32, (i, shapes[i])
        assert torch.equal(Y[i].view(torch.int32), Y1[i].view(torch.int32)), (i, shapes[i])
    elutq.elutq_chain_forget(plan)
