"""Randomised plans for the chained decode entry: lists of 4 to 12 calls with mixed bit-widths and group sizes (so
that a plan is cut into several launches, whose hand-overs - completion counters across launches, the reduction a
launch leaves to its successor - are exercised), some calls reading what an earlier call wrote, some accumulating.
Every output is compared with the fp64 oracle applied call by call in list order (intermediates rounded to fp16
where the chain rounds them), and the whole plan is run three times to check that epochs leave nothing behind.
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

TOL_F16 = 1e-3
DIMS = [128, 256, 512, 1024, 1536, 2048, 4096]          # feature sizes the random layers connect (multiples of 128)


LONG_DIMS = [128, 256, 512, 1024, 2048]                 # long lists: small layers (the oracle stays in seconds)


def _random_plan(seed, n_lo=4, n_hi=13, dims=DIMS):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(n_lo, n_hi))
    calls = []
    for i in range(n):
        q = int(rng.integers(1, 5))
        G = int(rng.choice([128, 128, 128, 64, 32]))
        K = int(rng.choice(dims))
        N = int(rng.choice(dims)) - int(rng.choice([0, 0, 0, 3, 17]))        # some ragged row counts
        # with probability 1/3 the call reads the output of an earlier call of matching width
        src = None
        if i > 0 and rng.random() < 0.34:
            cands = [j for j, c in enumerate(calls) if c["N"] == K and not c["f32"]]
            if cands:
                src = int(rng.choice(cands))
        f32 = bool(rng.random() < 0.25)
        acc = bool(rng.random() < 0.2)
        calls.append(dict(q=q, G=G, N=N, K=K, src=src, f32=f32, acc=acc))
    return calls


@pytest.mark.parametrize("seed", list(range(16)))
def test_random_plans_match_the_oracle_call_by_call(seed):
    _check_plan(seed, _random_plan(1000 + seed))


@pytest.mark.parametrize("seed", [100, 101, 102, 103])
def test_long_random_plans_match_the_oracle_call_by_call(seed):
    # 40 to 64 small calls: the scratch regions are reused many times over (a call waits for the reduction of the call
    # that used its region last, six to twelve calls before it), the calls' shares wrap around the CTAs several times, and many calls are in flight side by side
    _check_plan(seed, _random_plan(1000 + seed, 40, 65, LONG_DIMS))


def _check_plan(seed, spec):
    layers = [workloads.hlq_layer(seed, f"chain-rand/{seed}/{i}", c["q"], c["G"], c["N"], c["K"], signed_scales=(i % 3 == 0))
              for i, c in enumerate(spec)]
    packed = [pack_layer(l) for l in layers]
    Xs = [synth.activations(seed, f"chain-rand/{seed}/x{i}", 1, c["K"]) for i, c in enumerate(spec)]
    Y0 = [synth.activations(seed, f"chain-rand/{seed}/y{i}", 1, c["N"]) for i, c in enumerate(spec)]   # initial Y (for accumulate)
    Yd = []
    for i, c in enumerate(spec):
        y0 = torch.from_numpy(Y0[i].view(np.int16)).view(torch.float16)
        Yd.append(y0.float().cuda() if c["f32"] else y0.cuda())
    xd = [Yd[c["src"]] if c["src"] is not None else x_dev(Xs[i]) for i, c in enumerate(spec)]
    calls = []
    for i, c in enumerate(spec):
        flags = (elutq.FLAG_OUT_F32 if c["f32"] else 0) | (elutq.FLAG_ACCUMULATE if c["acc"] else 0)
        calls.append((xd[i], packed[i], Yd[i], c["N"], c["K"], flags))
    plan = elutq.elutq_chain_plan(calls)

    def reference():
        out = []
        for i, c in enumerate(spec):
            x = out[c["src"]].astype(np.float16) if c["src"] is not None else Xs[i]
            y = hlq.matmul(x, layers[i].planes, layers[i].scales, layers[i].offsets, c["G"])
            if c["acc"]:
                y = y + Y0[i].astype(np.float64)
            out.append(y if c["f32"] else y.astype(np.float16).astype(np.float64))
        return out

    ref = reference()
    for rep in range(3):
        for i, c in enumerate(spec):                       # restore the initial contents (accumulating calls add to them)
            y0 = torch.from_numpy(Y0[i].view(np.int16)).view(torch.float16)
            Yd[i].copy_(y0.float() if c["f32"] else y0)
        elutq.elutq_chain_run(plan, len(calls))
        assert elutq.elutq_chain_status(plan) == 0, (seed, rep)
        for i, c in enumerate(spec):
            y = Yd[i].float().cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(y)), (seed, rep, i, c)
            # a call fed by an fp16-rounded intermediate inherits that rounding on both sides; the bound stays the fp16 one
            assert hlq.rel_fro_error(y, ref[i]) <= 2 * TOL_F16, (seed, rep, i, c)
    elutq.elutq_chain_forget(plan)
