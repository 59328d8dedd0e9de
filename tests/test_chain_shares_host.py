"""Host logic of the chained decode entry's plan, without a GPU: how one call is cut over the CTAs of a launch.

Invariants checked for the benchmark's layer shapes and a sweep of others: every (row block, chunk) of the call
belongs to exactly one CTA's share; a share is a row-block range of one chunk group; the shares begin at the CTA the
caller names and wrap around; a CTA without a share is all zeros; a small call that is independent of its neighbours
gets two rounds of items per look-up warp (26 per CTA) instead of being spread over every CTA, a dependent one does
not.
"""

import itertools

import pytest

import paper_2510_19482_b200 as elutq

SMS = 148
LOOKUP_WARPS = 26
SHAPES = [(4096, 4096), (6144, 4096), (28672, 4096), (4096, 14336), (10240, 8192), (8192, 8192), (57344, 8192),
          (8192, 28672), (16, 128), (17, 96), (100, 1024), (333, 1536), (5000, 4096), (40, 512 * 160), (1, 128)]


def _cover(shares, n_rb, n_kc):
    seen = {}
    for cta, (rb0, rb1, kc0, nseg, grp) in enumerate(shares):
        if nseg == 0:
            assert (rb0, rb1, kc0, grp) == (0, 0, 0, 0), cta
            continue
        assert 0 <= rb0 < rb1 <= n_rb and 0 <= kc0 and kc0 + nseg <= n_kc, (cta, rb0, rb1, kc0, nseg)
        for rb, kc in itertools.product(range(rb0, rb1), range(kc0, kc0 + nseg)):
            assert (rb, kc) not in seen, (cta, seen[(rb, kc)], rb, kc)
            seen[(rb, kc)] = cta
    return seen


@pytest.mark.parametrize("N,K", SHAPES)
@pytest.mark.parametrize("independent", [True, False])
def test_every_item_of_a_call_belongs_to_exactly_one_cta(N, K, independent):
    n_rb, n_kc = (N + 15) // 16, (K + 511) // 512
    shares, (cpc, ranges, groups, n_ctas) = elutq.elutq_chain_shares(N, K, SMS, 0, independent)
    seen = _cover(shares, n_rb, n_kc)
    assert len(seen) == n_rb * n_kc
    assert n_ctas == groups * ranges <= SMS and groups == -(-n_kc // cpc)
    assert sum(1 for s in shares if s[3]) == n_ctas
    # a share is one chunk group (chunks grp * cpc ...) and the shares of a group tile the row blocks in order
    for rb0, rb1, kc0, nseg, grp in shares:
        if nseg:
            assert kc0 == grp * cpc and nseg == min(cpc, n_kc - kc0)
    for g in range(groups):
        rows = sorted((s[0], s[1]) for s in shares if s[3] and s[4] == g)
        assert rows[0][0] == 0 and rows[-1][1] == n_rb and all(a[1] == b[0] for a, b in zip(rows, rows[1:]))
        sizes = [b - a for a, b in rows]
        assert max(sizes) - min(sizes) <= 1                       # balanced ranges


@pytest.mark.parametrize("N,K", [(4096, 4096), (6144, 4096), (28672, 4096), (100, 1024)])
@pytest.mark.parametrize("first", [0, 1, 40, 147, 148 + 5])
def test_shares_begin_at_the_named_cta_and_wrap_around(N, K, first):
    base, part = elutq.elutq_chain_shares(N, K, SMS, 0, True)
    rot, part2 = elutq.elutq_chain_shares(N, K, SMS, first, True)
    assert part == part2
    for cta in range(SMS):
        assert rot[(cta + first) % SMS] == base[cta]


def test_small_independent_calls_take_two_rounds_of_items_per_lookup_warp():
    for N, K in [(4096, 4096), (6144, 4096)]:
        n_rb = N // 16
        ind, (cpc_i, ranges_i, groups_i, n_i) = elutq.elutq_chain_shares(N, K, SMS, 0, True)
        dep, (cpc_d, ranges_d, groups_d, n_d) = elutq.elutq_chain_shares(N, K, SMS, 0, False)
        assert cpc_i == cpc_d == 1 and groups_i == groups_d
        assert ranges_i == -(-n_rb // (2 * LOOKUP_WARPS)) < ranges_d            # fewer CTAs, ...
        assert max(s[1] - s[0] for s in ind if s[3]) <= 2 * LOOKUP_WARPS          # ... at most two rounds of items each
        assert n_d > SMS - groups_d                                               # the dependent form fills the launch
    # a large layer is cut the same way either way
    assert elutq.elutq_chain_shares(28672, 4096, SMS, 0, True) == elutq.elutq_chain_shares(28672, 4096, SMS, 0, False)


def test_argument_checks_and_long_rows_on_few_ctas():
    with pytest.raises(Exception):
        elutq.elutq_chain_shares(0, 128, SMS)
    with pytest.raises(Exception):
        elutq.elutq_chain_shares(16, 128, 0)
    # more chunks than 8 per CTA would cover: a CTA then takes as many chunks as it must
    shares, (cpc, ranges, groups, n_ctas) = elutq.elutq_chain_shares(16, 512 * 200, 8)
    assert n_ctas <= 8 and cpc * groups >= 200 and len(_cover(shares, 1, 200)) == 200
