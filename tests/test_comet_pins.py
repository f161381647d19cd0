"""Pins for the COMET oracle (Section 5.1, Section 6): invariants the paper states, bounds, brute force on small
cases, closed forms -- and, at the end, the library's native implementation against the oracle, value by value."""
import itertools
import math

import numpy as np
import pytest

from oracle import comet_oracle as C


def _pairs_seen(sets):
    seen = set()
    for s in sets:
        seen |= {tuple(sorted(x)) for x in itertools.combinations(s, 2)}
    return seen


@pytest.mark.parametrize("l,c_l", [(2, 2), (5, 2), (8, 2), (9, 3), (12, 4), (16, 2), (7, 7)])
def test_greedy_sets_cover_every_pair_one_swap_at_a_time(l, c_l):
    sets = C.greedy_sets(l, c_l)
    assert sets[0] == list(range(c_l))
    assert _pairs_seen(sets) == {(a, b) for a in range(l) for b in range(a + 1, l)}
    for a, b in zip(sets, sets[1:]):
        assert len(a) == len(b) == c_l and len(set(b)) == c_l
        assert sum(x != y for x, y in zip(a, b)) == 1          # one logical partition swapped, in place
    # every swap but the rare zero-gain one sees a new pair, and a swap sees at most c_l - 1 of them
    lower = 1 + math.ceil((l * (l - 1) // 2 - c_l * (c_l - 1) // 2) / (c_l - 1))
    assert lower <= len(sets) <= lower + l * (l - 1) // 2 // 2 + 2


def _shortest_cover(l, c_l):
    """Fewest sets of any one-swap sequence from {0..c_l-1} that covers all pairs (breadth-first search)."""
    all_pairs = frozenset((a, b) for a in range(l) for b in range(a + 1, l))
    start = frozenset(range(c_l))
    seen0 = frozenset(tuple(sorted(x)) for x in itertools.combinations(start, 2))
    frontier = {(start, seen0)}
    n = 1
    while True:
        if any(seen == all_pairs for _, seen in frontier):
            return n
        nxt = set()
        for cur, seen in frontier:
            for e in cur:
                for a in range(l):
                    if a in cur:
                        continue
                    new = (cur - {e}) | {a}
                    nxt.add((new, seen | frozenset(tuple(sorted((a, x))) for x in new if x != a)))
        frontier = nxt
        n += 1


@pytest.mark.parametrize("l,c_l", [(3, 2), (4, 2), (5, 2), (5, 3), (6, 3)])
def test_greedy_sets_are_near_the_shortest_sequence(l, c_l):
    assert len(C.greedy_sets(l, c_l)) <= _shortest_cover(l, c_l) + 1


def test_grouping_is_a_balanced_random_partition():
    p, l = 24, 6
    counts = np.zeros((p, l))
    for seed in range(600):
        g = C.logical_grouping(p, l, seed)
        assert sorted(np.bincount(g, minlength=l).tolist()) == [p // l] * l
        for q, lg in enumerate(g):
            counts[q, lg] += 1
    expect = 600 / l
    chi2 = ((counts - expect) ** 2 / expect).sum()
    assert chi2 < 24 * 5 + 6 * math.sqrt(2 * 24 * 5)          # p (l - 1) degrees of freedom, six sigma
    assert C.logical_grouping(p, l, 1) != C.logical_grouping(p, l, 2)
    with pytest.raises(ValueError):
        C.logical_grouping(10, 4, 0)


def test_bucket_assignment_is_valid_uniform_and_balanced():
    p, l, c_l = 12, 6, 3
    hits = {}
    loads = []
    for seed in range(300):
        plan = C.comet_plan(p, l, c_l, seed)
        lop, sets, bs = plan["logical_of_physical"], plan["sets"], plan["bucket_set"]
        load = np.zeros(len(sets))
        for i in range(p):
            for j in range(p):
                k = bs[i][j]
                assert lop[i] in sets[k] and lop[j] in sets[k]
                load[k] += 1
                cands = tuple(x for x, s in enumerate(sets) if lop[i] in s and lop[j] in s)
                hits.setdefault((len(cands), cands.index(k)), 0)
                hits[(len(cands), cands.index(k))] += 1
        loads.append(load)
    # the choice among n candidates is uniform: for every n, the positions are hit equally often
    by_n = {}
    for (n, pos), h in hits.items():
        by_n.setdefault(n, np.zeros(n))[pos] += h
    for n, v in by_n.items():
        if n > 1 and v.sum() > 500:
            expect = v.sum() / n
            assert ((v - expect) ** 2 / expect).sum() < (n - 1) + 6 * math.sqrt(2 * (n - 1)) + 6
    # deferred processing balances the sets (Section 5.1): no set is left (nearly) empty on average
    mean_load = np.mean(loads, axis=0)
    assert mean_load.min() > 0.3 * mean_load.mean()


def test_edge_permutation_bias_closed_forms_and_greedy_comparison():
    # one set: every tally reaches 1 at once
    assert C.edge_permutation_bias(3, 1, [[0] * 3 for _ in range(3)]) == 0.0
    # two partitions, three sets: bucket (0,0) first, (1,1) last -> after set 0 partition 0 has 2 of its 4 counts
    bs = [[0, 1], [1, 2]]
    assert C.edge_permutation_bias(2, 3, bs) == pytest.approx(0.5)
    # processing every bucket as soon as its two partitions meet (the greedy policies of Section 5.1) front-loads
    # the epoch; the random deferred assignment spreads the buckets over the sets that can train them (Section 5.1:
    # balanced workloads) and is never more biased, on the same sequence of sets
    p, l, c_l = 24, 12, 4
    for seed in range(12):
        plan = C.comet_plan(p, l, c_l, seed)
        lop, sets = plan["logical_of_physical"], plan["sets"]
        first = [[min(k for k, s in enumerate(sets) if lop[i] in s and lop[j] in s) for j in range(p)] for i in range(p)]
        b_rand = C.edge_permutation_bias(p, len(sets), plan["bucket_set"])
        b_first = C.edge_permutation_bias(p, len(sets), first)
        assert 0.0 <= b_rand <= b_first + 1e-12 <= 1.0 + 1e-12
        load_rand = np.bincount(np.array(plan["bucket_set"]).ravel(), minlength=len(sets))
        load_first = np.bincount(np.array(first).ravel(), minlength=len(sets))
        assert load_rand.sum() == load_first.sum() == p * p
        assert load_rand.max() < 0.8 * load_first.max()


def test_autotune_rules():
    # NO = 1e6 * 100 * 4 = 4e8, EO = 5e7 * 12 = 6e8, D = 1e6: alpha4 = min(400, sqrt(600) = 24.49) -> p = 24
    # PO = 4e8 / 24 = 1.667e7, EBO = 6e8 / 576 = 1.0417e6; CPU = 3e8, F = 5e7:
    # c = 8: 1.333e8 + 2 * 64 * 1.0417e6 = 2.667e8 (+F = 3.167e8) too much; c = 6: 1e8 + 7.5e7 + 5e7 = 2.25e8 fits,
    # and c / 2 = 3 divides 24 -> c = 6, l = 2 * 24 / 6 = 8
    assert C.autotune(1_000_000, 100, 50_000_000, 12, 300_000_000, 1_000_000, 50_000_000, 1024) == (24, 8, 6)
    # the node term can be the smaller one, and max_parts caps p
    p, l, c = C.autotune(1000, 10, 10**9, 12, 10**12, 1000, 0, 1024)
    assert p == 40 and c == 40 and l == 2                      # NO / D = 40; everything fits
    assert C.autotune(10**8, 100, 10**9, 12, 10**12, 4096, 0, 64)[0] == 64
    for args in [(86_000_000, 100, 338_000_000, 12, 60 * 2**30, 2**20, 8 * 2**30, 4096),
                 (1_000_000, 64, 20_000_000, 8, 2**28, 2**16, 2**24, 256)]:
        p, l, c = C.autotune(*args)
        no, eo = args[0] * args[1] * 4, args[2] * args[3]
        fits = lambda cc: cc * no / p + 2 * cc * cc * eo / (p * p) + args[6] < args[4]
        assert fits(c) and c % 2 == 0 and p % (c // 2) == 0 and l * c == 2 * p
        assert not any(fits(cc) and p % (cc // 2) == 0 for cc in range(c + 2, p + 1, 2))   # c is maximal
    with pytest.raises(ValueError):
        C.autotune(10**9, 1000, 10**9, 12, 1000, 4096, 0, 64)


# ---------------------------------------------------------------- the library's native planner against the oracle
@pytest.mark.parametrize("p,l,c_l,seed", [(2, 2, 2, 0), (12, 6, 3, 1), (16, 8, 2, 2), (24, 12, 4, 3), (32, 8, 8, 4), (30, 15, 2, 5),
                                          (64, 16, 4, 2**63 + 11)])
def test_native_plan_equals_oracle(p, l, c_l, seed):
    import paper_2202_02365_b200 as mg
    got = mg.comet_plan(p, l, c_l, seed)
    ref = C.comet_plan(p, l, c_l, seed)
    assert got["logical_of_physical"].tolist() == ref["logical_of_physical"]
    assert got["sets"].tolist() == ref["sets"]
    assert got["bucket_set"].tolist() == ref["bucket_set"]
    assert got["physical_sets"] == C.physical_sets(ref)
    assert mg.comet_bias(got["bucket_set"], len(ref["sets"])) == pytest.approx(
        C.edge_permutation_bias(p, len(ref["sets"]), ref["bucket_set"]), abs=1e-15)


def test_native_autotune_and_errors():
    import paper_2202_02365_b200 as mg
    for args in [(1_000_000, 100, 50_000_000, 12, 300_000_000, 1_000_000, 50_000_000, 1024),
                 (1000, 10, 10**9, 12, 10**12, 1000, 0, 1024), (10**8, 100, 10**9, 12, 10**12, 4096, 0, 64),
                 (86_000_000, 100, 338_000_000, 12, 60 * 2**30, 2**20, 8 * 2**30, 4096)]:
        assert mg.comet_autotune(*args) == C.autotune(*args)
    with pytest.raises(mg.MgError) as e:
        mg.comet_autotune(10**9, 1000, 10**9, 12, 1000, 4096, 0, 64)
    assert e.value.code == -5
    for bad in [(10, 4, 2), (8, 4, 1), (8, 4, 5), (0, 1, 1)]:
        with pytest.raises(mg.MgError) as e:
            mg.comet_plan(*bad, 0)
        assert e.value.code == -1
