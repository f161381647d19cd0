"""CPU oracle for the COMET partition-replacement policy and its auto-tuning rules.

TEST INFRASTRUCTURE ONLY (see dense_oracle.py): only the test-suite may import it; the
product package never does, and this file imports nothing from the product package.

It follows Section 5.1 (two-level partitioning, greedy one-swap sequence of partition sets,
random assignment of edge buckets to partition sets) and Section 6 (Edge Permutation Bias,
rules for p, c and l) in the paper's order and notation.

Points the paper leaves open, and the reading taken here:
  * random grouping of the p physical partitions into l logical ones: physical partitions
    are ordered by a Philox word keyed by (seed, partition) and cut into l consecutive
    groups of p / l (p must be a multiple of l).
  * the one-swap greedy order (the paper cites the greedy algorithm of its predecessor
    and prints none): the first set holds logical partitions 0 .. c_l - 1; every later set
    replaces ONE member e by ONE outside partition a, chosen to maximise the number of
    not-yet-seen pairs {a, x}, x in the set without e; ties go to the smallest a, then to the
    member e that has the fewest unseen pairs left with outside partitions, then to the
    smallest e.  When no swap sees a new pair, the outside partition with the most unseen
    pairs comes in (smallest id on ties) for the member chosen by the same rule.  The
    sequence ends when every pair of logical partitions has shared a set.
  * edge bucket (i, j) (ordered pair of physical partitions, i = j included): among the
    sets that hold both logical partitions, the one numbered
    floor(word * count / 2^32), word = Philox(seed; i, j, 0xB0C4E7, 0)[0].
  * Edge Permutation Bias B under the paper's uniform-degree assumption: all nodes of a
    physical partition share one tally, a bucket (i, j) adds one to the tallies of i and j
    (two for i = j), tallies are normalised by their final value.
  * auto-tuning: p = floor(min(NO / D, sqrt(EO / D))), at least 2 and at most max_parts;
    c = the largest even c <= p with c * PO + 2 * c^2 * EBO + F < CPU such that c / 2 divides
    p (c_l = 2 logical partitions of c / 2 physical ones fill the buffer); l = 2 p / c.
"""
from __future__ import annotations

import math

from oracle.dense_oracle import philox4x32_10, to_range

GROUP_TAG = 0xC0E7
BUCKET_TAG = 0xB0C4E7


def logical_grouping(p: int, l: int, seed: int):
    """logical_of_physical[q] for q in [0, p): random groups of p / l physical partitions."""
    if l <= 0 or p <= 0 or p % l:
        raise ValueError("p must be a positive multiple of l")
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    key = (seed & 0xFFFFFFFF, seed >> 32)
    words = [philox4x32_10((q, 0, GROUP_TAG, 0), key)[0] for q in range(p)]
    order = sorted(range(p), key=lambda q: (words[q], q))
    per = p // l
    out = [0] * p
    for rank, q in enumerate(order):
        out[q] = rank // per
    return out


def greedy_sets(l: int, c_l: int):
    """The sequence S of sets of logical partitions (each a list of c_l ids, in buffer-slot
    order: a swap puts the new partition into the slot of the one it replaces)."""
    if not (2 <= c_l <= l):
        raise ValueError("need 2 <= c_l <= l")
    unseen = {(a, b) for a in range(l) for b in range(a + 1, l)}

    def pair(a, b):
        return (a, b) if a < b else (b, a)

    cur = list(range(c_l))
    for i in range(c_l):
        for j in range(i + 1, c_l):
            unseen.discard(pair(cur[i], cur[j]))
    sets = [list(cur)]
    while unseen:
        outside = [a for a in range(l) if a not in cur]
        left = {x: sum(1 for a in outside if pair(a, x) in unseen) for x in cur}   # what a member still owes
        best = None
        for a in outside:
            for e in cur:
                gain = sum(1 for x in cur if x != e and pair(a, x) in unseen)
                cand = (-gain, a, left[e], e)
                if best is None or cand < best[0]:
                    best = (cand, a, e)
        gain, a, e = -best[0][0], best[1], best[2]
        if gain == 0:
            # nothing new with the current members: bring in the partition that misses the most pairs
            a = min(outside, key=lambda y: (-sum(1 for z in range(l) if z != y and pair(y, z) in unseen), y))
            e = min(cur, key=lambda x: (left[x], x))
        cur[cur.index(e)] = a
        for x in cur:
            if x != a:
                unseen.discard(pair(a, x))
        sets.append(list(cur))
    return sets


def assign_buckets(p: int, logical_of_physical, sets, seed: int):
    """bucket_set[i][j] = index of the partition set that trains edge bucket (i, j)."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    key = (seed & 0xFFFFFFFF, seed >> 32)
    members = [set(s) for s in sets]
    out = [[-1] * p for _ in range(p)]
    for i in range(p):
        for j in range(p):
            li, lj = logical_of_physical[i], logical_of_physical[j]
            cands = [k for k, m in enumerate(members) if li in m and lj in m]
            word = philox4x32_10((i, j, BUCKET_TAG, 0), key)[0]
            out[i][j] = cands[to_range(word, len(cands))]
    return out


def comet_plan(p: int, l: int, c_l: int, seed: int):
    grouping = logical_grouping(p, l, seed)
    sets = greedy_sets(l, c_l)
    return {"logical_of_physical": grouping, "sets": sets,
            "bucket_set": assign_buckets(p, grouping, sets, seed)}


def physical_sets(plan):
    """Each S_i as the ascending list of physical partitions it holds."""
    lop = plan["logical_of_physical"]
    return [sorted(q for q in range(len(lop)) if lop[q] in s) for s in plan["sets"]]


def edge_permutation_bias(p: int, n_sets: int, bucket_set):
    """B = max_i max_{v1, v2} (t_i^{v1} - t_i^{v2}) with per-partition tallies (Section 6)."""
    total = [0] * p
    per_set = [[0] * p for _ in range(n_sets)]
    for i in range(p):
        for j in range(p):
            k = bucket_set[i][j]
            per_set[k][i] += 1
            per_set[k][j] += 1
            total[i] += 1
            total[j] += 1
    tally = [0] * p
    bias = 0.0
    for k in range(n_sets):
        for q in range(p):
            tally[q] += per_set[k][q]
        t = [tally[q] / total[q] for q in range(p)]
        bias = max(bias, max(t) - min(t))
    return bias


def autotune(n_nodes: int, dim: int, n_edges: int, bytes_per_edge: int, cpu_bytes: int, block_bytes: int,
             fudge_bytes: int, max_parts: int):
    """(p, l, c) by the rules of Section 6."""
    node_overhead = n_nodes * dim * 4
    edge_overhead = n_edges * bytes_per_edge
    alpha4 = min(node_overhead / block_bytes, math.sqrt(edge_overhead / block_bytes))
    p = max(2, min(int(math.floor(alpha4)), max_parts))
    part_overhead = node_overhead / p
    bucket_overhead = edge_overhead / (p * p)
    best = None
    for c in range(2, p + 1, 2):
        if c * part_overhead + 2 * c * c * bucket_overhead + fudge_bytes < cpu_bytes and p % (c // 2) == 0:
            best = c
    if best is None:
        raise ValueError("no buffer capacity fits the memory")
    return p, 2 * p // best, best
