"""Pins for the CPU oracle: each check ties it to something other than itself —
published known-answer vectors, the paper's worked example, brute force on tiny
graphs, closed forms, whole-graph linear algebra, library routines."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import dense_oracle as O
from paper_2202_02365_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _fields(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":", 1)
        out[key.strip()] = val.strip()
    return out


def _ints(s):
    return [int(x) for x in s.split()]


def _csr_from_edges(n, edges):
    rows = [[] for _ in range(n)]
    for s, d in edges:
        rows[d].append(s)
    off, nb = [0], []
    for r in rows:
        nb.extend(sorted(r))
        off.append(len(nb))
    return np.array(off), np.array(nb, dtype=np.int64)


def _random_graph(n, m, seed):
    g = inputs.erdos_renyi_graph(n, m, seed)
    return g.row_offsets.numpy(), g.nbrs.numpy().astype(np.int64)


# ---------------------------------------------------------------- Philox
def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert list(O.philox4x32_10(w[0:4], w[4:6])) == w[6:10]
        n += 1
    assert n == 3


def test_draw_word_keying():
    # word t of a block is output (t % 4) of counter (node, 0, hop, t // 4)
    blk = O.philox4x32_10((12345, 0, 2, 1), (0xDEADBEEF, 0x1234))
    seed = (0x1234 << 32) | 0xDEADBEEF
    assert [O.draw_word(seed, 12345, 2, 4 + i) for i in range(4)] == list(blk)
    # every key component matters
    base = O.draw_word(seed, 12345, 2, 5)
    assert len({base, O.draw_word(seed + 1, 12345, 2, 5), O.draw_word(seed, 12346, 2, 5),
                O.draw_word(seed, 12345, 1, 5), O.draw_word(seed, 12345, 2, 6),
                O.draw_word(seed ^ (1 << 40), 12345, 2, 5)}) == 6


def test_to_range_is_floor_of_scaled_word():
    for w, n in [(0, 7), (0xFFFFFFFF, 7), (0x80000000, 10), (0x12345678, 1000003)]:
        assert O.to_range(w, n) == int(np.floor(w / 2.0**32 * n))
        assert 0 <= O.to_range(w, n) < n


# ---------------------------------------------------------------- one-hop sample
def test_small_degree_returns_whole_row():
    row = [4, 9, 9, 17]
    for f in (4, 5, 100):
        assert O.one_hop_sample(row, f, 1, 3, 0) == row


def test_large_degree_returns_f_distinct_positions_in_order():
    row = list(range(100, 160))       # distinct values -> positions are recoverable
    for f in (1, 2, 7, 31, 33, 59):
        for node in range(20):
            s = O.one_hop_sample(row, f, 99, node, 1)
            assert len(s) == f
            assert len(set(s)) == f
            assert s == sorted(s)
            assert set(s) <= set(row)


def test_sample_depends_only_on_its_key():
    row = list(range(50))
    a = O.one_hop_sample(row, 5, 7, 11, 0)
    assert a == O.one_hop_sample(row, 5, 7, 11, 0)
    others = [O.one_hop_sample(row, 5, 8, 11, 0), O.one_hop_sample(row, 5, 7, 12, 0),
              O.one_hop_sample(row, 5, 7, 11, 1)]
    assert any(o != a for o in others)


def test_inclusion_is_uniform():
    # every position is kept with probability f/d, every pair with f(f-1)/(d(d-1))
    d, f, trials = 12, 4, 6000
    row = list(range(d))
    single = np.zeros(d)
    pair = np.zeros((d, d))
    for node in range(trials):
        s = O.one_hop_sample(row, f, 2024, node, 0)
        for x in s:
            single[x] += 1
        for x, y in itertools.combinations(s, 2):
            pair[x, y] += 1
    exp = trials * f / d
    chi2 = ((single - exp) ** 2 / exp).sum()
    assert chi2 < 35.0                      # 11 dof, p ~ 2e-4
    exp2 = trials * f * (f - 1) / (d * (d - 1))
    vals = pair[np.triu_indices(d, 1)]
    chi2p = ((vals - exp2) ** 2 / exp2).sum()
    assert chi2p < 120.0                    # 65 dof, p ~ 4e-5


def test_all_subsets_reachable_tiny():
    # d = 5, f = 2: all 10 subsets appear, about equally often
    seen = {}
    for node in range(4000):
        s = tuple(O.one_hop_sample([0, 1, 2, 3, 4], 2, 5, node, 0))
        seen[s] = seen.get(s, 0) + 1
    assert len(seen) == 10
    assert min(seen.values()) > 300 and max(seen.values()) < 500


# ---------------------------------------------------------------- Algorithm 1
def test_worked_example_layout():
    g = _fields(os.path.join(GOLD, "dense_worked_example.txt"))
    edges = [tuple(_ints(e)) for e in g["edges"].split(",")]
    off, nb = _csr_from_edges(5, edges)
    d = O.sample_dense(O.GraphView(off, nb), _ints(g["targets"]), _ints(g["fanouts"]), seed=0)
    for key in ("node_ids", "node_id_offsets", "nbrs", "nbr_offsets", "repr_map"):
        assert d[key] == _ints(g[key]), key
    u = O.update_dense(d)
    assert u["node_ids"] == _ints(g["after_layer1_node_ids"])
    assert u["nbrs"] == _ints(g["after_layer1_nbrs"])
    assert u["repr_map"] == _ints(g["after_layer1_repr_map"])
    assert u["nbr_offsets"] == _ints(g["after_layer1_nbr_offsets"])
    assert u["node_id_offsets"] == _ints(g["after_layer1_node_id_offsets"])


def _bfs_levels(off, nb, targets, k, allowed=None):
    seen = set(targets)
    levels = [list(targets)]
    frontier = list(targets)
    for _ in range(k):
        nxt = set()
        for v in frontier:
            for u in nb[off[v]:off[v + 1]]:
                u = int(u)
                if (allowed is None or u in allowed) and u not in seen:
                    nxt.add(u)
        seen |= nxt
        frontier = sorted(nxt)
        levels.append(frontier)
    return levels


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_full_fanout_gives_bfs_levels(seed):
    off, nb = _random_graph(60, 150, seed)
    maxdeg = int(np.diff(off).max())
    targets = [5, 17, 3]
    k = 3
    d = O.sample_dense(O.GraphView(off, nb), targets, [maxdeg] * k, seed=4)
    levels = _bfs_levels(off, nb, targets, k)
    nio = d["node_id_offsets"]
    for j in range(k + 1):                       # Delta_{k-j} = BFS level j
        i = k - j
        assert d["node_ids"][nio[i]:nio[i + 1]] == levels[j]
    # every sampled node carries its exact neighbourhood
    sampled = d["node_ids"][nio[1]:]
    for r, v in enumerate(sampled):
        got = d["nbrs"][d["nbr_offsets"][r]:d["nbr_offsets"][r + 1]]
        assert got == [int(u) for u in nb[off[v]:off[v + 1]]]


def _memoised_khop(view, targets, fanouts, seed):
    """Ordinary layer-by-layer k-hop sampling over the *whole* frontier, with a
    node's one-hop sample remembered from the first hop that needed it."""
    memo = {}
    known = list(targets)
    for hop, f in enumerate(fanouts):
        for v in list(known):
            if v not in memo:
                memo[v] = O.one_hop_sample(view.row(v), f, seed, v, hop)
        for v in list(known):
            for u in memo[v]:
                if u not in known:
                    known.append(u)
    return memo, set(known)


@pytest.mark.parametrize("seed", [0, 3])
def test_delta_sampling_equals_memoised_full_frontier_sampling(seed):
    off, nb = _random_graph(200, 1600, seed)
    view = O.GraphView(off, nb)
    targets = [1, 50, 7, 120, 33]
    fanouts = [4, 3, 2]
    d = O.sample_dense(view, targets, fanouts, seed=11)
    memo, known = _memoised_khop(view, targets, fanouts, 11)
    assert set(d["node_ids"]) == known
    assert len(d["node_ids"]) == len(known)                      # no duplicates
    nio = d["node_id_offsets"]
    sampled = d["node_ids"][nio[1]:]
    assert set(sampled) == set(memo)                             # sampled exactly once each
    for r, v in enumerate(sampled):
        assert d["nbrs"][d["nbr_offsets"][r]:d["nbr_offsets"][r + 1]] == memo[v]
    # a node's fanout is that of the first hop that needed it
    k = len(fanouts)
    for i in range(1, k + 1):
        f = fanouts[k - i]
        for r in range(nio[i] - nio[1], nio[i + 1] - nio[1]):
            v = sampled[r]
            deg = off[v + 1] - off[v]
            assert d["nbr_offsets"][r + 1] - d["nbr_offsets"][r] == min(deg, f)
    # each delta ascending (targets keep caller order)
    for i in range(k):
        seg = d["node_ids"][nio[i]:nio[i + 1]]
        assert seg == sorted(seg)
    assert d["node_ids"][nio[k]:] == targets
    # repr_map points at the right rows, and never before the delta it may use
    for e, r in enumerate(d["repr_map"]):
        assert d["node_ids"][r] == d["nbrs"][e]


def test_neighbours_of_delta_j_live_in_later_rows():
    # neighbours of Delta_j lie in Delta_{j-1} .. Delta_k, so Algorithm 2's shift
    # of repr_map never goes negative
    off, nb = _random_graph(300, 3000, 5)
    d = O.sample_dense(O.GraphView(off, nb), list(range(0, 40, 2)), [3, 3, 3], seed=1)
    cur = d
    for _ in range(2):
        cur = O.update_dense(cur)
        assert min(cur["repr_map"]) >= 0
        for e, r in enumerate(cur["repr_map"]):
            assert cur["node_ids"][r] == cur["nbrs"][e]
        assert cur["nbr_offsets"][0] == 0 and cur["node_id_offsets"][0] == 0
        assert cur["nbr_offsets"][-1] == len(cur["nbrs"])
        assert cur["node_id_offsets"][-1] == len(cur["node_ids"])


def test_input_errors():
    off, nb = _random_graph(20, 40, 0)
    v = O.GraphView(off, nb, n_parts=4, resident_parts=[0, 1])
    with pytest.raises(ValueError):
        O.sample_dense(v, [1, 1], [2], 0)
    with pytest.raises(ValueError):
        O.sample_dense(v, [19], [2], 0)           # partition 3 is not resident
    with pytest.raises(ValueError):
        O.sample_dense(v, [20], [2], 0)


# ---------------------------------------------------------------- in-buffer filter
@pytest.mark.parametrize("resident", [[0, 2], [1, 2, 3], [3]])
def test_buffer_filter_equals_sampling_the_induced_subgraph(resident):
    n, parts = 120, 4
    off, nb = _random_graph(n, 1500, 9)
    size = (n + parts - 1) // parts
    res = lambda u: (u // size) in resident
    # induced subgraph built edge by edge
    edges = [(int(u), v) for v in range(n) for u in nb[off[v]:off[v + 1]] if res(int(u)) and res(v)]
    off2, nb2 = _csr_from_edges(n, edges)
    targets = [v for v in range(n) if res(v)][::7]
    a = O.sample_dense(O.GraphView(off, nb, parts, resident), targets, [3, 2], seed=5)
    b = O.sample_dense(O.GraphView(off2, nb2), targets, [3, 2], seed=5)
    assert a == b
    assert all(res(u) for u in a["node_ids"])
    # with full fanout: BFS levels of the resident subgraph only
    maxdeg = int(np.diff(off).max())
    c = O.sample_dense(O.GraphView(off, nb, parts, resident), targets[:3], [maxdeg] * 2, seed=5)
    lv = _bfs_levels(off, nb, targets[:3], 2, allowed={u for u in range(n) if res(u)})
    nio = c["node_id_offsets"]
    assert c["node_ids"][nio[0]:nio[1]] == lv[2] and c["node_ids"][nio[1]:nio[2]] == lv[1]


def test_partition_id_array():
    """GraphView with one partition id per node (Section 5.2: training nodes in the first partitions, the rest at
    random): (a) the array that spells out the contiguous split changes nothing; (b) under any array the filter equals
    sampling the explicitly induced subgraph; (c) resident nodes are counted partition after partition, ascending id
    inside a partition, and negatives are drawn from exactly those; (d) the policy's array keeps every training node
    resident while only the first partitions are in the buffer."""
    n, parts = 120, 4
    off, nb = _random_graph(n, 1500, 9)
    size = (n + parts - 1) // parts
    same = np.arange(n) // size
    for resident in ([0, 2], [1, 2, 3]):
        targets = [v for v in range(n) if v // size in resident][::7]
        a = O.sample_dense(O.GraphView(off, nb, parts, resident), targets, [3, 2], seed=5)
        b = O.sample_dense(O.GraphView(off, nb, parts, resident, part_of_node=same), targets, [3, 2], seed=5)
        assert a == b
        assert (O.lp_negatives(O.GraphView(off, nb, parts, resident), 2, 50, 3)
                == O.lp_negatives(O.GraphView(off, nb, parts, resident, part_of_node=same), 2, 50, 3))
    rng = np.random.default_rng(3)
    pn = rng.integers(0, parts, n)
    for resident in ([0, 2], [3], [0, 1, 3]):
        res = lambda u: pn[u] in resident
        edges = [(int(u), v) for v in range(n) for u in nb[off[v]:off[v + 1]] if res(int(u)) and res(v)]
        off2, nb2 = _csr_from_edges(n, edges)
        view = O.GraphView(off, nb, parts, resident, part_of_node=pn)
        targets = [v for v in range(n) if res(v)][::5]
        assert O.sample_dense(view, targets, [3, 2], seed=5) == O.sample_dense(O.GraphView(off2, nb2), targets, [3, 2], seed=5)
        with pytest.raises(ValueError):
            O.sample_dense(view, [next(v for v in range(n) if not res(v))], [2], 0)
        want = [v for p in sorted(resident) for v in range(n) if pn[v] == p]
        assert view.resident_nodes() == want and view.n_resident_nodes() == len(want)
        assert [view.resident_node_at(i) for i in range(len(want))] == want
        negs = O.lp_negatives(view, 3, 400, seed=8)
        assert all(res(u) for row in negs for u in row)
        counts = np.bincount([want.index(u) for row in negs for u in row], minlength=len(want))
        expect = 1200 / len(want)
        assert ((counts - expect) ** 2 / expect).sum() < 2.0 * len(want)          # uniform over the resident nodes
    train = torch.randperm(n, generator=torch.Generator().manual_seed(1))[:50]
    policy = inputs.training_first_partitioning(n, parts, train, seed=2).numpy()
    k_train = (50 + size - 1) // size
    assert set(policy[train.numpy()].tolist()) == set(range(k_train))
    rest = np.setdiff1d(np.arange(n), train.numpy())
    assert set(policy[rest].tolist()) <= set(range(k_train, parts)) and len(set(policy[rest].tolist())) == parts - k_train
    view = O.GraphView(off, nb, parts, list(range(k_train)), part_of_node=policy)
    assert all(view.is_resident(int(t)) for t in train)
    d = O.sample_dense(view, train.tolist()[:10], [4, 4], seed=1)
    assert all(policy[u] < k_train for u in d["node_ids"])


# ---------------------------------------------------------------- forward
def test_hand_computed_means():
    g = _fields(os.path.join(GOLD, "dense_worked_example.txt"))
    hm = _fields(os.path.join(GOLD, "hand_means.txt"))
    edges = [tuple(_ints(e)) for e in g["edges"].split(",")]
    off, nb = _csr_from_edges(5, edges)
    d = O.sample_dense(O.GraphView(off, nb), _ints(g["targets"]), [10, 10], seed=0)
    h0 = np.array([float(x) for x in hm["h0"].split()]).reshape(5, 2)
    layer = (np.eye(2), 2 * np.eye(2), np.array([0.5, -0.5]))
    outs = O.forward(d, h0, [layer, layer], return_all=True)
    np.testing.assert_allclose(outs[0].ravel(), [float(x) for x in hm["layer1"].split()], rtol=0, atol=1e-12)
    np.testing.assert_allclose(outs[1].ravel(), [float(x) for x in hm["layer2"].split()], rtol=0, atol=1e-12)


def _whole_graph_sage(off, nb, feats, layers):
    """GraphSage-mean on every node of the graph with dense adjacency algebra."""
    n = len(off) - 1
    a = np.zeros((n, n))
    for v in range(n):
        for u in nb[off[v]:off[v + 1]]:
            a[v, int(u)] += 1.0                   # multi-edges count
    deg = a.sum(1, keepdims=True)
    a_mean = np.divide(a, deg, out=np.zeros_like(a), where=deg > 0)
    h = feats.astype(np.float64)
    for i, (ws, wn, b) in enumerate(layers):
        h = h @ ws.astype(np.float64) + (a_mean @ h) @ wn.astype(np.float64) + b.astype(np.float64)
        if i + 1 < len(layers):
            h = np.maximum(h, 0)
    return h


@pytest.mark.parametrize("k", [1, 2, 3])
def test_full_fanout_forward_equals_whole_graph_graphsage(k):
    off, nb = _random_graph(80, 400, 21)
    rng = np.random.default_rng(0)
    feats = rng.standard_normal((80, 6))
    dims = [6, 5, 4, 3][:k + 1]
    layers = [(w.numpy(), n_.numpy(), b.numpy()) for w, n_, b in inputs.random_bias_layers(dims, 3)]
    targets = [9, 2, 40, 77, 31]
    maxdeg = int(np.diff(off).max())
    d = O.sample_dense(O.GraphView(off, nb), targets, [maxdeg] * k, seed=0)
    out = O.forward(d, feats[d["node_ids"]], layers)
    ref = _whole_graph_sage(off, nb, feats, layers)[targets]
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-12)


def test_forward_special_cases_and_library_crosscheck():
    off, nb = _random_graph(150, 1200, 2)
    d = O.sample_dense(O.GraphView(off, nb), [3, 100, 42, 7], [4, 3], seed=8)
    rng = np.random.default_rng(1)
    h0 = rng.standard_normal((len(d["node_ids"]), 5))
    eye, zero, b0 = np.eye(5), np.zeros((5, 5)), np.zeros(5)
    n0 = d["node_id_offsets"][1]
    # W_nbr = 0, W_self = I: layer output is the self rows
    np.testing.assert_array_equal(O.sage_layer(d, h0, eye, zero, b0, relu=False), h0[n0:])
    # additive layer of Algorithm 3 = self + count * mean
    mean_only = O.sage_layer(d, h0, zero, eye, b0, relu=False)
    cnt = np.diff(d["nbr_offsets"])[:, None]
    np.testing.assert_allclose(O.additive_layer(d, h0), h0[n0:] + cnt * mean_only, rtol=1e-12, atol=1e-12)
    # library cross-check: index_select + index_add_ + matmul in fp64
    layers = [(w.double(), n_.double(), b.double()) for w, n_, b in inputs.random_bias_layers([5, 4], 5)]
    ws, wn, b = layers[0]
    ht = torch.from_numpy(h0)
    rm = torch.tensor(d["repr_map"])
    seg = torch.repeat_interleave(torch.arange(len(cnt)), torch.from_numpy(cnt.ravel()))
    agg = torch.zeros((len(cnt), 5), dtype=torch.float64).index_add_(0, seg, ht.index_select(0, rm))
    agg = agg / torch.clamp(torch.from_numpy(cnt).double(), min=1)
    ref = torch.relu(ht[n0:] @ ws + agg @ wn + b)
    got = O.sage_layer(d, h0, ws.numpy(), wn.numpy(), b.numpy(), relu=True)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-12, atol=1e-12)


def test_isolated_node_gets_self_term_only():
    off, nb = _csr_from_edges(3, [(0, 1)])
    d = O.sample_dense(O.GraphView(off, nb), [2, 1], [2], seed=0)
    h0 = np.array([[1.0, 1.0], [2.0, 3.0], [5.0, 7.0]])[d["node_ids"]]
    out = O.forward(d, h0, [(np.eye(2), np.eye(2), np.zeros(2))])
    np.testing.assert_array_equal(out, [[5.0, 7.0], [3.0, 4.0]])


# ---------------------------------------------------------------- link prediction
def test_negatives_are_resident_and_uniform():
    off, nb = _random_graph(100, 300, 0)
    v = O.GraphView(off, nb, n_parts=5, resident_parts=[1, 3])
    negs = O.lp_negatives(v, n_chunks=4, negs_per_chunk=500, seed=77)
    flat = [u for row in negs for u in row]
    assert all(v.is_resident(u) for u in flat)
    counts = np.bincount(flat, minlength=100)
    res = np.array([v.is_resident(u) for u in range(100)])
    assert counts[~res].sum() == 0
    exp = len(flat) / res.sum()
    assert ((counts[res] - exp) ** 2 / exp).sum() < 80.0        # 39 dof
    assert v.resident_nodes() == [v.resident_node_at(i) for i in range(v.n_resident_nodes())]
    assert negs != O.lp_negatives(v, 4, 500, seed=78)


def test_lp_prepare_indices():
    off, nb = _random_graph(50, 200, 0)
    v = O.GraphView(off, nb)
    src, dst = [3, 9, 3, 44], [9, 1, 20, 3]
    p = O.lp_prepare(v, src, dst, n_chunks=2, negs_per_chunk=3, seed=1)
    t = p["targets"]
    assert t == sorted(set(t))
    assert [t[i] for i in p["src_idx"]] == src and [t[i] for i in p["dst_idx"]] == dst
    for row_ids, row_idx in zip(p["neg_ids"], p["neg_idx"]):
        assert [t[i] for i in row_idx] == row_ids
    assert set(t) == set(src) | set(dst) | {u for r in p["neg_ids"] for u in r}


def test_distmult_closed_forms():
    rng = np.random.default_rng(3)
    h = rng.standard_normal((30, 8))
    rel_emb = rng.standard_normal((5, 8))
    n, chunks, negs = 12, 3, 4
    prep = {"src_idx": list(rng.integers(0, 30, n)), "dst_idx": list(rng.integers(0, 30, n)),
            "neg_idx": [list(rng.integers(0, 30, negs)) for _ in range(chunks)]}
    rel = rng.integers(0, 5, n)
    pos, nd, ns = O.distmult_scores(h, rel_emb, prep, rel, chunks)
    s, o = np.array(prep["src_idx"]), np.array(prep["dst_idx"])
    chunk_of = (np.arange(n) * chunks) // n
    neg = np.array(prep["neg_idx"])[chunk_of]                      # [n, negs]
    ht, rt = torch.from_numpy(h), torch.from_numpy(rel_emb)
    np.testing.assert_allclose(pos, torch.einsum("id,id,id->i", ht[s], rt[rel], ht[o]).numpy(), rtol=1e-12)
    np.testing.assert_allclose(nd, torch.einsum("id,id,itd->it", ht[s], rt[rel], ht[neg]).numpy(), rtol=1e-12)
    np.testing.assert_allclose(ns, torch.einsum("itd,id,id->it", ht[neg], rt[rel], ht[o]).numpy(), rtol=1e-12)
    # relation == 1: a plain dot product / matmul
    pos1, nd1, _ = O.distmult_scores(h, np.ones((5, 8)), prep, rel, chunks)
    np.testing.assert_allclose(pos1, (h[s] * h[o]).sum(1), rtol=1e-12)
    np.testing.assert_allclose(nd1, np.stack([h[neg[i]] @ h[s[i]] for i in range(n)]), rtol=1e-12)
    # symmetric in source and destination
    prep2 = dict(prep, src_idx=prep["dst_idx"], dst_idx=prep["src_idx"])
    pos2, nd2, ns2 = O.distmult_scores(h, rel_emb, prep2, rel, chunks)
    np.testing.assert_allclose(pos2, pos, rtol=1e-12)
    np.testing.assert_allclose(nd2, ns, rtol=1e-12)


# ---------------------------------------------------------------- incoming + outgoing sampling (Section 4.1, Section 7.1)
def _out_csr(n, off, nb):
    """Rows by source, built edge by edge from the rows by destination."""
    rows = [[] for _ in range(n)]
    for d in range(n):
        for s in nb[off[d]:off[d + 1]]:
            rows[int(s)].append(d)
    o, out = [0], []
    for r in rows:
        out.extend(sorted(r))
        o.append(len(out))
    return np.array(o), np.array(out, dtype=np.int64)


def _undirected_bfs_levels(off, nb, ooff, onb, targets, k):
    seen = set(targets)
    frontier = list(targets)
    levels = [list(targets)]
    for _ in range(k):
        nxt = set()
        for v in frontier:
            for u in list(nb[off[v]:off[v + 1]]) + list(onb[ooff[v]:ooff[v + 1]]):
                if int(u) not in seen:
                    nxt.add(int(u))
        seen |= nxt
        frontier = sorted(nxt)
        levels.append(frontier)
    return levels


@pytest.mark.parametrize("seed", [0, 1])
def test_inout_full_fanout_gives_undirected_bfs_levels(seed):
    off, nb = _random_graph(70, 160, seed)
    ooff, onb = _out_csr(70, off, nb)
    assert ooff[-1] == off[-1]
    f = int(max(np.diff(off).max(), np.diff(ooff).max()))
    targets = [2, 41, 9]
    k = 3
    view = O.GraphView(off, nb, out_row_offsets=ooff, out_nbrs=onb)
    d = O.sample_dense(view, targets, [f] * k, seed=8, direction="inout")
    levels = _undirected_bfs_levels(off, nb, ooff, onb, targets, k)
    nio = d["node_id_offsets"]
    for j in range(k + 1):
        i = k - j
        assert d["node_ids"][nio[i]:nio[i + 1]] == levels[j]
    sampled = d["node_ids"][nio[1]:]
    for r, v in enumerate(sampled):              # incoming row, then outgoing row
        got = d["nbrs"][d["nbr_offsets"][r]:d["nbr_offsets"][r + 1]]
        assert got == [int(u) for u in nb[off[v]:off[v + 1]]] + [int(u) for u in onb[ooff[v]:ooff[v + 1]]]
    for e, r in enumerate(d["repr_map"]):
        assert d["node_ids"][r] == d["nbrs"][e]


def test_inout_segments_and_reductions():
    off, nb = _random_graph(150, 1500, 5)
    ooff, onb = _out_csr(150, off, nb)
    view = O.GraphView(off, nb, out_row_offsets=ooff, out_nbrs=onb)
    targets = [3, 77, 140, 21]
    fanouts = [3, 2]
    d = O.sample_dense(view, targets, fanouts, seed=13, direction="inout")
    d_in = O.sample_dense(view, targets, fanouts, seed=13, direction="in")
    nio = d["node_id_offsets"]
    k = len(fanouts)
    sampled = d["node_ids"][nio[1]:]
    for i in range(1, k + 1):
        f = fanouts[k - i]
        for r in range(nio[i] - nio[1], nio[i + 1] - nio[1]):
            v = sampled[r]
            seg = d["nbrs"][d["nbr_offsets"][r]:d["nbr_offsets"][r + 1]]
            din, dout = int(off[v + 1] - off[v]), int(ooff[v + 1] - ooff[v])
            assert len(seg) == min(din, f) + min(dout, f)
            head, tail = seg[:min(din, f)], seg[min(din, f):]
            in_row = [int(u) for u in nb[off[v]:off[v + 1]]]
            out_row = [int(u) for u in onb[ooff[v]:ooff[v + 1]]]
            # each part is a sub-sequence of its row (ascending positions, distinct slots)
            it = iter(in_row)
            assert all(any(u == w for w in it) for u in head)
            it = iter(out_row)
            assert all(any(u == w for w in it) for u in tail)
            # the incoming part is exactly what incoming-only sampling of the same node at the same hop gives
            assert head == O.one_hop_sample(view.row(v), f, 13, v, k - i)
    # the targets' incoming parts coincide with incoming-only sampling of the same call
    for r in range(len(targets)):
        a = d["nbrs"][d["nbr_offsets"][nio[k] - nio[1] + r]:d["nbr_offsets"][nio[k] - nio[1] + r + 1]]
        b = d_in["nbrs"][d_in["nbr_offsets"][d_in["node_id_offsets"][k] - d_in["node_id_offsets"][1] + r]:
                         d_in["nbr_offsets"][d_in["node_id_offsets"][k] - d_in["node_id_offsets"][1] + r + 1]]
        v = targets[r]
        assert a[:len(b)] == b or int(off[v + 1] - off[v]) == 0
    # no outgoing edges at all: "inout" is incoming-only sampling, bit for bit
    empty = O.GraphView(off, nb, out_row_offsets=np.zeros(151, dtype=np.int64), out_nbrs=np.zeros(0, dtype=np.int64))
    assert O.sample_dense(empty, targets, fanouts, 13, direction="inout") == d_in
    # no incoming edges and a full fanout: "inout" over (nothing, A) is incoming-only sampling over A
    full = int(np.diff(off).max())
    swapped = O.GraphView(np.zeros(151, dtype=np.int64), np.zeros(0, dtype=np.int64), out_row_offsets=off, out_nbrs=nb)
    assert O.sample_dense(swapped, targets, [full, full], 13, direction="inout") == \
        O.sample_dense(O.GraphView(off, nb), targets, [full, full], 13, direction="in")


def test_inout_directions_use_different_random_words():
    # a node whose incoming and outgoing rows are the same list must not get the same subset twice by construction:
    # over many seeds the two parts differ, and each direction's inclusion is uniform
    row = np.arange(100, 140)
    off = np.array([0, 40] + [40] * 140)
    view = O.GraphView(off, row, out_row_offsets=off, out_nbrs=row)
    same = 0
    hits_out = np.zeros(40)
    n_seeds = 1500
    for s in range(n_seeds):
        d = O.sample_dense(view, [0], [8], seed=s, direction="inout")
        seg = d["nbrs"][:16]
        assert len(seg) == 16
        head, tail = seg[:8], seg[8:]
        same += head == tail
        assert tail == O.one_hop_sample(row, 8, s, 0, 0, O.OUT_SLOT_BASE)
        for u in tail:
            hits_out[u - 100] += 1
    assert same <= 2
    expect = n_seeds * 8 / 40
    chi2 = ((hits_out - expect) ** 2 / expect).sum()
    assert chi2 < 75.0      # 39 degrees of freedom: P(chi2 > 75) < 1e-3


def test_inout_input_errors():
    off, nb = _random_graph(30, 60, 0)
    with pytest.raises(ValueError):
        O.sample_dense(O.GraphView(off, nb), [1], [2], 0, direction="inout")     # no outgoing edge list
    with pytest.raises(ValueError):
        O.sample_dense(O.GraphView(off, nb), [1], [2], 0, direction="out")


def test_sum_aggregator_reduces_to_algorithm_3_and_to_count_times_mean():
    off, nb = _random_graph(120, 900, 2)
    view = O.GraphView(off, nb)
    d = O.sample_dense(view, [4, 9, 100], [3, 2], seed=5)
    rng = np.random.default_rng(0)
    h0 = rng.standard_normal((len(d["node_ids"]), 6))
    eye, zero = np.eye(6), np.zeros(6)
    # identity weights, no bias, no activation: the printed Algorithm 3
    np.testing.assert_allclose(O.sage_layer(d, h0, eye, eye, zero, relu=False, aggregator="sum"), O.additive_layer(d, h0),
                               rtol=0, atol=1e-12)
    # sum = count x mean, row by row, through arbitrary weights
    w_s, w_n, b = rng.standard_normal((6, 5)), rng.standard_normal((6, 5)), rng.standard_normal(5)
    n_rows = len(d["node_ids"]) - d["node_id_offsets"][1]
    counts = np.diff(d["nbr_offsets"])[:n_rows, None]
    mean_part = O.sage_layer(d, h0, np.zeros((6, 5)), w_n, zero[:5], relu=False)
    sum_part = O.sage_layer(d, h0, np.zeros((6, 5)), w_n, zero[:5], relu=False, aggregator="sum")
    np.testing.assert_allclose(sum_part, counts * mean_part, rtol=1e-12, atol=1e-12)
    # the whole forward pass with the sum against per-layer index_add_ in torch
    layers = [(w_s, w_n, b), (rng.standard_normal((5, 4)), rng.standard_normal((5, 4)), rng.standard_normal(4))]
    got = O.forward(d, h0, layers, aggregator="sum")
    cur, h = d, torch.tensor(h0)
    for i, (ws, wn, bb) in enumerate(layers):
        rows = len(cur["node_ids"]) - cur["node_id_offsets"][1]
        seg = torch.repeat_interleave(torch.arange(rows), torch.tensor(np.diff(cur["nbr_offsets"])[:rows]))
        agg = torch.zeros((rows, h.shape[1]), dtype=torch.float64).index_add_(0, seg, h[torch.tensor(cur["repr_map"], dtype=torch.int64)])
        h = h[cur["node_id_offsets"][1]:] @ torch.tensor(ws) + agg @ torch.tensor(wn) + torch.tensor(bb)
        if i == 0:
            h = torch.relu(h)
        cur = O.update_dense(cur)
    np.testing.assert_allclose(got, h.numpy(), rtol=1e-12, atol=1e-12)
    with pytest.raises(ValueError):
        O.sage_layer(d, h0, eye, eye, zero, relu=False, aggregator="max")


# ---------------------------------------------------------------- graph attention over DENSE
def test_gat_uniform_attention_is_the_mean_over_self_and_neighbours():
    off, nb = _random_graph(90, 700, 1)
    d = O.sample_dense(O.GraphView(off, nb), [3, 30, 60, 7], [4, 2], seed=2)
    rng = np.random.default_rng(1)
    h0 = rng.standard_normal((len(d["node_ids"]), 5))
    w, b = rng.standard_normal((5, 3)), rng.standard_normal(3)
    got = O.gat_layer(d, h0, w, np.zeros(3), np.zeros(3), b, relu=False)
    n_rows = len(d["node_ids"]) - d["node_id_offsets"][1]
    counts = np.diff(d["nbr_offsets"])[:n_rows, None]
    total = O.sage_layer(d, h0, w, w, np.zeros(3), relu=False, aggregator="sum")      # (self + sum of neighbours) W
    np.testing.assert_allclose(got, total / (counts + 1) + b, rtol=1e-12, atol=1e-12)


def test_gat_full_fanout_equals_dense_masked_softmax_algebra():
    off, nb = _random_graph(50, 260, 4)
    n = 50
    maxdeg = int(np.diff(off).max())
    targets = list(range(0, 50, 3))
    d = O.sample_dense(O.GraphView(off, nb), targets, [maxdeg], seed=0)
    rng = np.random.default_rng(3)
    feats = rng.standard_normal((n, 6))
    w, a_s, a_d, b = rng.standard_normal((6, 4)), rng.standard_normal(4), rng.standard_normal(4), rng.standard_normal(4)
    got = O.gat_layer(d, feats[d["node_ids"]], w, a_s, a_d, b, relu=True)
    # whole graph, dense: multiplicity matrix + identity, masked softmax row by row in torch
    A = torch.zeros((n, n), dtype=torch.float64)
    for v in range(n):
        for u in nb[off[v]:off[v + 1]]:
            A[v, int(u)] += 1
    A += torch.eye(n, dtype=torch.float64)
    Z = torch.tensor(feats) @ torch.tensor(w)
    E = torch.nn.functional.leaky_relu((Z @ torch.tensor(a_d))[:, None] + (Z @ torch.tensor(a_s))[None, :], 0.2)
    P = A * torch.exp(E - E.max())
    P = P / P.sum(1, keepdim=True)
    want = torch.relu(P @ Z + torch.tensor(b))[targets].numpy()
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)


def test_gat_sharp_attention_picks_the_best_scoring_row_and_isolated_nodes_keep_themselves():
    # node 0 aggregates from 1, 2, 3; node 4 has no neighbours
    off = np.array([0, 3, 3, 3, 3, 3])
    nb = np.array([1, 2, 3])
    d = O.sample_dense(O.GraphView(off, nb), [0, 4], [5], seed=0)
    h0 = np.array([[0.0, 1.0], [1.0, 2.0], [3.0, 3.0], [2.0, 4.0], [5.0, 5.0]])[d["node_ids"]]
    eye = np.eye(2)
    out = O.gat_layer(d, h0, eye, np.array([50.0, 0.0]), np.zeros(2), np.zeros(2), relu=False)
    rows = {v: out[i] for i, v in enumerate(d["node_ids"][d["node_id_offsets"][1]:])}
    np.testing.assert_allclose(rows[0], [3.0, 3.0], atol=1e-12)      # neighbour 2 has the largest first coordinate
    np.testing.assert_allclose(rows[4], [5.0, 5.0], atol=1e-12)      # attends to itself only
    # hand-computed softmax: scores ln 1, ln 2, ln 3, ln 4 for (self, 1, 2, 3) -> weights 0.1 .. 0.4
    h1 = np.array([[np.log(1.0)], [np.log(2.0)], [np.log(3.0)], [np.log(4.0)], [0.0]])[d["node_ids"]]
    vals = O.gat_layer(d, h1, np.ones((1, 1)), np.ones(1), np.zeros(1), np.zeros(1), relu=False)
    want = 0.1 * np.log(1.0) + 0.2 * np.log(2.0) + 0.3 * np.log(3.0) + 0.4 * np.log(4.0)
    got0 = vals[[i for i, v in enumerate(d["node_ids"][d["node_id_offsets"][1]:]) if v == 0][0]]
    np.testing.assert_allclose(got0, [want], rtol=1e-12)


def test_gat_forward_two_layers_uses_algorithm_2_between_layers():
    off, nb = _random_graph(80, 500, 6)
    maxdeg = int(np.diff(off).max())
    targets = [1, 11, 21]
    d = O.sample_dense(O.GraphView(off, nb), targets, [maxdeg, maxdeg], seed=0)
    rng = np.random.default_rng(5)
    feats = rng.standard_normal((80, 4))
    layers = [(rng.standard_normal((4, 3)), rng.standard_normal(3), rng.standard_normal(3), rng.standard_normal(3)),
              (rng.standard_normal((3, 2)), rng.standard_normal(2), rng.standard_normal(2), rng.standard_normal(2))]
    got = O.gat_forward(d, feats[d["node_ids"]], layers)
    # with full fanouts the two layers are whole-graph attention layers on the 2-hop ball
    A = torch.zeros((80, 80), dtype=torch.float64)
    for v in range(80):
        for u in nb[off[v]:off[v + 1]]:
            A[v, int(u)] += 1
    A += torch.eye(80, dtype=torch.float64)
    H = torch.tensor(feats)
    for i, (w, a_s, a_d, b) in enumerate(layers):
        Z = H @ torch.tensor(w)
        E = torch.nn.functional.leaky_relu((Z @ torch.tensor(a_d))[:, None] + (Z @ torch.tensor(a_s))[None, :], 0.2)
        P = A * torch.exp(E - E.max())
        H = (P / P.sum(1, keepdim=True)) @ Z + torch.tensor(b)
        if i == 0:
            H = torch.relu(H)
    np.testing.assert_allclose(got, H[targets].numpy(), rtol=1e-9, atol=1e-11)


def test_gat_heads_are_independent_single_head_layers_on_column_blocks():
    """Multi-head attention: one head reproduces the single-head layer; H heads equal H single-head layers run on the
    column blocks of W, a_src, a_dst and concatenated; with zero attention vectors every head is the plain mean."""
    off, nb = _random_graph(90, 700, 31)
    d = O.sample_dense(O.GraphView(off, nb), [4, 40, 77, 12], [4, 3], seed=3)
    rng = np.random.default_rng(6)
    h0 = rng.standard_normal((len(d["node_ids"]), 6))
    w, a_s, a_d, b = rng.standard_normal((6, 12)), rng.standard_normal(12), rng.standard_normal(12), rng.standard_normal(12)
    np.testing.assert_array_equal(O.gat_layer(d, h0, w, a_s, a_d, b, relu=True), O.gat_layer(d, h0, w, a_s, a_d, b, relu=True, heads=1))
    for heads in (2, 3, 4):
        dh = 12 // heads
        got = O.gat_layer(d, h0, w, a_s, a_d, b, relu=False, heads=heads)
        blocks = [O.gat_layer(d, h0, w[:, i * dh:(i + 1) * dh], a_s[i * dh:(i + 1) * dh], a_d[i * dh:(i + 1) * dh],
                              b[i * dh:(i + 1) * dh], relu=False) for i in range(heads)]
        np.testing.assert_allclose(got, np.concatenate(blocks, axis=1), rtol=1e-13, atol=1e-13)
        uniform = O.gat_layer(d, h0, w, 0 * a_s, 0 * a_d, b, relu=False, heads=heads)
        np.testing.assert_allclose(uniform, O.gat_layer(d, h0, w, 0 * a_s, 0 * a_d, b, relu=False), rtol=1e-13, atol=1e-13)
    with pytest.raises(ValueError):
        O.gat_layer(d, h0, w, a_s, a_d, b, relu=False, heads=5)
    # two layers: heads apply to every layer
    layers = [(w, a_s, a_d, b), (rng.standard_normal((12, 4)), rng.standard_normal(4), rng.standard_normal(4), rng.standard_normal(4))]
    two = O.gat_forward(d, h0, layers, heads=2)
    h1 = O.gat_layer(d, h0, *layers[0], relu=True, heads=2)
    np.testing.assert_allclose(two, O.gat_layer(O.update_dense(d), h1, *layers[1], relu=False, heads=2), rtol=1e-13, atol=1e-13)


# ---------------------------------------------------------------- backward pass
@pytest.mark.parametrize("aggregator", ["mean", "sum"])
def test_backward_equals_central_finite_differences(aggregator):
    off, nb = _random_graph(70, 420, 9)
    d = O.sample_dense(O.GraphView(off, nb), [2, 33, 64, 8, 50], [3, 2], seed=1)
    rng = np.random.default_rng(2)
    h0 = rng.standard_normal((len(d["node_ids"]), 4))
    layers = [(rng.standard_normal((4, 5)) * 0.7, rng.standard_normal((4, 5)) * 0.7, rng.standard_normal(5) * 0.3),
              (rng.standard_normal((5, 3)) * 0.7, rng.standard_normal((5, 3)) * 0.7, rng.standard_normal(3) * 0.3)]
    g_out = rng.standard_normal((5, 3))

    def loss(h0_, layers_):
        return float((O.forward(d, h0_, layers_, aggregator=aggregator) * g_out).sum())

    grads, d_h0 = O.backward(d, h0, layers, g_out, aggregator=aggregator)
    eps = 1e-6
    checks = 0
    for li in range(2):
        for pi in range(3):
            arr = layers[li][pi]
            for idx in list(np.ndindex(arr.shape))[::3]:
                plus = [tuple(np.array(x, copy=True) for x in l) for l in layers]
                minus = [tuple(np.array(x, copy=True) for x in l) for l in layers]
                plus[li][pi][idx] += eps
                minus[li][pi][idx] -= eps
                fd = (loss(h0, plus) - loss(h0, minus)) / (2 * eps)
                assert abs(fd - grads[li][pi][idx]) <= 1e-6 * max(1.0, abs(fd))
                checks += 1
    for r in range(0, h0.shape[0], 2):
        for c in range(4):
            hp, hm = h0.copy(), h0.copy()
            hp[r, c] += eps
            hm[r, c] -= eps
            fd = (loss(hp, layers) - loss(hm, layers)) / (2 * eps)
            assert abs(fd - d_h0[r, c]) <= 1e-6 * max(1.0, abs(fd))
            checks += 1
    assert checks > 80
    # rows of the outermost delta only receive gradient through the neighbour term; a node nobody sampled gets none
    used = set(d["repr_map"]) | set(range(d["node_id_offsets"][1], len(d["node_ids"])))
    for r in range(len(d["node_ids"])):
        if r not in used:
            assert not d_h0[r].any()


def test_backward_against_torch_autograd():
    off, nb = _random_graph(60, 500, 3)
    d = O.sample_dense(O.GraphView(off, nb), [1, 2, 3, 40], [4, 3, 2], seed=4)
    rng = np.random.default_rng(8)
    h0 = rng.standard_normal((len(d["node_ids"]), 3))
    dims = [3, 4, 4, 2]
    layers = [(rng.standard_normal((a, b)), rng.standard_normal((a, b)), rng.standard_normal(b)) for a, b in zip(dims[:-1], dims[1:])]
    g_out = rng.standard_normal((4, 2))
    grads, d_h0 = O.backward(d, h0, layers, g_out)
    # the same network in torch, built from index_select / index_add_ on the DENSE arrays
    th0 = torch.tensor(h0, requires_grad=True)
    tl = [tuple(torch.tensor(x, requires_grad=True) for x in l) for l in layers]
    cur, h = d, th0
    for i, (ws, wn, b) in enumerate(tl):
        first = cur["node_id_offsets"][1]
        rows = len(cur["node_ids"]) - first
        counts = torch.tensor(np.diff(cur["nbr_offsets"])[:rows])
        seg = torch.repeat_interleave(torch.arange(rows), counts)
        agg = torch.zeros((rows, h.shape[1]), dtype=torch.float64).index_add(0, seg, h[torch.tensor(cur["repr_map"], dtype=torch.int64)])
        agg = agg / counts.clamp(min=1)[:, None]
        h = h[first:] @ ws + agg @ wn + b
        if i + 1 < len(tl):
            h = torch.relu(h)
        cur = O.update_dense(cur)
    (h * torch.tensor(g_out)).sum().backward()
    np.testing.assert_allclose(d_h0, th0.grad.numpy(), rtol=1e-10, atol=1e-12)
    for (gs, gn, gb), (ws, wn, b) in zip(grads, tl):
        np.testing.assert_allclose(gs, ws.grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(gn, wn.grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(gb, b.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_backward_with_a_given_relu_branch():
    """relu_masks: the ReLU passes the gradient where the mask says, not where the oracle's own pre-activation is
    positive.  Pinned by (a) its own branch reproducing the default, (b) torch autograd on the same network with the
    ReLU replaced by a multiplication with random masks, (c) central finite differences of that masked network."""
    off, nb = _random_graph(60, 500, 13)
    d = O.sample_dense(O.GraphView(off, nb), [5, 6, 7, 30], [3, 3, 2], seed=2)
    rng = np.random.default_rng(4)
    h0 = rng.standard_normal((len(d["node_ids"]), 3))
    dims = [3, 4, 5, 2]
    layers = [(rng.standard_normal((a, b)), rng.standard_normal((a, b)), rng.standard_normal(b)) for a, b in zip(dims[:-1], dims[1:])]
    g_out = rng.standard_normal((4, 2))
    outs = O.forward(d, h0, layers, return_all=True)
    own = [o > 0 for o in outs[:-1]]
    g_def, dh_def = O.backward(d, h0, layers, g_out)
    g_own, dh_own = O.backward(d, h0, layers, g_out, relu_masks=own)
    np.testing.assert_array_equal(dh_def, dh_own)
    for a, b in zip(g_def, g_own):
        for x, y in zip(a, b):
            np.testing.assert_array_equal(x, y)
    masks = [rng.random(o.shape) < 0.6 for o in outs[:-1]]
    grads, d_h0 = O.backward(d, h0, layers, g_out, relu_masks=masks)

    def masked_net(h, ls, lib):
        cur = d
        for i, (ws, wn, b) in enumerate(ls):
            first = cur["node_id_offsets"][1]
            rows = len(cur["node_ids"]) - first
            counts = np.diff(cur["nbr_offsets"])[:rows]
            if lib is torch:
                seg = torch.repeat_interleave(torch.arange(rows), torch.tensor(counts))
                agg = torch.zeros((rows, h.shape[1]), dtype=torch.float64).index_add(0, seg, h[torch.tensor(cur["repr_map"], dtype=torch.int64)])
                agg = agg / torch.tensor(counts).clamp(min=1)[:, None]
            else:
                agg = np.zeros((rows, h.shape[1]))
                np.add.at(agg, np.repeat(np.arange(rows), counts), h[np.asarray(cur["repr_map"], dtype=np.int64)])
                agg = agg / np.maximum(counts, 1)[:, None]
            h = h[first:] @ ws + agg @ wn + b
            if i + 1 < len(ls):
                h = h * (torch.tensor(masks[i], dtype=torch.float64) if lib is torch else masks[i])
            cur = O.update_dense(cur)
        return h

    th0 = torch.tensor(h0, requires_grad=True)
    tl = [tuple(torch.tensor(x, requires_grad=True) for x in l) for l in layers]
    (masked_net(th0, tl, torch) * torch.tensor(g_out)).sum().backward()
    np.testing.assert_allclose(d_h0, th0.grad.numpy(), rtol=1e-10, atol=1e-12)
    for (gs, gn, gb), (ws, wn, b) in zip(grads, tl):
        np.testing.assert_allclose(gs, ws.grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(gn, wn.grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(gb, b.grad.numpy(), rtol=1e-10, atol=1e-12)
    eps = 1e-6
    for li, pi, idx in [(0, 0, (1, 2)), (0, 1, (2, 0)), (1, 1, (3, 4)), (2, 0, (0, 1)), (1, 2, (2,))]:
        plus = [tuple(np.array(x, copy=True) for x in l) for l in layers]
        minus = [tuple(np.array(x, copy=True) for x in l) for l in layers]
        plus[li][pi][idx] += eps
        minus[li][pi][idx] -= eps
        fd = float(((masked_net(h0, plus, np) - masked_net(h0, minus, np)) * g_out).sum()) / (2 * eps)
        assert abs(fd - grads[li][pi][idx]) <= 1e-6 * max(1.0, abs(fd))


def test_per_node_form_and_arrays_are_two_views_of_one_sample():
    """sample_levels / emit_dense / read_dense: the arrays list exactly the per-node samples, level by level, and
    reading them back gives the per-node form again; shortening DENSE (Algorithm 2) equals sampling one hop less
    from the same levels."""
    off, nb = _random_graph(150, 1300, 17)
    view = O.GraphView(off, nb)
    targets, fanouts = [9, 80, 3, 41], [4, 3, 2]
    levels, sampled = O.sample_levels(view, targets, fanouts, seed=6)
    d = O.emit_dense(levels, sampled)
    assert d == O.sample_dense(view, targets, fanouts, seed=6)
    lv2, sm2 = O.read_dense(d)
    assert lv2 == levels and sm2 == sampled
    assert levels[0] == targets and all(l == sorted(l) for l in levels[1:])
    flat = [v for l in levels for v in l]
    assert len(set(flat)) == len(flat)
    assert set(sampled) == set(v for l in levels[:-1] for v in l)
    for h, l in enumerate(levels[:-1]):
        for v in l:
            row = [int(u) for u in nb[off[v]:off[v + 1]]]
            assert len(sampled[v]) == min(len(row), fanouts[h])
            it = iter(row)
            assert all(u in it for u in sampled[v])          # a sub-sequence of the stored row
    # the node set of level h+1 is what level h's samples reach for the first time
    seen = set(levels[0])
    for h in range(len(fanouts)):
        new = set(u for v in levels[h] for u in sampled[v]) - seen
        assert sorted(new) == levels[h + 1]
        seen |= new
    # one layer later: the farthest level and the samples next to it are gone, nothing else moved
    u = O.update_dense(d)
    lv3, sm3 = O.read_dense(u)
    assert lv3 == levels[:-1]
    assert sm3 == {v: sampled[v] for l in levels[:-2] for v in l}
    n_gone, e_gone = len(levels[-1]), sum(len(sampled[v]) for v in levels[-2])
    assert u["node_ids"] == d["node_ids"][n_gone:]
    assert u["nbrs"] == d["nbrs"][e_gone:]
    assert u["repr_map"] == [r - n_gone for r in d["repr_map"][e_gone:]]


def test_adagrad_closed_forms():
    w = np.array([1.0, -2.0, 0.5, 3.0])
    g = np.array([0.5, -4.0, 0.0, 2.0])
    # first step from a zero state: every coordinate with a gradient moves by lr against its sign
    w1, s1 = O.adagrad_step(w, g, np.zeros(4), lr=0.1, eps=1e-12)
    np.testing.assert_allclose(w1, w - 0.1 * np.sign(g), atol=1e-9)
    np.testing.assert_allclose(s1, g * g)
    # the same gradient again: steps shrink like 1 / sqrt(t)
    w2, s2 = O.adagrad_step(w1, g, s1, lr=0.1, eps=1e-12)
    np.testing.assert_allclose(w2, w1 - 0.1 * np.sign(g) / np.sqrt(2.0), atol=1e-9)
    # against torch's optimiser over five steps of changing gradients
    rng = np.random.default_rng(0)
    tw = torch.tensor(w, requires_grad=True)
    opt = torch.optim.Adagrad([tw], lr=0.05, eps=1e-10)
    cw, cs = w.copy(), np.zeros(4)
    for _ in range(5):
        gi = rng.standard_normal(4)
        tw.grad = torch.tensor(gi)
        opt.step()
        cw, cs = O.adagrad_step(cw, gi, cs, 0.05, 1e-10)
    np.testing.assert_allclose(cw, tw.detach().numpy(), rtol=1e-10)
