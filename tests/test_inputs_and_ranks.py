"""CPU tests of the seeded input generators and of the multi-rank (replicas-only) host logic of bench.py."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import torch

from paper_2202_02365_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_csr_is_the_incoming_adjacency_with_sorted_rows():
    src = torch.tensor([3, 1, 2, 2, 0, 3, 3])
    dst = torch.tensor([0, 0, 0, 1, 1, 3, 0])
    g = inputs.build_csr(src, dst, 4)
    assert g.row_offsets.tolist() == [0, 4, 6, 6, 7]
    assert g.nbrs.tolist() == [1, 2, 3, 3, 0, 2, 3]          # duplicates and the self-loop 3->3 are kept
    rel = torch.arange(7)
    g2 = inputs.build_csr(src, dst, 4, rel)
    # relation ids travel with their edges
    for slot, (u, r) in enumerate(zip(g2.nbrs.tolist(), g2.edge_rel.tolist())):
        v = int(np.searchsorted(g2.row_offsets.numpy(), slot, side="right") - 1)
        assert int(src[r]) == u and int(dst[r]) == v


def test_rmat_is_seeded_power_law_and_in_range():
    a = inputs.rmat_graph(20_000, 300_000, seed=1)
    b = inputs.rmat_graph(20_000, 300_000, seed=1)
    c = inputs.rmat_graph(20_000, 300_000, seed=2)
    assert torch.equal(a.nbrs, b.nbrs) and torch.equal(a.row_offsets, b.row_offsets)
    assert not torch.equal(a.nbrs, c.nbrs)
    assert a.n_edges == 300_000 and int(a.nbrs.min()) >= 0 and int(a.nbrs.max()) < 20_000
    deg = (a.row_offsets[1:] - a.row_offsets[:-1]).numpy()
    assert deg.max() > 40 * deg.mean()                       # hubs
    assert (deg == 0).mean() > 0.2                           # many empty rows
    for v in np.random.default_rng(0).integers(0, 20_000, 50):
        row = a.nbrs[a.row_offsets[v]:a.row_offsets[v + 1]]
        assert bool((row[1:] >= row[:-1]).all())
    # contiguous-id partitions are balanced in edges because ids are permuted
    part_edges = np.add.reduceat(deg, np.arange(0, 20_000, 1250))
    assert part_edges.max() < 2.0 * part_edges.mean()


def test_targets_batches_and_swap_order():
    t = inputs.distinct_targets(1000, 300, seed=3)
    assert t.dtype == torch.int32 and len(set(t.tolist())) == 300
    big = inputs.distinct_targets(1 << 30, 5000, seed=3)
    assert len(set(big.tolist())) == 5000 and int(big.max()) < (1 << 30)
    tb = inputs.train_set_batches(100_000, 11_000, 1000, 11, seed=5)
    assert tb.shape == (11, 1000)
    assert all(len(set(row.tolist())) == 1000 for row in tb)
    assert len(set(tb.reshape(-1).tolist())) == 11_000       # one epoch covers the train set once
    states = inputs.swap_order(32, 10, seed=7)
    assert len(states) == 23 and set().union(*map(set, states)) == set(range(32))
    for a, b in zip(states, states[1:]):
        assert len(a) == len(b) == 10 and len(set(a) ^ set(b)) == 2      # exactly one partition swapped
    m = inputs.resident_node_mask(10, 4, [1, 3])
    assert m.tolist() == [False] * 3 + [True] * 3 + [False] * 3 + [True]


def test_lp_edges_are_resident_slots():
    g = inputs.rmat_graph(5000, 60_000, seed=2, n_relations=9)
    mask = inputs.resident_node_mask(5000, 5, [0, 4])
    src, rel, dst = inputs.lp_edges(g, mask, 400, seed=1)
    assert mask[src.long()].all() and mask[dst.long()].all()
    off, nb, er = g.row_offsets, g.nbrs, g.edge_rel
    for s, r, d in list(zip(src.tolist(), rel.tolist(), dst.tolist()))[:50]:
        row = nb[off[d]:off[d + 1]].tolist()
        rels = er[off[d]:off[d + 1]].tolist()
        assert (s, r) in set(zip(row, rels))


def test_two_ranks_take_disjoint_work_and_reduce_with_max():
    """bench.py --gpus N runs replicas: every rank draws its own mini-batches (seed 100 + rank), the step
    time is the maximum over ranks and the value the sum of the ranks' units over it.  gloo, 2 ranks."""
    script = textwrap.dedent("""
        import os, sys, torch, torch.distributed as dist
        sys.path.insert(0, %r)
        from paper_2202_02365_b200 import inputs
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        batches = inputs.train_set_batches(50_000, 8_000, 100, 6, seed=100 + rank)
        mine = torch.zeros(50_000, dtype=torch.int64); mine[batches.reshape(-1).long()] = 1
        both = mine.clone(); dist.all_reduce(both)
        ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        units = torch.tensor([6.0]); dist.all_reduce(units)
        if rank == 0:
            # different seeds: the ranks' train sets overlap only by chance (16 %% each of the node set)
            print("RESULT", int((both == 2).sum()), int(mine.sum()), float(ms), float(units) / (float(ms) / 1e3))
        dist.destroy_process_group()
    """ % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", "-c", script],
                         capture_output=True, text=True, env=env, timeout=240)
    if out.returncode != 0 and "-c" in out.stderr:            # torchrun without -c support: run from a file
        path = os.path.join(ROOT, ".pytest_cache", "two_ranks.py")
        os.makedirs(os.path.dirname(path), exist_ok=True)
        open(path, "w").write(script)
        out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                              "--master-addr", "127.0.0.1", "--master-port", "29533", path],
                             capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("RESULT")][0].split()
    overlap, mine, ms, value = int(line[1]), int(line[2]), float(line[3]), float(line[4])
    assert mine == 600 and overlap < 60                       # 600 distinct targets per rank, mostly different
    assert ms == 15.0 and abs(value - 12.0 / 0.015) < 1e-6    # max over ranks; whole-job units over it
