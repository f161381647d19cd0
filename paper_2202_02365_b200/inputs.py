"""Seeded synthetic inputs shaped like the paper's workloads (Table 1).

This module only *makes inputs*: graphs, partition splits, feature tables,
weights, target sets and residency orders.  It contains none of the method's
arithmetic (no sampling, no DENSE construction, no aggregation) and is the one
module that both the CUDA path's callers and the CPU oracle's callers use, so
that both sides see the same bytes.

All generators take an explicit seed and a torch device.  The same seed on a
different device type gives a different (but equally distributed) graph, so a
caller generates once and hands the same arrays to both sides.

Graph shapes:
  * Erdos-Renyi: every edge has independent uniform endpoints (duplicates and
    self-loops kept).
  * R-MAT (a, b, c, d) = (0.57, 0.19, 0.19, 0.05): one uniform draw per level
    picks the quadrant; pairs that fall outside [0, N) are redrawn; node ids are
    then passed through a seeded random permutation so that contiguous-id
    partitions are balanced (the paper assigns nodes to partitions randomly,
    Section 5.2).
The CSR handed to the library is the *incoming* adjacency (row = destination,
Figure 1), rows sorted by source id.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


@dataclass
class Graph:
    """CSR of the sampling adjacency.  row v = the nodes v aggregates from."""
    n_nodes: int
    row_offsets: torch.Tensor   # int64 [n_nodes + 1]
    nbrs: torch.Tensor          # int32 [n_edges], each row ascending
    edge_rel: torch.Tensor | None = None  # int32 [n_edges], relation of each CSR slot

    @property
    def n_edges(self) -> int:
        return int(self.nbrs.numel())


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def erdos_renyi_edges(n_nodes: int, n_edges: int, seed: int, device="cpu"):
    g = _gen(seed, device)
    src = torch.randint(0, n_nodes, (n_edges,), generator=g, device=device, dtype=torch.int64)
    dst = torch.randint(0, n_nodes, (n_edges,), generator=g, device=device, dtype=torch.int64)
    return src, dst


def rmat_edges(n_nodes: int, n_edges: int, seed: int, device="cpu",
               a: float = 0.57, b: float = 0.19, c: float = 0.19, d: float = 0.05,
               chunk: int = 1 << 26, permute: bool = True):
    """R-MAT endpoints in [0, n_nodes), ids permuted.  Returns (src, dst) int64."""
    assert abs(a + b + c + d - 1.0) < 1e-9
    g = _gen(seed, device)
    scale = max(1, math.ceil(math.log2(max(2, n_nodes))))
    src = torch.empty(n_edges, dtype=torch.int64, device=device)
    dst = torch.empty(n_edges, dtype=torch.int64, device=device)

    def draw(m: int):
        s = torch.zeros(m, dtype=torch.int64, device=device)
        t = torch.zeros(m, dtype=torch.int64, device=device)
        for _ in range(scale):
            r = torch.rand(m, generator=g, device=device)
            sbit = r >= (a + b)                       # quadrants c, d: source bit set
            tbit = ((r >= a) & (r < a + b)) | (r >= a + b + c)   # quadrants b, d
            s = (s << 1) | sbit.to(torch.int64)
            t = (t << 1) | tbit.to(torch.int64)
        return s, t

    for lo in range(0, n_edges, chunk):
        hi = min(n_edges, lo + chunk)
        s, t = draw(hi - lo)
        bad = (s >= n_nodes) | (t >= n_nodes)
        while bool(bad.any()):
            idx = bad.nonzero(as_tuple=True)[0]
            s2, t2 = draw(int(idx.numel()))
            s[idx] = s2
            t[idx] = t2
            bad = (s >= n_nodes) | (t >= n_nodes)
        src[lo:hi] = s
        dst[lo:hi] = t
    if permute:
        perm = torch.randperm(n_nodes, generator=g, device=device)
        src = perm[src]
        dst = perm[dst]
    return src, dst


def build_csr(src: torch.Tensor, dst: torch.Tensor, n_nodes: int,
              rel: torch.Tensor | None = None) -> Graph:
    """Incoming-adjacency CSR: row = destination, neighbors = sources ascending."""
    key = dst.to(torch.int64) * n_nodes + src.to(torch.int64)
    del src, dst
    if rel is None:
        key = torch.sort(key).values
        order = None
    else:
        key, order = torch.sort(key, stable=True)
    rows = torch.div(key, n_nodes, rounding_mode="floor")
    nbrs = (key - rows * n_nodes).to(torch.int32)
    del key
    counts = torch.bincount(rows, minlength=n_nodes)
    del rows
    offsets = torch.zeros(n_nodes + 1, dtype=torch.int64, device=nbrs.device)
    torch.cumsum(counts, 0, out=offsets[1:])
    erel = rel[order].to(torch.int32) if rel is not None else None
    return Graph(n_nodes, offsets, nbrs, erel)


def transpose_csr(graph: Graph) -> Graph:
    """The second edge list of the same edges: row = source, neighbours = destinations ascending."""
    n = graph.n_nodes
    counts = graph.row_offsets[1:] - graph.row_offsets[:-1]
    dst = torch.repeat_interleave(torch.arange(n, dtype=torch.int64, device=graph.nbrs.device), counts)
    key = torch.sort(graph.nbrs.to(torch.int64) * n + dst).values
    del dst
    rows = torch.div(key, n, rounding_mode="floor")
    nbrs = (key - rows * n).to(torch.int32)
    del key
    out_counts = torch.bincount(rows, minlength=n)
    del rows
    offsets = torch.zeros(n + 1, dtype=torch.int64, device=nbrs.device)
    torch.cumsum(out_counts, 0, out=offsets[1:])
    return Graph(n, offsets, nbrs, None)


def erdos_renyi_graph(n_nodes, n_edges, seed=0, device="cpu") -> Graph:
    s, d = erdos_renyi_edges(n_nodes, n_edges, seed, device)
    return build_csr(s, d, n_nodes)


def rmat_graph(n_nodes, n_edges, seed=0, device="cpu", n_relations: int = 0) -> Graph:
    s, d = rmat_edges(n_nodes, n_edges, seed, device)
    rel = None
    if n_relations:
        g = _gen(seed + 7919, device)
        rel = torch.randint(0, n_relations, (n_edges,), generator=g, device=device, dtype=torch.int32)
    return build_csr(s, d, n_nodes, rel)


def contiguous_partition(n_nodes: int, n_parts: int):
    """Partition size of the contiguous equal split: ceil(N / P); last one short."""
    return (n_nodes + n_parts - 1) // n_parts


def normal_features(n_nodes: int, dim: int, seed: int, device="cpu",
                    dtype=torch.float32, std: float = 1.0, chunk_rows: int = 1 << 22,
                    out: torch.Tensor | None = None, pin: bool = False) -> torch.Tensor:
    """N(0, std^2) table [n_nodes, dim], generated chunk by chunk."""
    g = _gen(seed, device)
    if out is None:
        out = torch.empty((n_nodes, dim), dtype=dtype, device=device,
                          pin_memory=(pin and str(device) == "cpu"))
    for lo in range(0, n_nodes, chunk_rows):
        hi = min(n_nodes, lo + chunk_rows)
        blk = torch.randn((hi - lo, dim), generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            blk *= std
        out[lo:hi] = blk.to(dtype)
    return out


def block_features(n_rows: int, dim: int, seed: int, block: int, device="cpu", dtype=torch.float32, std: float = 1.0,
                   out: torch.Tensor | None = None, chunk_rows: int = 1 << 20) -> torch.Tensor:
    """N(0, std^2) rows of ONE partition block, a pure function of (seed, block, device type): any block of a table
    that is too large to keep (config 4: 187 GB) can be made again on its own, for the partition buffer's staging
    blocks and for the oracle's H^0 rows alike.  `out` (any device, e.g. a pinned host block) receives the rows."""
    g = _gen(int(seed) * 1_000_003 + int(block), device)
    if out is None:
        out = torch.empty((n_rows, dim), dtype=dtype, device=device)
    for lo in range(0, n_rows, chunk_rows):
        hi = min(n_rows, lo + chunk_rows)
        blk = torch.randn((hi - lo, dim), generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            blk *= std
        out[lo:hi].copy_(blk.to(dtype))
    return out


def glorot_layers(dims, seed: int):
    """GraphSage weights for widths dims[0] -> dims[1] -> ...; Glorot-uniform, bias 0.

    Returns a list of (w_self [d_in, d_out], w_nbr [d_in, d_out], bias [d_out]) fp32 CPU.
    """
    g = _gen(seed, "cpu")
    layers = []
    for d_in, d_out in zip(dims[:-1], dims[1:]):
        lim = math.sqrt(6.0 / (d_in + d_out))
        ws = (torch.rand((d_in, d_out), generator=g) * 2 - 1) * lim
        wn = (torch.rand((d_in, d_out), generator=g) * 2 - 1) * lim
        layers.append((ws.float().contiguous(), wn.float().contiguous(),
                       torch.zeros(d_out, dtype=torch.float32)))
    return layers


def random_bias_layers(dims, seed: int):
    """As glorot_layers but with a non-zero bias, so tests can catch a dropped bias."""
    g = _gen(seed + 1, "cpu")
    out = []
    for ws, wn, b in glorot_layers(dims, seed):
        out.append((ws, wn, (torch.rand(b.shape, generator=g) - 0.5).float()))
    return out


def distinct_targets(population: int | torch.Tensor, n: int, seed: int) -> torch.Tensor:
    """n distinct node ids drawn uniformly (CPU int32), in draw order."""
    g = _gen(seed, "cpu")
    if isinstance(population, int):
        if population <= (1 << 24):
            return torch.randperm(population, generator=g)[:n].to(torch.int32)
        # large id spaces: draw with a margin and keep the first n distinct values
        while True:
            cand = torch.randint(0, population, (int(n * 1.2) + 16,), generator=g)
            uniq, first = _first_occurrence_unique(cand)
            if uniq.numel() >= n:
                return uniq[:n].to(torch.int32)
    pop = population.cpu()
    idx = torch.randperm(pop.numel(), generator=g)[:n]
    return pop[idx].to(torch.int32)


def _first_occurrence_unique(x: torch.Tensor):
    vals, inv = torch.unique(x, return_inverse=True)
    first = torch.full((vals.numel(),), x.numel(), dtype=torch.int64)
    first.scatter_reduce_(0, inv, torch.arange(x.numel()), reduce="amin")
    order = torch.argsort(first)
    return vals[order], first[order]


def train_set_batches(n_nodes: int, train_size: int, batch: int, n_batches: int, seed: int):
    """A uniformly drawn train set, shuffled once, cut into consecutive blocks.

    Returns int32 [n_batches, batch]; every row holds distinct ids.
    """
    ids = distinct_targets(n_nodes, train_size, seed)
    need = batch * n_batches
    reps = (need + ids.numel() - 1) // ids.numel()
    if reps > 1:
        ids = ids.repeat(reps)
    return ids[:need].reshape(n_batches, batch).contiguous()


def swap_order(n_parts: int, capacity: int, seed: int):
    """Residency sequence: a random `capacity`-subset, then one random resident
    partition replaced by one random not-yet-seen partition until all have been
    resident (the random-replacement fallback of Section 5.2).

    Returns a list of sorted partition-id lists, one per buffer state.
    """
    g = _gen(seed, "cpu")
    perm = torch.randperm(n_parts, generator=g).tolist()
    cur = perm[:capacity]
    unseen = perm[capacity:]
    states = [sorted(cur)]
    while unseen:
        out = int(torch.randint(0, len(cur), (1,), generator=g))
        cur = cur[:out] + cur[out + 1:] + [unseen.pop(0)]
        states.append(sorted(cur))
    return states


def training_first_partitioning(n_nodes: int, n_parts: int, train_nodes: torch.Tensor, seed: int) -> torch.Tensor:
    """A partition id per node (uint8) after Section 5.2's policy: the training nodes fill the first partitions in
    order, every other node goes to a uniformly random one of the remaining partitions."""
    g = _gen(seed, "cpu")
    size = contiguous_partition(n_nodes, n_parts)
    train_nodes = train_nodes.cpu().long()
    n_train_parts = max(1, (train_nodes.numel() + size - 1) // size)
    assert n_train_parts < n_parts
    part = torch.randint(n_train_parts, n_parts, (n_nodes,), generator=g, dtype=torch.int64)
    part[train_nodes] = torch.arange(train_nodes.numel()) // size
    return part.to(torch.uint8)


def resident_node_mask(n_nodes: int, n_parts: int, resident_parts, device="cpu", part_of_node: torch.Tensor | None = None) -> torch.Tensor:
    size = contiguous_partition(n_nodes, n_parts)
    part = torch.arange(n_nodes, device=device) // size if part_of_node is None else part_of_node.to(device).long()
    res = torch.zeros(n_parts, dtype=torch.bool, device=device)
    res[torch.as_tensor(list(resident_parts), device=device)] = True
    return res[part]


def lp_edges(graph: Graph, resident_mask: torch.Tensor | None, n_edges: int, seed: int):
    """Training edges for link prediction: CSR slots drawn uniformly among those
    whose endpoints are both resident.  Returns (src, rel, dst) int32 CPU tensors.
    """
    g = _gen(seed, "cpu")                  # the draws come from the CPU generator whatever device holds the graph
    off, nbrs = graph.row_offsets, graph.nbrs
    dev = nbrs.device
    rm = None if resident_mask is None else resident_mask.to(dev)
    n_slots = int(nbrs.numel())
    src_l, rel_l, dst_l = [], [], []
    have = 0
    while have < n_edges:
        slots = torch.randint(0, n_slots, (int((n_edges - have) * 1.5) + 64,), generator=g).to(dev)
        dst = torch.searchsorted(off, slots, right=True) - 1
        src = nbrs[slots].to(torch.int64)
        if rm is not None:
            keep = rm[dst] & rm[src]
            slots, dst, src = slots[keep], dst[keep], src[keep]
        rel = graph.edge_rel[slots] if graph.edge_rel is not None else torch.zeros_like(src)
        src_l.append(src.cpu()); rel_l.append(rel.to(torch.int64).cpu()); dst_l.append(dst.cpu())
        have += int(src.numel())
    src = torch.cat(src_l)[:n_edges].to(torch.int32)
    rel = torch.cat(rel_l)[:n_edges].to(torch.int32)
    dst = torch.cat(dst_l)[:n_edges].to(torch.int32)
    return src, rel, dst
