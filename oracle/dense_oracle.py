"""CPU oracle for DENSE sampling, the GraphSage forward over DENSE and DistMult.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, by-eye-checkable
statement of what the CUDA library must compute.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it; the product
package never does, and this file imports nothing from the product package.

It follows the paper's algorithms in the paper's order and notation:
  * Algorithm 1  (multi-hop neighbourhood sampling)      -> sample_dense
  * Section 4.1  (oneHopSample, computeNextDelta)        -> one_hop_sample, compute_next_delta
  * Section 4.2  (repr_map, Steps 1 and 2 of the forward)-> build_repr_map, forward
  * Algorithm 2  (DENSE update after a layer)            -> update_dense
  * Algorithm 3  (layer aggregation; mean instead of sum)-> sage_layer / additive_layer
Floating point is fp64 throughout.

Points the paper leaves open, and the reading taken here:
  * which f neighbours are kept when a node has more than f: f distinct
    positions of the (resident-filtered) row, chosen by Floyd's subset algorithm
    with one counter-based Philox4x32-10 word per slot, keyed by
    (seed, node, hop, slot); kept in ascending position.  The particular subset
    is this build's definition: PARITY UNPINNED by the paper (it prints no
    sample); what the paper does fix (Section 4.1: all neighbours when degree <=
    f, exactly f otherwise) is pinned by tests, as is uniformity of inclusion.
  * order of a delta: ascending node id.  Targets keep the caller's order.
  * arrays carry terminal sentinels: node_id_offsets has k+2 entries (last =
    len(node_ids)), nbr_offsets has one entry per sampled node plus one (last =
    len(nbrs)); Algorithm 2 indexes one past the end on the last layer without
    them.
  * sampling direction: the rows handed to GraphView are what is sampled (the
    harness builds them by destination: incoming neighbours, Figure 1).  With a
    second set of rows by source (Section 4.1 keeps both sorted edge lists) and
    direction "inout", a node gets up to f incoming neighbours followed by up to
    f outgoing ones (Section 7.1 samples from both incoming and outgoing
    edges); the outgoing draws use slots 65536 + t, so the two directions of a
    node never share a random word.
  * fanouts are given ordered away from the targets (Section 7.1): api
    fanouts[h] is Algorithm 1's fanouts[k - h]; hop h = 0 samples the targets.
  * GraphSage layer: act(self . W_self + mean(neighbours) . W_nbr + b), the mean
    over the sampled neighbours (0 when there are none), ReLU between layers and
    none after the last.
  * DistMult: score(s, r, o) = sum_d h_s[d] * rel_r[d] * h_o[d].
  * graph attention (the paper names GAT by citation only): one head, the node itself is
    one of the attended rows, LeakyReLU slope 0.2, ReLU between layers and none after
    the last, bias after the weighted sum.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# Philox4x32-10 (Salmon et al., SC'11): public round constants.
# ----------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Ten Philox rounds on a 4-word counter with a 2-word key; returns 4 words."""
    c0, c1, c2, c3 = (int(x) & _MASK32 for x in counter)
    k0, k1 = (int(x) & _MASK32 for x in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0, p1 & _MASK32,
                          (p0 >> 32) ^ c3 ^ k1, p0 & _MASK32)
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return (c0, c1, c2, c3)


def draw_word(seed: int, node: int, hop: int, slot: int) -> int:
    """The 32-bit random word of (seed, node, hop, slot).

    key = (seed low, seed high); counter = (node low, node high, hop, slot // 4);
    the word used is number slot % 4 of the block.
    """
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    node = int(node)
    block = philox4x32_10((node & _MASK32, (node >> 32) & _MASK32, hop, slot >> 2),
                          (seed & _MASK32, seed >> 32))
    return block[slot & 3]


def to_range(word: int, n: int) -> int:
    """Map a 32-bit word to [0, n) by multiply-high."""
    return (int(word) * int(n)) >> 32


# ----------------------------------------------------------------------------
# Section 4.1: one-hop sampling over the in-memory (resident) subgraph
# ----------------------------------------------------------------------------
class GraphView:
    """The in-memory subgraph: CSR rows restricted to resident endpoints.

    Section 3: sampling sees only nodes and edges of partitions in the buffer.
    Partitions are contiguous id ranges of `part_size` nodes.
    """

    def __init__(self, row_offsets, nbrs, n_parts: int = 1, resident_parts=None,
                 out_row_offsets=None, out_nbrs=None):
        self.row_offsets = np.asarray(row_offsets, dtype=np.int64)
        self.nbrs = np.asarray(nbrs)
        # optional second edge list, sorted by source: row v = destinations of v's outgoing edges
        self.out_row_offsets = None if out_row_offsets is None else np.asarray(out_row_offsets, dtype=np.int64)
        self.out_nbrs = None if out_nbrs is None else np.asarray(out_nbrs)
        self.n_nodes = len(self.row_offsets) - 1
        self.n_parts = int(n_parts)
        self.part_size = (self.n_nodes + self.n_parts - 1) // self.n_parts
        if resident_parts is None:
            resident_parts = range(self.n_parts)
        self.resident_parts = sorted(int(p) for p in resident_parts)
        self._res = set(self.resident_parts)

    def is_resident(self, u: int) -> bool:
        return (int(u) // self.part_size) in self._res

    def row(self, v: int):
        """R(v): the stored row of v, in stored order, resident neighbours only."""
        r = self.nbrs[self.row_offsets[v]:self.row_offsets[v + 1]]
        if len(self._res) == self.n_parts:
            return r
        keep = np.isin(r // self.part_size, self.resident_parts)
        return r[keep]

    def out_row(self, v: int):
        """The outgoing row of v (second edge list), resident neighbours only."""
        if self.out_row_offsets is None:
            raise ValueError("no outgoing edge list")
        r = self.out_nbrs[self.out_row_offsets[v]:self.out_row_offsets[v + 1]]
        if len(self._res) == self.n_parts:
            return r
        keep = np.isin(r // self.part_size, self.resident_parts)
        return r[keep]

    def resident_nodes(self):
        """Resident node ids in ascending partition order (= ascending id)."""
        out = []
        for p in self.resident_parts:
            out.extend(range(p * self.part_size, min((p + 1) * self.part_size, self.n_nodes)))
        return out

    def n_resident_nodes(self) -> int:
        return sum(min((p + 1) * self.part_size, self.n_nodes) - p * self.part_size
                   for p in self.resident_parts)

    def resident_node_at(self, idx: int) -> int:
        """idx-th resident node without building the list."""
        for p in self.resident_parts:
            lo = p * self.part_size
            sz = min((p + 1) * self.part_size, self.n_nodes) - lo
            if idx < sz:
                return lo + idx
            idx -= sz
        raise IndexError(idx)


OUT_SLOT_BASE = 65536   # first slot of the outgoing direction's draws


def one_hop_sample(row, f: int, seed: int, node: int, hop: int, slot_base: int = 0):
    """Up to f neighbours of one node (Section 4.1): the whole row when it has at
    most f entries, otherwise f distinct positions (Floyd's subset algorithm,
    slot t drawing from [0, d - f + t]), returned in ascending position."""
    d = len(row)
    if d <= f:
        return [int(u) for u in row]
    chosen = set()
    for t in range(f):
        j = d - f + t
        x = to_range(draw_word(seed, node, hop, slot_base + t), j + 1)
        chosen.add(j if x in chosen else x)
    return [int(row[p]) for p in sorted(chosen)]


def one_hop_sample_all(view: GraphView, delta, f: int, seed: int, hop: int, direction: str = "in"):
    """oneHopSample(delta, f): concatenated neighbours and each node's start.
    direction "inout": up to f incoming, then up to f outgoing neighbours per node."""
    if direction not in ("in", "inout"):
        raise ValueError("direction must be 'in' or 'inout'")
    d_nbrs, d_offsets = [], []
    for v in delta:
        d_offsets.append(len(d_nbrs))
        d_nbrs.extend(one_hop_sample(view.row(v), f, seed, v, hop))
        if direction == "inout":
            d_nbrs.extend(one_hop_sample(view.out_row(v), f, seed, v, hop, OUT_SLOT_BASE))
    return d_nbrs, d_offsets


def compute_next_delta(d_nbrs, node_ids):
    """computeNextDelta: the unique nodes among the new neighbours that are not
    in node_ids yet (Section 4.1), in ascending id."""
    return sorted(set(d_nbrs) - set(node_ids))


def sample_dense(view: GraphView, target_nodes, fanouts, seed: int, direction: str = "in"):
    """Algorithm 1.  `fanouts` is ordered away from the targets (per direction
    when direction is "inout").

    Returns a dict with node_ids, node_id_offsets (k+2 entries), nbrs,
    nbr_offsets (sampled nodes + 1 entries) and repr_map.
    """
    k = len(fanouts)
    target_nodes = [int(t) for t in target_nodes]
    if len(set(target_nodes)) != len(target_nodes):
        raise ValueError("duplicate target")            # Algorithm 1: unique ids
    for t in target_nodes:
        if not (0 <= t < view.n_nodes):
            raise ValueError("target out of range")
        if not view.is_resident(t):
            raise ValueError("target not resident")      # X_i is a subset of S_i

    node_id_offsets = [0]
    node_ids = list(target_nodes)
    nbr_offsets = []
    nbrs = []
    delta = list(target_nodes)                           # Delta_k
    for i in range(k, 0, -1):
        hop = k - i
        f = fanouts[hop]                                 # Algorithm 1's fanouts[i]
        d_nbrs, d_offsets = one_hop_sample_all(view, delta, f, seed, hop, direction)
        nbr_offsets = d_offsets + [o + len(d_nbrs) for o in nbr_offsets]
        nbrs = d_nbrs + nbrs
        delta = compute_next_delta(d_nbrs, node_ids)     # Delta_{i-1}
        node_id_offsets = [0] + [o + len(delta) for o in node_id_offsets]
        node_ids = delta + node_ids
    dense = {
        "node_ids": node_ids,
        "node_id_offsets": node_id_offsets + [len(node_ids)],   # sentinel
        "nbrs": nbrs,
        "nbr_offsets": nbr_offsets + [len(nbrs)],               # sentinel
    }
    dense["repr_map"] = build_repr_map(dense)
    return dense


def build_repr_map(dense):
    """repr_map[e] = row of H^0 (aligned with node_ids) holding nbrs[e] (Section 4.2)."""
    where = {}
    for r, v in enumerate(dense["node_ids"]):
        assert v not in where, "node_ids must be duplicate-free"
        where[v] = r
    return [where[u] for u in dense["nbrs"]]


# ----------------------------------------------------------------------------
# Section 4.2: forward pass over DENSE
# ----------------------------------------------------------------------------
def update_dense(dense):
    """Algorithm 2: drop Delta_{i-1} and the neighbours of Delta_i."""
    nio = dense["node_id_offsets"]
    node_ids, nbr_offsets = dense["node_ids"], dense["nbr_offsets"]
    nbrs, repr_map = dense["nbrs"], dense["repr_map"]
    delta_prev = node_ids[:nio[1]]
    delta_i = node_ids[nio[1]:nio[2]]
    delta_i_nbrs = nbrs[:nbr_offsets[len(delta_i)]]
    return {
        "nbrs": nbrs[len(delta_i_nbrs):],
        "repr_map": [r - len(delta_prev) for r in repr_map[len(delta_i_nbrs):]],
        "nbr_offsets": [o - len(delta_i_nbrs) for o in nbr_offsets[len(delta_i):]],
        "node_ids": node_ids[nio[1]:],
        "node_id_offsets": [o - len(delta_prev) for o in nio[1:]],
    }


def _segment_reduce(nbr_repr, nbr_offsets, n_rows, mean: bool):
    out = np.zeros((n_rows, nbr_repr.shape[1]), dtype=np.float64)
    for r in range(n_rows):
        lo, hi = nbr_offsets[r], nbr_offsets[r + 1]
        if hi > lo:
            s = nbr_repr[lo:hi].sum(axis=0)
            out[r] = s / (hi - lo) if mean else s
    return out


def additive_layer(dense, h_prev):
    """Algorithm 3 as printed: H = segment_sum(H_prev[repr_map]) + self."""
    h_prev = np.asarray(h_prev, dtype=np.float64)
    n_rows = len(dense["node_ids"]) - dense["node_id_offsets"][1]
    nbr_repr = h_prev[np.asarray(dense["repr_map"], dtype=np.int64)]
    nbr_aggr = _segment_reduce(nbr_repr, dense["nbr_offsets"], n_rows, mean=False)
    self_repr = h_prev[dense["node_id_offsets"][1]:]
    return nbr_aggr + self_repr


def sage_layer(dense, h_prev, w_self, w_nbr, bias, relu: bool, aggregator: str = "mean"):
    """Algorithm 3 with self/neighbour linears; the neighbour term is GraphSage's mean over
    the sampled neighbours ("mean") or their sum ("sum", the aggregation Algorithm 3 prints)."""
    if aggregator not in ("mean", "sum"):
        raise ValueError("aggregator must be 'mean' or 'sum'")
    h_prev = np.asarray(h_prev, dtype=np.float64)
    n_rows = len(dense["node_ids"]) - dense["node_id_offsets"][1]
    nbr_repr = h_prev[np.asarray(dense["repr_map"], dtype=np.int64)]
    nbr_aggr = _segment_reduce(nbr_repr, dense["nbr_offsets"], n_rows, mean=(aggregator == "mean"))
    self_repr = h_prev[dense["node_id_offsets"][1]:]
    out = (self_repr @ np.asarray(w_self, dtype=np.float64)
           + nbr_aggr @ np.asarray(w_nbr, dtype=np.float64)
           + np.asarray(bias, dtype=np.float64))
    return np.maximum(out, 0.0) if relu else out


def gat_layer(dense, h_prev, w, a_src, a_dst, bias, relu: bool, slope: float = 0.2):
    """One graph-attention layer (the GAT of Velickovic et al., which Section 7.1 trains as the second model) over
    DENSE, single head: z = h W for every input row; for output row i with sampled neighbours j (repeats count) and
    itself, e_ij = LeakyReLU(a_dst . z_i + a_src . z_j), alpha = softmax over {i} + neighbours, h'_i = sum alpha_ij z_j
    + bias.  A node without neighbours attends to itself only."""
    h_prev = np.asarray(h_prev, dtype=np.float64)
    z = h_prev @ np.asarray(w, dtype=np.float64)
    s_src = z @ np.asarray(a_src, dtype=np.float64)
    s_dst = z @ np.asarray(a_dst, dtype=np.float64)
    first = dense["node_id_offsets"][1]
    n_rows = len(dense["node_ids"]) - first
    repr_map, nbr_offsets = dense["repr_map"], dense["nbr_offsets"]
    out = np.zeros((n_rows, z.shape[1]), dtype=np.float64)
    for r in range(n_rows):
        me = first + r
        src = [me] + [repr_map[e] for e in range(nbr_offsets[r], nbr_offsets[r + 1])]
        e = np.array([s_dst[me] + s_src[j] for j in src])
        e = np.where(e > 0, e, slope * e)
        a = np.exp(e - e.max())
        a /= a.sum()
        out[r] = (a[:, None] * z[src]).sum(axis=0)
    out = out + np.asarray(bias, dtype=np.float64)
    return np.maximum(out, 0.0) if relu else out


def gat_forward(dense, h0, layers, slope: float = 0.2):
    """k attention layers with Algorithm 2 between them; layers: (w, a_src, a_dst, bias); ReLU on all but the last."""
    h = np.asarray(h0, dtype=np.float64)
    cur = {key: list(val) for key, val in dense.items()}
    for i, (w, a_src, a_dst, bias) in enumerate(layers):
        h = gat_layer(cur, h, w, a_src, a_dst, bias, relu=(i + 1 < len(layers)), slope=slope)
        cur = update_dense(cur)
    return h


def forward(dense, h0, layers, return_all: bool = False, aggregator: str = "mean"):
    """k layers: Step 1 (layer output) then Step 2 (Algorithm 2), Section 4.2.

    h0: [len(node_ids), d0] base representations aligned with node_ids.
    layers: list of (w_self [d_in, d_out], w_nbr [d_in, d_out], bias [d_out]).
    Returns H^k, one row per target in the caller's order.
    """
    h = np.asarray(h0, dtype=np.float64)
    assert h.shape[0] == len(dense["node_ids"])
    cur = {key: list(val) for key, val in dense.items()}
    outs = []
    for i, (w_self, w_nbr, bias) in enumerate(layers):
        h = sage_layer(cur, h, w_self, w_nbr, bias, relu=(i + 1 < len(layers)), aggregator=aggregator)
        outs.append(h)
        cur = update_dense(cur)
    return outs if return_all else h


def backward(dense, h0, layers, d_out, aggregator: str = "mean"):
    """Gradients of a scalar loss through forward(): d_out = dL/dH^k, one row per target.

    The chain rule through Algorithm 3 (self and neighbour linears, mean or sum over the
    sampled neighbours through repr_map, ReLU on all but the last layer) and Algorithm 2
    (layer l's rows are the rows of layer l-1 without the outermost delta).  Returns
    (grads, d_h0): grads[l] = (dW_self, dW_nbr, dbias) of layer l + 1, d_h0 = dL/dH^0 with one
    row per entry of node_ids (the gradient of the base representations, Section 3)."""
    h = np.asarray(h0, dtype=np.float64)
    cur = {key: list(val) for key, val in dense.items()}
    saved = []
    for i, (w_self, w_nbr, bias) in enumerate(layers):
        first = cur["node_id_offsets"][1]
        n_rows = len(cur["node_ids"]) - first
        nbr_repr = h[np.asarray(cur["repr_map"], dtype=np.int64)]
        agg = _segment_reduce(nbr_repr, cur["nbr_offsets"], n_rows, mean=(aggregator == "mean"))
        pre = (h[first:] @ np.asarray(w_self, dtype=np.float64) + agg @ np.asarray(w_nbr, dtype=np.float64)
               + np.asarray(bias, dtype=np.float64))
        saved.append((cur, h, agg, pre))
        h = np.maximum(pre, 0.0) if i + 1 < len(layers) else pre
        cur = update_dense(cur)
    d_h = np.asarray(d_out, dtype=np.float64)
    grads = [None] * len(layers)
    for i in range(len(layers) - 1, -1, -1):
        cur, h_in, agg, pre = saved[i]
        w_self, w_nbr = (np.asarray(x, dtype=np.float64) for x in layers[i][:2])
        d_pre = d_h * (pre > 0.0) if i + 1 < len(layers) else d_h
        first = cur["node_id_offsets"][1]
        n_rows = len(cur["node_ids"]) - first
        grads[i] = (h_in[first:].T @ d_pre, agg.T @ d_pre, d_pre.sum(axis=0))
        d_in = np.zeros_like(h_in)
        d_in[first:] += d_pre @ w_self.T
        d_agg = d_pre @ w_nbr.T
        for r in range(n_rows):
            lo, hi = cur["nbr_offsets"][r], cur["nbr_offsets"][r + 1]
            if hi > lo:
                share = d_agg[r] / (hi - lo) if aggregator == "mean" else d_agg[r]
                for e in range(lo, hi):
                    d_in[cur["repr_map"][e]] += share
        d_h = d_in
    return grads, d_h


def adagrad_step(w, g, state, lr: float, eps: float):
    """Adagrad (Duchi et al.), the optimiser the paper's system trains with besides SGD: the state accumulates squared
    gradients, the step of every coordinate is scaled by the root of its state.  Returns (w', state')."""
    g = np.asarray(g, dtype=np.float64)
    state = np.asarray(state, dtype=np.float64) + g * g
    return np.asarray(w, dtype=np.float64) - lr * g / (np.sqrt(state) + eps), state


# ----------------------------------------------------------------------------
# Link prediction: shared uniform negatives, target union, DistMult
# ----------------------------------------------------------------------------
def lp_negatives(view: GraphView, n_chunks: int, negs_per_chunk: int, seed: int):
    """Negative node of (chunk c, slot t): Philox word 0 of counter
    (c, t, 0xFFFFFFFF, 0) under key seed, mapped to the resident nodes taken in
    ascending partition order.  Uniform with repetition, true edges not filtered."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    n_res = view.n_resident_nodes()
    out = []
    for c in range(n_chunks):
        row = []
        for t in range(negs_per_chunk):
            w = philox4x32_10((c, t, 0xFFFFFFFF, 0), (seed & _MASK32, seed >> 32))[0]
            row.append(view.resident_node_at(to_range(w, n_res)))
        out.append(row)
    return out


def lp_prepare(view: GraphView, src, dst, n_chunks: int, negs_per_chunk: int, seed: int):
    """Targets = ascending unique(src | dst | negatives) and everyone's index in it."""
    negs = lp_negatives(view, n_chunks, negs_per_chunk, seed)
    targets = sorted(set(int(s) for s in src) | set(int(d) for d in dst)
                     | set(u for row in negs for u in row))
    where = {v: i for i, v in enumerate(targets)}
    return {
        "targets": targets,
        "src_idx": [where[int(s)] for s in src],
        "dst_idx": [where[int(d)] for d in dst],
        "neg_ids": negs,
        "neg_idx": [[where[u] for u in row] for row in negs],
    }


def distmult_scores(h, rel_emb, prep, rel, n_chunks: int):
    """pos[i], neg_dst[i, t] (destination replaced by the chunk's negative t) and
    neg_src[i, t] (source replaced).  Edge i is in chunk floor(i * n_chunks / B)."""
    h = np.asarray(h, dtype=np.float64)
    rel_emb = np.asarray(rel_emb, dtype=np.float64)
    n = len(prep["src_idx"])
    negs = len(prep["neg_idx"][0]) if n_chunks else 0
    pos = np.zeros(n)
    neg_dst = np.zeros((n, negs))
    neg_src = np.zeros((n, negs))
    for i in range(n):
        hs, ho, r = h[prep["src_idx"][i]], h[prep["dst_idx"][i]], rel_emb[int(rel[i])]
        pos[i] = np.sum(hs * r * ho)
        c = (i * n_chunks) // n
        hn = h[np.asarray(prep["neg_idx"][c], dtype=np.int64)]
        neg_dst[i] = hn @ (hs * r)
        neg_src[i] = hn @ (r * ho)
    return pos, neg_dst, neg_src
