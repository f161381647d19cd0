"""CPU oracle for DENSE sampling, the GraphSage forward over DENSE and DistMult.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, by-eye-checkable
statement of what the CUDA library must compute.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it; the product
package never does, and this file imports nothing from the product package.

What it computes, and where the paper defines it:
  * Algorithm 1, Section 4.1 (multi-hop sampling of only the newly reached nodes; oneHopSample,
    computeNextDelta): sample_levels keeps one sampled neighbour list per node in a dict and finds
    each hop's new nodes with Python sets; emit_dense lays the result out as the DENSE arrays.
  * Section 4.2 (repr_map; a layer's output, then the shortened DENSE): forward, sage_layer,
    additive_layer (the example layer of Algorithm 3), update_dense (the result of Algorithm 2,
    obtained by dropping the per-node data the next layer no longer needs and laying it out again).
Floating point is fp64 throughout; nothing is blocked, fused or vectorised beyond one matmul per layer.

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
    Partitions are contiguous id ranges of `part_size` nodes, or, with `part_of_node`
    (one partition id per node), whatever that array says -- Section 5.2 places the
    training nodes in the first partitions and assigns the others at random.
    """

    def __init__(self, row_offsets, nbrs, n_parts: int = 1, resident_parts=None,
                 out_row_offsets=None, out_nbrs=None, part_of_node=None):
        self.row_offsets = np.asarray(row_offsets, dtype=np.int64)
        self.nbrs = np.asarray(nbrs)
        # optional second edge list, sorted by source: row v = destinations of v's outgoing edges
        self.out_row_offsets = None if out_row_offsets is None else np.asarray(out_row_offsets, dtype=np.int64)
        self.out_nbrs = None if out_nbrs is None else np.asarray(out_nbrs)
        self.n_nodes = len(self.row_offsets) - 1
        self.n_parts = int(n_parts)
        self.part_size = (self.n_nodes + self.n_parts - 1) // self.n_parts
        self.part_of_node = None if part_of_node is None else np.asarray(part_of_node, dtype=np.int64)
        if self.part_of_node is not None:
            assert len(self.part_of_node) == self.n_nodes and self.part_of_node.max(initial=0) < self.n_parts
        if resident_parts is None:
            resident_parts = range(self.n_parts)
        self.resident_parts = sorted(int(p) for p in resident_parts)
        self._res = set(self.resident_parts)
        self._members = {}

    def part(self, u):
        """Partition of node u (or of every node of an array)."""
        if self.part_of_node is not None:
            return self.part_of_node[u]
        return u // self.part_size

    def nodes_of_part(self, p: int):
        """Ids of partition p's nodes, ascending (a range for the contiguous split, else an array, made once)."""
        if self.part_of_node is None:
            return range(p * self.part_size, min((p + 1) * self.part_size, self.n_nodes))
        if p not in self._members:
            self._members[p] = np.nonzero(self.part_of_node == p)[0]
        return self._members[p]

    def is_resident(self, u: int) -> bool:
        return int(self.part(int(u))) in self._res

    def _filter(self, r):
        if len(self._res) == self.n_parts:
            return r
        return r[np.isin(self.part(r), self.resident_parts)]

    def row(self, v: int):
        """R(v): the stored row of v, in stored order, resident neighbours only."""
        return self._filter(self.nbrs[self.row_offsets[v]:self.row_offsets[v + 1]])

    def out_row(self, v: int):
        """The outgoing row of v (second edge list), resident neighbours only."""
        if self.out_row_offsets is None:
            raise ValueError("no outgoing edge list")
        return self._filter(self.out_nbrs[self.out_row_offsets[v]:self.out_row_offsets[v + 1]])

    def resident_nodes(self):
        """Resident node ids in ascending partition order, ascending id inside a partition."""
        out = []
        for p in self.resident_parts:
            out.extend(int(v) for v in self.nodes_of_part(p))
        return out

    def n_resident_nodes(self) -> int:
        return sum(len(self.nodes_of_part(p)) for p in self.resident_parts)

    def resident_node_at(self, idx: int) -> int:
        """idx-th resident node in that order."""
        for p in self.resident_parts:
            ids = self.nodes_of_part(p)
            if idx < len(ids):
                return int(ids[idx])
            idx -= len(ids)
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


def _check_targets(view: GraphView, target_nodes):
    """Algorithm 1 takes unique target ids; Section 3: a batch's targets lie in resident partitions."""
    if len(set(target_nodes)) != len(target_nodes):
        raise ValueError("duplicate target")
    for t in target_nodes:
        if not (0 <= t < view.n_nodes):
            raise ValueError("target out of range")
        if not view.is_resident(t):
            raise ValueError("target not resident")


def sample_levels(view: GraphView, target_nodes, fanouts, seed: int, direction: str = "in"):
    """What Algorithm 1 / Section 4.1 computes, kept per node instead of in arrays.

    levels[h] = the nodes first reached after h hops (levels[0] = the targets in the caller's
    order; every later level in ascending id) -- the paper's Delta_{k-h}.  sampled[v] = the one-hop
    sample of v, drawn exactly once, at the hop whose level v belongs to, with that hop's fanout
    (`fanouts` is ordered away from the targets; per direction when direction is "inout": up to f
    incoming neighbours followed by up to f outgoing ones).  The nodes of the last level are
    reached but not sampled."""
    if direction not in ("in", "inout"):
        raise ValueError("direction must be 'in' or 'inout'")
    target_nodes = [int(t) for t in target_nodes]
    _check_targets(view, target_nodes)
    seen = set(target_nodes)
    levels = [list(target_nodes)]
    sampled = {}
    for hop, f in enumerate(fanouts):
        reached = set()
        for v in levels[hop]:                    # only the newly reached nodes are sampled
            picks = one_hop_sample(view.row(v), f, seed, v, hop)
            if direction == "inout":
                picks = picks + one_hop_sample(view.out_row(v), f, seed, v, hop, OUT_SLOT_BASE)
            sampled[v] = picks
            reached.update(picks)
        new = reached - seen                     # unique, and not in any earlier level
        seen |= new
        levels.append(sorted(new))
    return levels, sampled


def emit_dense(levels, sampled):
    """The DENSE arrays of Section 4.1 for per-node samples: node_ids lists the levels from the farthest one to the
    targets; nbrs lists the samples of the sampled nodes in node_ids order; the offsets carry a terminal entry;
    repr_map[e] = position of nbrs[e] in node_ids (Section 4.2)."""
    node_ids, node_id_offsets = [], []
    for level in reversed(levels):
        node_id_offsets.append(len(node_ids))
        node_ids.extend(level)
    node_id_offsets.append(len(node_ids))
    where = {}
    for r, v in enumerate(node_ids):
        assert v not in where, "a node belongs to one level only"
        where[v] = r
    nbrs, nbr_offsets = [], []
    for v in node_ids[node_id_offsets[1]:]:      # the farthest level has no samples
        nbr_offsets.append(len(nbrs))
        nbrs.extend(sampled[v])
    nbr_offsets.append(len(nbrs))
    return {"node_ids": node_ids, "node_id_offsets": node_id_offsets, "nbrs": nbrs, "nbr_offsets": nbr_offsets,
            "repr_map": [where[u] for u in nbrs]}


def sample_dense(view: GraphView, target_nodes, fanouts, seed: int, direction: str = "in"):
    """Multi-hop sampling into DENSE (Algorithm 1): node_ids, node_id_offsets (k+2 entries), nbrs, nbr_offsets
    (sampled nodes + 1 entries) and repr_map."""
    levels, sampled = sample_levels(view, target_nodes, fanouts, seed, direction)
    return emit_dense(levels, sampled)


def read_dense(dense):
    """Back from the arrays to per-node form: (levels from the targets outwards, sampled)."""
    nio, node_ids = dense["node_id_offsets"], dense["node_ids"]
    levels = [list(node_ids[nio[j]:nio[j + 1]]) for j in range(len(nio) - 1)][::-1]
    sampled = {}
    for r, v in enumerate(node_ids[nio[1]:]):
        sampled[v] = list(dense["nbrs"][dense["nbr_offsets"][r]:dense["nbr_offsets"][r + 1]])
    return levels, sampled


# ----------------------------------------------------------------------------
# Section 4.2: forward pass over DENSE
# ----------------------------------------------------------------------------
def update_dense(dense):
    """What DENSE looks like after a layer (Algorithm 2, Section 4.2): the farthest level has served as input for
    the last time, and the samples of the level next to it were consumed by the layer, so both go; that level is
    now the farthest one, without samples.  Positions (offsets, repr_map) are those of the shortened arrays."""
    levels, sampled = read_dense(dense)
    gone = levels.pop()                          # farthest level
    assert not any(v in sampled for v in gone)
    for v in levels[-1]:
        del sampled[v]
    return emit_dense(levels, sampled)


def _neighbour_rows(dense, r):
    """Rows of the layer's input that output row r aggregates (through repr_map, repeats included)."""
    return dense["repr_map"][dense["nbr_offsets"][r]:dense["nbr_offsets"][r + 1]]


def _aggregate(dense, h_prev, mean: bool):
    """Per output row the sum (or mean) of its sampled neighbours' input rows; zero for a row without any."""
    first = dense["node_id_offsets"][1]          # input rows below `first` belong to the farthest level
    n_rows = len(dense["node_ids"]) - first
    out = np.zeros((n_rows, h_prev.shape[1]), dtype=np.float64)
    for r in range(n_rows):
        rows = _neighbour_rows(dense, r)
        if len(rows):
            s = h_prev[np.asarray(rows, dtype=np.int64)].sum(axis=0)
            out[r] = s / len(rows) if mean else s
    return out


def additive_layer(dense, h_prev):
    """The example layer of Section 4.2 (Algorithm 3): every output row is its own input row plus the sum of its
    sampled neighbours' input rows."""
    h_prev = np.asarray(h_prev, dtype=np.float64)
    return h_prev[dense["node_id_offsets"][1]:] + _aggregate(dense, h_prev, mean=False)


def sage_layer(dense, h_prev, w_self, w_nbr, bias, relu: bool, aggregator: str = "mean"):
    """GraphSage layer over DENSE: act(self . W_self + aggregate . W_nbr + bias); the aggregate is the mean over the
    sampled neighbours ("mean") or their sum ("sum", the aggregation of Algorithm 3)."""
    if aggregator not in ("mean", "sum"):
        raise ValueError("aggregator must be 'mean' or 'sum'")
    h_prev = np.asarray(h_prev, dtype=np.float64)
    self_repr = h_prev[dense["node_id_offsets"][1]:]
    nbr_aggr = _aggregate(dense, h_prev, mean=(aggregator == "mean"))
    out = (self_repr @ np.asarray(w_self, dtype=np.float64)
           + nbr_aggr @ np.asarray(w_nbr, dtype=np.float64)
           + np.asarray(bias, dtype=np.float64))
    return np.maximum(out, 0.0) if relu else out


def gat_layer(dense, h_prev, w, a_src, a_dst, bias, relu: bool, slope: float = 0.2, heads: int = 1):
    """One graph-attention layer (the GAT of Velickovic et al., which Section 7.1 trains as the second model) over
    DENSE: z = h W for every input row; for output row i with sampled neighbours j (repeats count) and itself,
    e_ij = LeakyReLU(a_dst . z_i + a_src . z_j), alpha = softmax over {i} + neighbours, h'_i = sum alpha_ij z_j + bias.
    A node without neighbours attends to itself only.  With `heads` > 1 the columns of z (and of a_src, a_dst) are cut
    into that many equal blocks, every block attends on its own with its own scores, and the blocks' results are
    concatenated (the width of the layer stays that of W)."""
    h_prev = np.asarray(h_prev, dtype=np.float64)
    z = h_prev @ np.asarray(w, dtype=np.float64)
    a_src = np.asarray(a_src, dtype=np.float64)
    a_dst = np.asarray(a_dst, dtype=np.float64)
    width = z.shape[1]
    if heads < 1 or width % heads:
        raise ValueError("the layer's width must be a multiple of the number of heads")
    dh = width // heads
    first = dense["node_id_offsets"][1]
    n_rows = len(dense["node_ids"]) - first
    out = np.zeros((n_rows, width), dtype=np.float64)
    for hd in range(heads):
        cols = slice(hd * dh, (hd + 1) * dh)
        zh = z[:, cols]
        s_src = zh @ a_src[cols]
        s_dst = zh @ a_dst[cols]
        for r in range(n_rows):
            me = first + r
            src = [me] + list(_neighbour_rows(dense, r))
            e = np.array([s_dst[me] + s_src[j] for j in src])
            e = np.where(e > 0, e, slope * e)
            a = np.exp(e - e.max())
            a /= a.sum()
            out[r, cols] = (a[:, None] * zh[src]).sum(axis=0)
    out = out + np.asarray(bias, dtype=np.float64)
    return np.maximum(out, 0.0) if relu else out


def gat_forward(dense, h0, layers, slope: float = 0.2, heads: int = 1):
    """k attention layers with Algorithm 2 between them; layers: (w, a_src, a_dst, bias); ReLU on all but the last."""
    h = np.asarray(h0, dtype=np.float64)
    cur = dense
    for i, (w, a_src, a_dst, bias) in enumerate(layers):
        h = gat_layer(cur, h, w, a_src, a_dst, bias, relu=(i + 1 < len(layers)), slope=slope, heads=heads)
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
    cur = dense
    outs = []
    for i, (w_self, w_nbr, bias) in enumerate(layers):
        h = sage_layer(cur, h, w_self, w_nbr, bias, relu=(i + 1 < len(layers)), aggregator=aggregator)
        outs.append(h)
        cur = update_dense(cur)
    return outs if return_all else h


def backward(dense, h0, layers, d_out, aggregator: str = "mean", relu_masks=None):
    """Gradients of a scalar loss through forward(): d_out = dL/dH^k, one row per target.

    The chain rule through the GraphSage layer (self and neighbour linears, mean or sum over the
    sampled neighbours through repr_map, ReLU on all but the last layer) and through the shortening
    of DENSE between layers (layer l's rows are the rows of layer l-1 without the farthest level).
    Returns (grads, d_h0): grads[l] = (dW_self, dW_nbr, dbias) of layer l + 1, d_h0 = dL/dH^0 with
    one row per entry of node_ids (the gradient of the base representations, Section 3).

    relu_masks (optional): for each layer but the last a boolean array shaped like that layer's
    output; the ReLU of that layer then passes the gradient where the mask is set instead of where
    this function's own pre-activation is positive.  A test that compares against a forward pass
    computed in lower precision hands over the branch that pass took, so that both sides
    differentiate the same piecewise-linear function."""
    h = np.asarray(h0, dtype=np.float64)
    cur = dense
    saved = []
    for i, (w_self, w_nbr, bias) in enumerate(layers):
        first = cur["node_id_offsets"][1]
        agg = _aggregate(cur, h, mean=(aggregator == "mean"))
        pre = (h[first:] @ np.asarray(w_self, dtype=np.float64) + agg @ np.asarray(w_nbr, dtype=np.float64)
               + np.asarray(bias, dtype=np.float64))
        last = i + 1 == len(layers)
        passes = None if last else (pre > 0.0 if relu_masks is None else np.asarray(relu_masks[i], dtype=bool))
        saved.append((cur, h, agg, passes))
        h = pre if last else np.where(passes, pre, 0.0)
        cur = update_dense(cur)
    d_h = np.asarray(d_out, dtype=np.float64)
    grads = [None] * len(layers)
    for i in range(len(layers) - 1, -1, -1):
        cur, h_in, agg, passes = saved[i]
        w_self, w_nbr = (np.asarray(x, dtype=np.float64) for x in layers[i][:2])
        d_pre = d_h if passes is None else d_h * passes
        first = cur["node_id_offsets"][1]
        grads[i] = (h_in[first:].T @ d_pre, agg.T @ d_pre, d_pre.sum(axis=0))
        d_in = np.zeros_like(h_in)
        d_in[first:] += d_pre @ w_self.T
        d_agg = d_pre @ w_nbr.T
        for r in range(d_pre.shape[0]):
            rows = _neighbour_rows(cur, r)
            if len(rows):
                share = d_agg[r] / len(rows) if aggregator == "mean" else d_agg[r]
                for src in rows:                 # a repeated neighbour receives its share once per repeat
                    d_in[src] += share
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
