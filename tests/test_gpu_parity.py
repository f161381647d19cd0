"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import paper_2202_02365_b200 as mg
from oracle import dense_oracle as O
from paper_2202_02365_b200 import inputs

pytestmark = pytest.mark.gpu

RTOL_AGG = 1e-5     # fp32 aggregation / fp32 GEMM outputs
RTOL_TC = 5e-3      # TF32 tensor-core GEMM outputs


def close(got, ref, rtol, per_row=False):
    """|got - ref| <= rtol * max(|ref|, rms(ref)) element-wise.  rms is taken over the whole matrix, or, with per_row,
    over the element's own row: for matrices whose rows differ in scale by orders of magnitude (the gradient rows of
    the base representations: a target's row against the row of a node three hops away)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    if ref.size == 0:
        return
    rms = np.sqrt(np.mean(ref ** 2, axis=1, keepdims=True)) if per_row else np.sqrt(np.mean(ref ** 2))
    bound = rtol * np.maximum(np.abs(ref), rms)
    err = np.abs(got - ref)
    worst = np.max(err / np.maximum(bound, 1e-300))
    big = (np.abs(ref) > rms / 100) & (np.abs(ref) > 0)   # the rms floor only matters below this; report the plain relative error above it
    from conftest import note_relative_error
    note_relative_error(rtol, float(np.max(err[big] / np.abs(ref[big]))) if big.any() else 0.0, float(worst))
    assert worst <= 1.0, f"worst error {worst:.3f} x the bound (rtol {rtol})"


def near(got, ref, rtol):
    """|got - ref| <= rtol * |ref| in the Frobenius norm (a second line beside close(), never instead of it)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    assert np.linalg.norm(got - ref) <= rtol * max(np.linalg.norm(ref), 1e-30)


def gpu_relu_branch(ctx, model, dense, batch, ref):
    """The side of every ReLU the GPU's forward pass took for mini-batch `batch`: the sign pattern of its kept layer
    outputs H^1 .. H^{k-1}, rows in the order of the paper's node_ids (as oracle.backward's relu_masks wants them)."""
    nio = ref["node_id_offsets"]
    k = len(nio) - 2
    return [ctx.layer_output(model, dense, l, batch, nio[-1] - nio[l]).cpu().numpy() > 0 for l in range(1, k)]


def oracle_view(graph, n_parts=1, resident=None):
    return O.GraphView(graph.row_offsets.cpu().numpy(), graph.nbrs.cpu().numpy(), n_parts, resident)


def assert_dense_equal(view, ref):
    for key in ("node_ids", "node_id_offsets", "nbrs", "nbr_offsets", "repr_map"):
        got = getattr(view, key).cpu().numpy().tolist()
        assert got == ref[key], f"{key} differs"


def make_ctx(graph, feats=None, offsets_dtype=torch.int64):
    ctx = mg.Context(0)
    ctx.load_graph(graph.row_offsets.to(offsets_dtype).cuda(), graph.nbrs.cuda())
    if feats is not None:
        ctx.load_features(feats.cuda())
    return ctx


@pytest.fixture(scope="module")
def tiny():
    g = inputs.erdos_renyi_graph(10_000, 200_000, seed=0)
    feats = inputs.normal_features(10_000, 16, seed=1)
    return g, feats


def test_config1_sample_bit_exact(tiny):
    g, feats = tiny
    ctx = make_ctx(g, feats, torch.int32)
    targets = inputs.distinct_targets(10_000, 512, seed=2)
    d = ctx.sample(targets, [10, 5], seed=123)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [10, 5], 123)
    assert_dense_equal(d.view(0), ref)
    nodes, ents = d.counts()
    nio = ref["node_id_offsets"]
    assert nodes[0].tolist() == [nio[3] - nio[2], nio[2] - nio[1], nio[1] - nio[0]]
    assert int(ents.sum()) == len(ref["nbrs"])


def test_config1_forward(tiny):
    g, feats = tiny
    ctx = make_ctx(g, feats)
    targets = inputs.distinct_targets(10_000, 512, seed=3)
    layers = inputs.random_bias_layers([16, 16, 16], seed=4)
    d = ctx.sample(targets, [10, 5], seed=7)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [10, 5], 7)
    h0 = feats.numpy()[ref["node_ids"]]
    got_h0 = ctx.gather_h0(d, 0, len(ref["node_ids"]), 16).cpu().numpy()
    np.testing.assert_array_equal(got_h0, h0)
    ref_outs = O.forward(ref, h0, [(w.numpy(), n.numpy(), b.numpy()) for w, n, b in layers], return_all=True)
    for prec, rtol in ((mg.GEMM_FP32, RTOL_AGG), (mg.GEMM_TF32, RTOL_TC)):
        model = ctx.model(layers, prec)
        out = torch.empty((512, 16), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        close(out.cpu().numpy(), ref_outs[-1], rtol)
        l1 = ctx.layer_output(model, d, 1, 0, ref_outs[0].shape[0]).cpu().numpy()
        close(l1, ref_outs[0], rtol)
        host_out = torch.empty((512, 16), dtype=torch.float32)
        ctx.forward(model, d, host_out)
        np.testing.assert_array_equal(host_out.numpy(), out.cpu().numpy())


def test_many_batches_match_single_and_oracle(tiny):
    g, feats = tiny
    ctx = make_ctx(g, feats)
    B, T = 7, 200
    sizes = [T, 0, 13, T, 1, 300, 64]
    tg = [inputs.distinct_targets(10_000, s, seed=10 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [1000 + 17 * i for i in range(B)]
    d = ctx.sample_many(torch.cat(tg), offs, [4, 3, 2], seeds)
    view = oracle_view(g)
    layers = inputs.random_bias_layers([16, 8, 8, 4], seed=5)
    model = ctx.model(layers, mg.GEMM_FP32)
    out = torch.empty((int(offs[-1]), 4), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    for b in range(B):
        ref = O.sample_dense(view, tg[b].tolist(), [4, 3, 2], seeds[b])
        assert_dense_equal(d.view(b), ref)
        if sizes[b]:
            ref_out = O.forward(ref, feats.numpy()[ref["node_ids"]], [(w.numpy(), n.numpy(), bb.numpy()) for w, n, bb in layers])
            close(out[offs[b]:offs[b + 1]].cpu().numpy(), ref_out, RTOL_AGG)
    # device-resident targets give the same sample; so does reusing the handle
    d2 = ctx.sample_many(torch.cat(tg).cuda(), offs, [4, 3, 2], seeds, out=d)
    assert d2 is d
    # the device keeps a delta in discovery order and the views translate to ascending ids; the forward pass does
    # not depend on the order, bit for bit, and viewing a mini-batch changes nothing on the device
    before = torch.empty_like(out)
    ctx.forward(model, d, before)
    assert_dense_equal(d.view(3), O.sample_dense(view, tg[3].tolist(), [4, 3, 2], seeds[3]))
    after = torch.empty_like(out)
    ctx.forward(model, d, after)
    assert torch.equal(before, out) and torch.equal(after, out)
    assert_dense_equal(d.view(0), O.sample_dense(view, tg[0].tolist(), [4, 3, 2], seeds[0]))   # idempotent


def test_export_of_all_mini_batches_at_once(tiny):
    """mg_dense_export_many: one sort for the whole sample gives every mini-batch's arrays in the paper's layout, bit
    for bit the oracle's and the per-batch view's; empty and one-target mini-batches included; the export runs beside
    a forward pass and is redone after the handle is sampled into again."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [200, 0, 13, 200, 1, 300, 64, 0]
    B = len(sizes)
    tg = [inputs.distinct_targets(10_000, s, seed=30 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    view = oracle_view(g)
    layers = inputs.random_bias_layers([16, 8, 8, 4], seed=5)
    model = ctx.model(layers, mg.GEMM_FP32)
    d = None
    for round_, fanouts in enumerate([[4, 3, 2], [6, 2], [1, 1, 1]]):
        seeds = [500 * round_ + 7 * i for i in range(B)]
        d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds, out=d)
        with pytest.raises(mg.MgError) as e:
            d.export_view(0)                         # a new sample: the previous export is gone
        assert e.value.code == -2
        d.export_many()
        if len(fanouts) == 3:
            out = torch.empty((int(offs[-1]), 4), dtype=torch.float32, device="cuda")
            ctx.forward(model, d, out)               # on the context's stream while the export runs on the sampling stream
        for b in range(B):
            ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b])
            assert_dense_equal(d.export_view(b), ref)
        assert_dense_equal(d.view(2), O.sample_dense(view, tg[2].tolist(), fanouts, seeds[2]))   # the per-batch path still works


def test_export_with_many_segments_and_segments_longer_than_a_tile():
    """The export sorts the ids inside their (mini-batch, delta) segments.  1,600 segments (more than the 1,024 the
    tile-table kernel takes per round, empty mini-batches among them), and, in a second sample, deltas of more than
    4,096 nodes (more than one sort tile per segment, the last one ragged): every checked mini-batch bit for bit the
    oracle's."""
    n = 60_000
    g = inputs.rmat_graph(n, 1_200_000, seed=41)
    ctx = make_ctx(g)
    view = oracle_view(g)
    # many short segments
    B = 400
    sizes = [(3 if b % 7 else 0) + (b % 3) for b in range(B)]
    tg = [inputs.distinct_targets(n, s_, seed=1000 + b) for b, s_ in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [11 * b + 1 for b in range(B)]
    fanouts = [3, 2, 2]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    d.export_many()
    for b in (0, 1, 7, 255, 256, 257, 341, 342, B - 2, B - 1):
        assert_dense_equal(d.export_view(b), O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]))
    # few long segments
    sizes = [1500, 2, 700]
    tg = [inputs.distinct_targets(n, s_, seed=2000 + b) for b, s_ in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    fanouts = [10, 6]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, [5, 6, 7])
    d.export_many()
    longest = 0
    for b in range(3):
        ref = O.sample_dense(view, tg[b].tolist(), fanouts, [5, 6, 7][b])
        assert_dense_equal(d.export_view(b), ref)
        longest = max(longest, int(np.diff(np.asarray(ref["node_id_offsets"])).max()))
    assert longest > 4096   # (the case is what it claims to be)


@pytest.mark.parametrize("fanouts", [[1], [3, 1], [33, 2], [40, 70]])
def test_odd_fanouts(fanouts):
    g = inputs.rmat_graph(3000, 60_000, seed=3)
    ctx = make_ctx(g)
    targets = inputs.distinct_targets(3000, 50, seed=1)
    d = ctx.sample(targets, fanouts, seed=99)
    assert_dense_equal(d.view(0), O.sample_dense(oracle_view(g), targets.tolist(), fanouts, 99))


def test_full_fanout_is_exact_neighbourhood():
    g = inputs.erdos_renyi_graph(500, 3000, seed=8)
    ctx = make_ctx(g)
    maxdeg = int((g.row_offsets[1:] - g.row_offsets[:-1]).max())
    targets = torch.tensor([4, 99, 250], dtype=torch.int32)
    d = ctx.sample(targets, [maxdeg, maxdeg], seed=0)
    assert_dense_equal(d.view(0), O.sample_dense(oracle_view(g), targets.tolist(), [maxdeg, maxdeg], 0))


def test_run_to_run_determinism(tiny):
    g, _ = tiny
    ctx = make_ctx(g)
    targets = inputs.distinct_targets(10_000, 512, seed=5)
    a = ctx.sample(targets, [10, 5], seed=1).view(0)
    b = ctx.sample(targets, [10, 5], seed=1).view(0)
    for key in ("node_ids", "nbrs", "nbr_offsets", "repr_map"):
        assert torch.equal(getattr(a, key), getattr(b, key))
    c = ctx.sample(targets, [10, 5], seed=2).view(0)
    assert not torch.equal(a.nbrs, c.nbrs) or a.nbrs.numel() != c.nbrs.numel()


def test_errors(tiny):
    g, feats = tiny
    ctx = make_ctx(g, feats)
    t = torch.tensor([1, 2, 3], dtype=torch.int32)
    with pytest.raises(mg.MgError) as e:
        ctx.sample(torch.tensor([1, 2, 1], dtype=torch.int32), [2], 0)
    assert e.value.code == -4
    with pytest.raises(mg.MgError) as e:
        ctx.sample(torch.tensor([1, 10_000], dtype=torch.int32), [2], 0)
    assert e.value.code == -1
    with pytest.raises(mg.MgError) as e:
        ctx.sample(t, [0], 0)
    assert e.value.code == -1
    with pytest.raises(mg.MgError) as e:
        ctx.sample(t, [5, 5], 0, caps={"max_entries_total": 4})
    assert e.value.code == -5
    with pytest.raises(mg.MgError) as e:
        ctx.sample(inputs.distinct_targets(10_000, 100, 0), [10, 10], 0, caps={"max_nodes_total": 150})
    assert e.value.code == -5
    # the context stays usable after every failure
    d = ctx.sample(t, [2], 0)
    assert d.view(0).node_ids.numel() >= 3
    empty = mg.Context(0)
    with pytest.raises(mg.MgError) as e:
        empty.sample(t, [2], 0)
    assert e.value.code == -2
    # a model whose depth differs from the sample
    model = ctx.model(inputs.glorot_layers([16, 16, 16], 0), mg.GEMM_FP32)
    with pytest.raises(mg.MgError) as e:
        ctx.forward(model, d, torch.empty((3, 16), device="cuda"))
    assert e.value.code == -2


def test_partition_buffer_filter_and_host_backing():
    n, parts, cap = 6000, 6, 3
    g = inputs.rmat_graph(n, 90_000, seed=4)
    feats16 = inputs.normal_features(n, 24, seed=2, dtype=torch.float16, pin=False).pin_memory()
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(parts)
    ctx.load_features(feats16, capacity_parts=cap, backing=mg.BACKING_HOST)
    layers = inputs.random_bias_layers([24, 8, 8], seed=6)
    model = ctx.model(layers, mg.GEMM_FP32)
    states = inputs.swap_order(parts, cap, seed=1)
    assert len(states) == parts - cap + 1
    for step, resident in enumerate(states):
        ctx.set_resident(resident, async_=True)
        ctx.commit_resident(10_000)
        mask = inputs.resident_node_mask(n, parts, resident)
        pool = torch.nonzero(mask).flatten()
        targets = inputs.distinct_targets(pool, 64, seed=step)
        d = ctx.sample(targets, [5, 3], seed=50 + step)
        view = oracle_view(g, parts, resident)
        ref = O.sample_dense(view, targets.tolist(), [5, 3], 50 + step)
        assert_dense_equal(d.view(0), ref)
        assert all(view.is_resident(u) for u in ref["node_ids"])
        out = torch.empty((64, 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        h0 = feats16.float().numpy()[ref["node_ids"]]
        np.testing.assert_array_equal(ctx.gather_h0(d, 0, len(ref["node_ids"]), 24).cpu().numpy(), h0)
        ref_out = O.forward(ref, h0, [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers])
        close(out.cpu().numpy(), ref_out, RTOL_AGG)
    # a target outside the buffer is refused
    outside = int(torch.nonzero(~inputs.resident_node_mask(n, parts, states[-1])).flatten()[0])
    with pytest.raises(mg.MgError) as e:
        ctx.sample(torch.tensor([outside], dtype=torch.int32), [2], 0)
    assert e.value.code == -3
    with pytest.raises(mg.MgError) as e:
        ctx.set_resident([0, 1, 2, 3])
    assert e.value.code == -5


def test_commit_timeout_keeps_the_old_set_and_stale_samples_are_refused():
    """The one bounded host wait: a commit with no time to wait returns MG_ERR_TIMEOUT while the partition copies
    are still running, the committed set stays in use, and a later commit with a real deadline succeeds.  A sample
    drawn under a set that lost a partition is refused afterwards (its feature rows are gone), host-side, before
    any kernel runs; a sample whose partitions all kept their slots is not."""
    n, parts, dim = 4_000_000, 8, 128
    g = inputs.rmat_graph(n, 20_000_000, seed=61, device="cuda")
    feats = torch.empty((n, dim), dtype=torch.float32).pin_memory()
    gen = torch.Generator(device="cuda"); gen.manual_seed(62)
    for lo in range(0, n, 1 << 20):
        hi = min(n, lo + (1 << 20))
        feats[lo:hi].copy_(torch.randn((hi - lo, dim), generator=gen, device="cuda"))
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets, g.nbrs)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    ctx.set_partitioning(parts)
    ctx.load_features(feats, capacity_parts=5, backing=mg.BACKING_HOST)
    layers = inputs.glorot_layers([dim, 32, 16], seed=63)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    model = ctx.model(layers, mg.GEMM_FP32)
    old, new, grown = [0, 1], [1, 4, 5, 6, 7], [1, 4, 5, 6, 7]
    ctx.set_resident(old)

    def check(resident, seed):
        pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident)).flatten()
        tg = inputs.distinct_targets(pool, 300, seed=seed)
        d = ctx.sample(tg, [5, 3], seed=seed)
        out = torch.empty((300, 16), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        ref = O.sample_dense(O.GraphView(g_host[0], g_host[1], parts, resident), tg.tolist(), [5, 3], seed)
        assert_dense_equal(d.view(0), ref)
        close(out.cpu().numpy(), O.forward(ref, feats[torch.as_tensor(ref["node_ids"])].numpy(), np_layers), RTOL_AGG)
        return d, out

    d_old, out_old = check(old, 1)
    ctx.set_resident(new, async_=True)            # four partitions of 256 MB each from host memory: tens of milliseconds
    with pytest.raises(mg.MgError) as e:
        ctx.commit_resident(0)
    assert e.value.code == -7
    check(old, 2)                                 # the old set is still the committed one
    with pytest.raises(mg.MgError) as e:
        ctx.set_resident(new, async_=True)        # one pending set at a time
    assert e.value.code == -2
    ctx.commit_resident(60_000)
    check(new, 3)
    # partition 0 left the buffer: the old sample's rows are gone
    out = torch.empty((300, 16), dtype=torch.float32, device="cuda")
    for call in (lambda: ctx.forward(model, d_old, out), lambda: ctx.forward_noalloc(model, d_old, out),
                 lambda: ctx.gather_h0(d_old, 0, 1, dim)):
        with pytest.raises(mg.MgError) as e:
            call()
        assert e.value.code == -2 and "resident" in str(e.value)
    # a set that only grows keeps every slot: a sample drawn before the commit stays usable
    ctx.set_resident([1, 4])
    d_small, out_small = check([1, 4], 4)
    ctx.set_resident([1, 4, 6])
    again = torch.empty_like(out_small)
    ctx.forward(model, d_small, again)
    assert torch.equal(again, out_small)


@pytest.mark.parametrize("backing", ["hbm", "host"])
def test_partition_id_array_with_training_nodes_in_the_first_partitions(backing):
    """A partition id per node instead of contiguous ranges (Section 5.2's policy: the training nodes fill the first
    partitions, every other node sits in a random one of the rest).  Sampling under the buffer, the forward pass, H^0
    rows and link-prediction negatives against the oracle given the same array; host backing reads a partition-major
    table (a partition's rows in ascending id) through the buffer's slots and swaps a partition in."""
    n, parts, dim = 60_000, 8, 32
    g = inputs.rmat_graph(n, 900_000, seed=71)
    feats = inputs.normal_features(n, dim, seed=72)
    train = torch.randperm(n, generator=torch.Generator().manual_seed(73))[:9000]
    pn = inputs.training_first_partitioning(n, parts, train, seed=74)
    assert int(pn[train].max()) == 1                         # 9,000 training nodes fill partitions 0 and 1 (7,500 each)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(parts, pn)
    if backing == "hbm":
        ctx.load_features(feats.cuda(), capacity_parts=4)
    else:
        order = torch.argsort(pn.long() * n + torch.arange(n))                    # partition-major, ascending id inside
        ctx.load_features(feats[order].contiguous().pin_memory(), capacity_parts=4, backing=mg.BACKING_HOST)
    layers = inputs.random_bias_layers([dim, 16, 8], seed=75)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    model = ctx.model(layers, mg.GEMM_FP32)
    g_host = (g.row_offsets.numpy(), g.nbrs.numpy())
    for step, resident in enumerate([[0, 1, 5], [1, 0, 5, 6], [0, 1, 2, 6]]):
        ctx.set_resident(resident)
        view = O.GraphView(g_host[0], g_host[1], parts, resident, part_of_node=pn.numpy())
        tg = train[torch.randperm(9000, generator=torch.Generator().manual_seed(80 + step))[:400]].to(torch.int32)
        d = ctx.sample(tg, [6, 4], seed=90 + step)
        ref = O.sample_dense(view, tg.tolist(), [6, 4], 90 + step)
        assert_dense_equal(d.view(0), ref)
        assert all(view.is_resident(u) for u in ref["node_ids"])
        np.testing.assert_array_equal(ctx.gather_h0(d, 0, len(ref["node_ids"]), dim).cpu().numpy(), feats.numpy()[ref["node_ids"]])
        out = torch.empty((400, 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        close(out.cpu().numpy(), O.forward(ref, feats.numpy()[ref["node_ids"]], np_layers), RTOL_AGG)
        model_tc = ctx.model(layers, mg.GEMM_TF32)
        ctx.forward(model_tc, d, out)
        close(out.cpu().numpy(), O.forward(ref, feats.numpy()[ref["node_ids"]], np_layers), RTOL_TC)
        # link prediction: negatives are drawn among the resident nodes, partition after partition
        mask = inputs.resident_node_mask(n, parts, resident, part_of_node=pn)
        src, rel, dst = inputs.lp_edges(g, mask, 300, seed=step)
        lp = ctx.lp_prepare(src, rel, dst, 3, 50, seed=7 + step)
        prep = O.lp_prepare(view, src.tolist(), dst.tolist(), 3, 50, 7 + step)
        got = lp.view()
        for key in ("targets", "src_idx", "dst_idx", "neg_ids", "neg_idx"):
            assert got[key].cpu().tolist() == prep[key], key
    with pytest.raises(mg.MgError) as e:
        ctx.sample(torch.tensor([int(torch.nonzero(pn == 7)[0])], dtype=torch.int32), [2], seed=0)   # partition 7 is not resident
    assert e.value.code == -3
    with pytest.raises(mg.MgError) as e:
        ctx.set_partitioning(4, pn)                          # ids up to 7 do not fit 4 partitions
    assert e.value.code == -1


def test_link_prediction_distmult():
    n, parts, cap = 8000, 4, 2
    g = inputs.rmat_graph(n, 100_000, seed=5, n_relations=37)
    emb = inputs.normal_features(n, 20, seed=3, std=0.001)
    rel_emb = inputs.normal_features(37, 12, seed=9)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(parts)
    ctx.load_features(emb.cuda(), capacity_parts=cap)
    resident = [1, 3]
    ctx.set_resident(resident)
    mask = inputs.resident_node_mask(n, parts, resident)
    src, rel, dst = inputs.lp_edges(g, mask, 500, seed=1)
    n_chunks, negs = 3, 70
    lp = ctx.lp_prepare(src, rel, dst, n_chunks, negs, seed=2024)
    view = oracle_view(g, parts, resident)
    prep = O.lp_prepare(view, src.tolist(), dst.tolist(), n_chunks, negs, 2024)
    got = lp.view()
    assert got["targets"].cpu().tolist() == prep["targets"]
    assert lp.targets().cpu().tolist() == prep["targets"]     # (the accessor that builds the target tensor alone)
    assert got["src_idx"].cpu().tolist() == prep["src_idx"]
    assert got["dst_idx"].cpu().tolist() == prep["dst_idx"]
    assert got["neg_ids"].cpu().tolist() == prep["neg_ids"]
    assert got["neg_idx"].cpu().tolist() == prep["neg_idx"]
    # one GraphSage layer over the targets, then DistMult
    layers = inputs.random_bias_layers([20, 12], seed=8)
    model = ctx.model(layers, mg.GEMM_FP32)
    d = ctx.sample(got["targets"], [20], seed=5)
    ref = O.sample_dense(view, prep["targets"], [20], 5)
    assert_dense_equal(d.view(0), ref)
    h = torch.empty((len(prep["targets"]), 12), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, h)
    ref_h = O.forward(ref, emb.numpy()[ref["node_ids"]], [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers])
    close(h.cpu().numpy(), ref_h, RTOL_AGG)
    rpos, rnd, rns = O.distmult_scores(ref_h, rel_emb.numpy(), prep, rel.tolist(), n_chunks)
    for prec, rtol in ((mg.GEMM_FP32, RTOL_AGG), (mg.GEMM_TF32, RTOL_TC)):
        pos, nd, ns = ctx.distmult_score(lp, h, rel_emb.cuda(), precision=prec)
        torch.cuda.synchronize()
        close(pos.cpu().numpy(), rpos, RTOL_AGG)      # positives are always fp32
        close(nd.cpu().numpy(), rnd, rtol)
        close(ns.cpu().numpy(), rns, rtol)
    # one corrupted side only
    pos, nd, ns = ctx.distmult_score(lp, h, rel_emb.cuda(), corrupt=mg.CORRUPT_DST)
    assert ns is None
    close(nd.cpu().numpy(), rnd, RTOL_TC)


@pytest.mark.parametrize("dim,n_edges,n_chunks,negs", [(100, 700, 3, 1000), (32, 129, 1, 17), (128, 300, 7, 256),
                                                       (32, 60_000, 5, 72)])
def test_distmult_tensor_core_shapes(dim, n_edges, n_chunks, negs):
    """DistMult negatives on the tensor cores: padded K, several blocks of negatives, ragged chunks; the last case
    has more than three tiles per SM."""
    n = 30_000
    g = inputs.rmat_graph(n, 300_000, seed=6, n_relations=11)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    src, rel, dst = inputs.lp_edges(g, None, n_edges, seed=2)
    lp = ctx.lp_prepare(src, rel, dst, n_chunks, negs, seed=7)
    view = oracle_view(g)
    prep = O.lp_prepare(view, src.tolist(), dst.tolist(), n_chunks, negs, 7)
    assert lp.view()["neg_idx"].cpu().tolist() == prep["neg_idx"]
    h = inputs.normal_features(len(prep["targets"]), dim, seed=4)
    rel_emb = inputs.normal_features(11, dim, seed=5)
    pos, nd, ns = ctx.distmult_score(lp, h.cuda(), rel_emb.cuda())
    torch.cuda.synchronize()
    rpos, rnd, rns = O.distmult_scores(h.numpy(), rel_emb.numpy(), prep, rel.tolist(), n_chunks)
    close(pos.cpu().numpy(), rpos, RTOL_AGG)
    close(nd.cpu().numpy(), rnd, RTOL_TC)
    close(ns.cpu().numpy(), rns, RTOL_TC)


@pytest.mark.parametrize("d_in,d_out", [(100, 100), (256, 256), (128, 256), (768, 256), (16, 520), (36, 4)])
def test_tensor_core_linear_layer_shapes(d_in, d_out):
    """One GraphSage layer at the widths of the five configurations (and ragged ones): several
    K slices, ring wrap-around, padded N tiles, more than one N tile, a ragged last row tile."""
    n = 5000
    g = inputs.rmat_graph(n, 60_000, seed=11)
    feats = inputs.normal_features(n, d_in, seed=12)
    ctx = make_ctx(g, feats)
    targets = inputs.distinct_targets(n, 777, seed=13)
    d = ctx.sample(targets, [6], seed=3)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [6], 3)
    assert_dense_equal(d.view(0), ref)
    layers = inputs.random_bias_layers([d_in, d_out], seed=14)
    want = O.forward(ref, feats.numpy()[ref["node_ids"]], [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers])
    for prec, rtol in ((mg.GEMM_TF32, RTOL_TC), (mg.GEMM_FP32, RTOL_AGG)):
        out = torch.empty((777, d_out), dtype=torch.float32, device="cuda")
        ctx.forward(ctx.model(layers, prec), d, out)
        close(out.cpu().numpy(), want, rtol)


@pytest.mark.parametrize("d_in,d_out,fanout", [(8, 16, 6), (72, 100, 6), (256, 256, 6), (264, 64, 3), (768, 256, 6), (200, 36, 30)])
def test_first_layer_on_fp16_operands(d_in, d_out, fanout):
    """Half-precision base representations: the first layer's GEMM runs on fp16 operands (fp16 rows as they are, the
    mean and the weights rounded to fp16, fp32 accumulate).  Widths below one 64-column slice, ragged slices, one and
    several 256-column groups, rows past the entry cache (fanout 30); a second layer on TF32 operands behind it; the
    sum aggregator and weights outside fp16's comfortable range keep TF32 operands and must agree as well."""
    n = 5000
    g = inputs.rmat_graph(n, 60_000, seed=11)
    feats = inputs.normal_features(n, d_in, seed=12).half()
    ctx = make_ctx(g, feats)
    targets = inputs.distinct_targets(n, 777, seed=13)
    d = ctx.sample(targets, [fanout, 4], seed=3)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [fanout, 4], 3)
    assert_dense_equal(d.view(0), ref)
    h0 = feats.float().numpy()[ref["node_ids"]]
    out = torch.empty((777, 8), dtype=torch.float32, device="cuda")
    for scale, aggregator in ((1.0, "mean"), (1.0, "sum"), (1e-5, "mean")):
        layers = inputs.random_bias_layers([d_in, d_out, 8], seed=14)
        layers[0] = (layers[0][0] * scale, layers[0][1] * scale, layers[0][2] * scale)
        np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
        model = ctx.model(layers, mg.GEMM_TF32)
        model.set_aggregator(aggregator)
        ctx.keep_layer_outputs(True)
        ctx.forward(model, d, out)
        outs = O.forward(ref, h0, np_layers, return_all=True, aggregator=aggregator)
        close(ctx.layer_output(model, d, 1, 0, outs[0].shape[0]).cpu().numpy(), outs[0], RTOL_TC)
        close(out.cpu().numpy(), outs[1], RTOL_TC)
        ctx.keep_layer_outputs(False)


@pytest.mark.parametrize("dims", [[128, 256, 256, 256], [64, 128, 128], [16, 128, 100, 128, 8]])
def test_fp16_intermediate_layer_outputs(dims):
    """The model option that keeps H^1 .. H^{k-1} as fp16 inside the forward pass: H^k within the tensor-core tolerance
    of the fp64 oracle, several mini-batches with ragged tiles; where the option cannot apply (an intermediate width
    that is not a multiple of 128, kept layer outputs, the sum aggregator) the fp32 path answers, equally checked."""
    n = 30_000
    g = inputs.rmat_graph(n, 600_000, seed=21)
    feats = inputs.normal_features(n, dims[0], seed=22)
    ctx = make_ctx(g, feats)
    k = len(dims) - 1
    fanouts = [6, 4, 3, 2][:k]
    sizes = [300, 1, 257]
    tg = [inputs.distinct_targets(n, s_, seed=23 + i) for i, s_ in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [7, 8, 9]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    layers = inputs.random_bias_layers(dims, seed=24)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    view = oracle_view(g)
    refs = [O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]) for b in range(3)]
    model = ctx.model(layers, mg.GEMM_TF32)
    out32 = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out32)
    model.set_intermediates(torch.float16)
    for aggregator, keep in (("mean", False), ("mean", True), ("sum", False)):
        model.set_aggregator(aggregator)
        ctx.keep_layer_outputs(keep)
        out = torch.full_like(out32, float("nan"))
        ctx.forward(model, d, out)
        for b in range(3):
            want = O.forward(refs[b], feats.numpy()[refs[b]["node_ids"]], np_layers, aggregator=aggregator)
            close(out[offs[b]:offs[b + 1]].cpu().numpy(), want, RTOL_TC)
        if aggregator == "mean" and not keep and all(w % 128 == 0 for w in dims[1:-1]):
            assert not torch.equal(out, out32)          # the fp16 path really ran (its rounding differs)
            with pytest.raises(mg.MgError):
                ctx.layer_output(model, d, 1, 0, 1)       # and kept no fp32 layer outputs
    ctx.keep_layer_outputs(False)


@pytest.mark.parametrize("dims,fanouts,fp16_feats", [([128, 256, 256], [5, 4], False), ([96, 200, 36], [3, 6], False),
                                                     ([128, 256, 128], [4, 4], True), ([128, 128, 64], [20, 3], False)])
def test_layer_weights_in_tensor_memory_and_streamed(dims, fanouts, fp16_feats, monkeypatch):
    """The fused layer kernel keeps a layer's weights in tensor memory (as the MMAs' first operand, the accumulator
    transposed) when all of K fits there and the layer's rows are short, and streams them through shared memory
    otherwise.  Both forms on the same sample: each within the tensor-core tolerance of the fp64 oracle and next to
    each other; widths that are no multiples of 32, ragged tiles, a mini-batch of one target, fp16 base
    representations, fp16 intermediates, and a layer of long rows (which streams in either case)."""
    n = 40_000
    g = inputs.rmat_graph(n, 700_000, seed=31)
    feats = inputs.normal_features(n, dims[0], seed=32)
    table = feats.half() if fp16_feats else feats
    ctx = make_ctx(g, table)
    sizes = [513, 1, 130]
    tg = [inputs.distinct_targets(n, s_, seed=33 + i) for i, s_ in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [17, 18, 19]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    layers = inputs.random_bias_layers(dims, seed=34)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    view = oracle_view(g)
    base = table.float().numpy()
    want = []
    for b in range(3):
        ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b])
        want.append(O.forward(ref, base[ref["node_ids"]], np_layers))
    model = ctx.model(layers, mg.GEMM_TF32)
    got = {}
    for intermediates in (torch.float32, torch.float16):
        model.set_intermediates(intermediates)
        for streamed in (False, True):
            if streamed:
                monkeypatch.setenv("MG_FUSED_NO_TS", "1")
            else:
                monkeypatch.delenv("MG_FUSED_NO_TS", raising=False)
            out = torch.full((int(offs[-1]), dims[-1]), float("nan"), dtype=torch.float32, device="cuda")
            ctx.forward(model, d, out)
            got[(intermediates, streamed)] = out.cpu().numpy()
            for b in range(3):
                close(got[(intermediates, streamed)][offs[b]:offs[b + 1]], want[b], RTOL_TC)
        # the two forms contract the same TF32 (or fp16) operands in the same K order
        close(got[(intermediates, False)], got[(intermediates, True)], 3e-4)
    monkeypatch.delenv("MG_FUSED_NO_TS", raising=False)


def test_config2_shaped_power_law_three_layers():
    """R-MAT, dim 128, hidden 256, fanouts [15, 10, 5], batches of 1000 (config 2 at 1/5 scale so
    the oracle finishes in seconds); hub rows, zero-degree nodes, several batches per pass."""
    n = 200_000
    g = inputs.rmat_graph(n, 4_000_000, seed=21)
    feats = inputs.normal_features(n, 128, seed=22)
    ctx = make_ctx(g, feats)
    B = 4
    tg = inputs.train_set_batches(n, 20_000, 1000, B, seed=23)
    offs = [1000 * i for i in range(B + 1)]
    seeds = [7 + i for i in range(B)]
    d = ctx.sample_many(tg.flatten(), offs, [15, 10, 5], seeds)
    layers = inputs.glorot_layers([128, 256, 256, 256], seed=24)
    model = ctx.model(layers, mg.GEMM_TF32)
    out = torch.empty((B * 1000, 256), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    view = oracle_view(g)
    for b in (0, B - 1):
        ref = O.sample_dense(view, tg[b].tolist(), [15, 10, 5], seeds[b])
        assert_dense_equal(d.view(b), ref)
        outs = O.forward(ref, feats.numpy()[ref["node_ids"]], [(w.numpy(), nn.numpy(), bb.numpy()) for w, nn, bb in layers],
                         return_all=True)
        close(out[b * 1000:(b + 1) * 1000].cpu().numpy(), outs[-1], RTOL_TC)
        for layer in (1, 2):
            got = ctx.layer_output(model, d, layer, b, outs[layer - 1].shape[0]).cpu().numpy()
            close(got, outs[layer - 1], RTOL_TC)


def _check_batches_against_oracle(g_host, feats, layers, fanouts, targets_by_batch, seeds, dense, out, offs, batches, rtol):
    inout = len(g_host) > 2
    view = O.GraphView(g_host[0], g_host[1], out_row_offsets=g_host[2] if inout else None, out_nbrs=g_host[3] if inout else None)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    for b in batches:
        ref = O.sample_dense(view, targets_by_batch[b].tolist(), fanouts, seeds[b], "inout" if inout else "in")
        assert_dense_equal(dense.view(b), ref)
        ids = torch.as_tensor(ref["node_ids"], dtype=torch.int64, device=feats.device)
        want = O.forward(ref, feats[ids].float().cpu().numpy(), np_layers)
        close(out[offs[b]:offs[b + 1]].cpu().numpy(), want, rtol)


def test_full_size_config2_in_bench_launch_configuration():
    """Config 2 at full size (R-MAT 1M nodes / 20M edges, dim 128, hidden 256, [15, 10, 5], 1000 targets),
    128 mini-batches per pass as bench.py runs it; three of the batches checked against the oracle."""
    import bench
    cfg = bench.CONFIGS["config2_rmat_1m"]
    g, feats, layers, _ = bench.build_workload(cfg, torch.device("cuda"), seed=0)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets, g.nbrs)
    ctx.load_features(feats)
    G, T = 128, cfg["batch"]
    tg = inputs.train_set_batches(cfg["n"], cfg["train"], T, G, seed=100)
    offs = [T * i for i in range(G + 1)]
    seeds = list(range(G))
    d = ctx.sample_many(tg.reshape(-1).cuda(), offs, cfg["fanouts"], seeds)
    model = ctx.model(layers, mg.GEMM_TF32)
    out = torch.empty((G * T, cfg["hidden"]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    _check_batches_against_oracle(g_host, feats, layers, cfg["fanouts"], tg, seeds, d, out, offs, [0, 77, G - 1], RTOL_TC)
    # backward pass at the same size: a loss that only looks at mini-batch 77 leaves gradients the oracle can compute
    # from that mini-batch alone.  The forward pass ran in TF32, so a pre-activation within rounding of zero may sit on
    # the other side of the ReLU than in fp64: the oracle differentiates the branch the GPU took (the sign pattern of
    # its kept layer outputs), and every gradient entry is then compared on its own.
    ctx.keep_layer_outputs(True)
    ctx.forward(model, d, out)
    b = 77
    g_out = torch.zeros_like(out)
    g_out[offs[b]:offs[b + 1]] = torch.randn((T, cfg["hidden"]), generator=torch.Generator().manual_seed(1)).cuda()
    grads, g_h0, ids = ctx.backward(model, d, g_out, want_h0_grad=True)
    ref = O.sample_dense(O.GraphView(g_host[0], g_host[1]), tg[b].tolist(), cfg["fanouts"], seeds[b])
    nid = torch.as_tensor(ref["node_ids"], dtype=torch.int64, device=feats.device)
    np_layers = [(w.numpy(), nn.numpy(), bb.numpy()) for w, nn, bb in layers]
    masks = gpu_relu_branch(ctx, model, d, b, ref)
    want, d_h0 = O.backward(ref, feats[nid].float().cpu().numpy(), np_layers, g_out[offs[b]:offs[b + 1]].cpu().numpy(),
                            relu_masks=masks)
    for l in range(len(np_layers)):
        for p in range(3):
            close(grads[l][p].cpu().numpy(), want[l][p], RTOL_TC)
            near(grads[l][p].cpu().numpy(), want[l][p], 5e-3)
    nodes, _ = d.counts()
    row0 = np.concatenate([[0], np.cumsum(nodes.sum(1).cpu().numpy())])
    lo, hi = int(row0[b]), int(row0[b + 1])
    where = {v: r for r, v in enumerate(ref["node_ids"])}
    ids_b = ids[lo:hi].cpu().numpy()
    close(g_h0[lo:hi].cpu().numpy(), d_h0[[where[int(v)] for v in ids_b]], RTOL_TC, per_row=True)
    near(g_h0[lo:hi].cpu().numpy(), d_h0[[where[int(v)] for v in ids_b]], 5e-3)
    assert not bool(g_h0[:lo].any()) and not bool(g_h0[hi:].any())     # the other mini-batches receive nothing


def test_full_size_config3_in_bench_launch_configuration():
    """Config 3 at full size (R-MAT 111M nodes / 1.62B edges, 16 partitions all resident, int64 offsets),
    128 mini-batches per pass with the capacities bench.py derives; two batches checked against the oracle."""
    import bench
    cfg = bench.CONFIGS["config3_papers100m_shaped"]
    free, _ = torch.cuda.mem_get_info()
    if free < 150 * (1 << 30):
        pytest.skip("needs a GPU with 150 GB free")
    g, feats, layers, _ = bench.build_workload(cfg, torch.device("cuda"), seed=0)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets, g.nbrs)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    gt = inputs.transpose_csr(g)          # the second edge list, for the incoming + outgoing part below
    del g
    torch.cuda.empty_cache()
    ctx.set_partitioning(cfg["parts"])
    ctx.load_features(feats, capacity_parts=cfg["parts"])
    ctx.set_resident(list(range(cfg["parts"])))
    G, T = 128, cfg["batch"]
    tg = inputs.train_set_batches(cfg["n"], cfg["train"], T, G, seed=100)
    offs = [T * i for i in range(G + 1)]
    seeds = [(1 << 40) + i for i in range(G)]
    probe = ctx.sample_many(tg.reshape(-1).cuda(), offs, cfg["fanouts"], seeds, caps={"max_nodes_per_batch": 1 << 19})
    nodes, ents = probe.counts()
    caps = {"max_nodes_total": int(nodes.sum() * 1.3) + 1024, "max_entries_total": int(ents.sum() * 1.3) + 1024,
            "max_nodes_per_batch": int(nodes.sum(1).max() * 1.5) + 64,
            "max_inner_nodes_per_batch": int(nodes[:, :-1].sum(1).max() * 1.5) + 64}
    probe.free()
    d = ctx.sample_many(tg.reshape(-1).cuda(), offs, cfg["fanouts"], seeds, caps=caps)
    model = ctx.model(layers, mg.GEMM_TF32)
    out = torch.empty((G * T, cfg["hidden"]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    _check_batches_against_oracle(g_host, feats, layers, cfg["fanouts"], tg, seeds, d, out, offs, [0, G - 1], RTOL_TC)
    # properties that hold at any size, on every batch: no duplicate node, every neighbour has a row
    n2, e2 = d.counts()
    assert torch.equal(n2, nodes) and torch.equal(e2, ents)          # same seeds, same sample
    for b in (1, 64):
        v = d.view(b)
        ids = v.node_ids.long()
        assert torch.unique(ids).numel() == ids.numel()
        assert torch.equal(ids[v.repr_map.long()], v.nbrs.long())
        nio = v.node_id_offsets.cpu().tolist()
        for j in range(len(nio) - 2):                                # deltas ascending (targets keep caller order)
            seg = ids[nio[j]:nio[j + 1]]
            assert bool((seg[1:] > seg[:-1]).all())
        assert ids[nio[-2]:].cpu().tolist() == tg[b].tolist()
    # the same graph sampled from incoming and outgoing edges (15 / 10 / 5 per direction), 16 mini-batches per pass as
    # bench.py's config3_papers100m_shaped_inout runs it; one mini-batch (about 600k nodes) checked against the oracle
    d.free()
    ctx.load_out_graph(gt.row_offsets, gt.nbrs)
    g_host = g_host + (gt.row_offsets.cpu().numpy(), gt.nbrs.cpu().numpy())
    del gt
    torch.cuda.empty_cache()
    ctx.set_sample_direction("inout")
    G2 = bench.CONFIGS["config3_papers100m_shaped_inout"]["group"]
    offs2 = offs[:G2 + 1]
    tg2 = tg[:G2].reshape(-1).cuda()
    probe = ctx.sample_many(tg2, offs2, cfg["fanouts"], seeds[:G2], caps={"max_nodes_per_batch": 1 << 23})
    nodes, ents = probe.counts()
    caps = {"max_nodes_total": int(nodes.sum() * 1.3) + 1024, "max_entries_total": int(ents.sum() * 1.3) + 1024,
            "max_nodes_per_batch": int(nodes.sum(1).max() * 1.5) + 64,
            "max_inner_nodes_per_batch": int(nodes[:, :-1].sum(1).max() * 1.5) + 64}
    probe.free()
    d = ctx.sample_many(tg2, offs2, cfg["fanouts"], seeds[:G2], caps=caps)
    out2 = torch.empty((G2 * T, cfg["hidden"]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out2)
    _check_batches_against_oracle(g_host, feats, layers, cfg["fanouts"], tg, seeds, d, out2, offs2, [G2 - 1], RTOL_TC)


def test_config4_out_of_core_at_its_stated_size():
    """Config 4 as stated: R-MAT 122M nodes / 1.30B edges, fp16 features of width 768, 32 partitions with a
    10-partition HBM buffer, in the launch configuration of bench.py's out-of-core workload.  The 187 GB table is never
    held: a partition block is a pure function of (seed, block), made into a pinned staging block when the buffer asks
    for it and made again for the oracle's H^0 rows.  Three buffer states of the random one-swap order; the next
    state's block is copied on the side stream while the current state's mini-batches run; only edges with both
    endpoints resident are sampled; one mini-batch per state is checked against the oracle."""
    import bench
    c = bench.OOC_CONFIG
    free, _ = torch.cuda.mem_get_info()
    if free < 110 * (1 << 30):
        pytest.skip("needs a GPU with 110 GB free")
    n, parts, cap, dim = c["n"], c["parts"], c["cap"], c["dim"]
    g = inputs.rmat_graph(n, c["m"], seed=40, device="cuda")
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets, g.nbrs)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    del g
    torch.cuda.empty_cache()
    ctx.set_partitioning(parts)
    ctx.load_features(None, capacity_parts=cap, backing=mg.BACKING_HOST, dtype=torch.float16, dim=dim)
    part_rows = inputs.contiguous_partition(n, parts)
    rows_of = lambda p: min(part_rows, n - p * part_rows)
    staging = [torch.empty((part_rows, dim), dtype=torch.float16).pin_memory() for _ in range(2)]

    def stage(p, slot):
        inputs.block_features(rows_of(p), dim, 41, p, device="cuda", dtype=torch.float16, out=staging[slot][:rows_of(p)])
        torch.cuda.synchronize()
        return staging[slot]

    with pytest.raises(mg.MgError) as e:
        ctx.set_resident([3])                       # no table and no block named for partition 3
    assert e.value.code == -2
    states = inputs.swap_order(parts, cap, seed=44)[:3]
    for i, p in enumerate(states[0]):
        ctx.set_partition_source(p, stage(p, 0))
        ctx.set_resident(sorted(states[0][:i + 1]))
    layers = inputs.glorot_layers([dim] + [c["hidden"]] * 3, seed=43)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    model = ctx.model(layers, mg.GEMM_TF32)
    G, T = c["group"], c["batch"]
    offs = [T * i for i in range(G + 1)]

    def oracle_h0(node_ids):
        ids = torch.as_tensor(node_ids, dtype=torch.int64)
        h0 = torch.empty((ids.numel(), dim), dtype=torch.float32)
        part = ids // part_rows
        for p in torch.unique(part).tolist():
            block = inputs.block_features(rows_of(p), dim, 41, p, device="cuda", dtype=torch.float16)
            sel = torch.nonzero(part == p).flatten()
            h0[sel] = block[(ids[sel] - p * part_rows).cuda()].float().cpu()
            del block
        return h0.numpy()

    for step, resident in enumerate(states):
        if step + 1 < len(states):
            q = [p for p in states[step + 1] if p not in resident][0]
            ctx.set_partition_source(q, stage(q, 1))
            ctx.set_resident(states[step + 1], async_=True)      # the incoming block loads on the side stream
        pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident, device="cuda")).flatten().to(torch.int32)
        gen = torch.Generator(device="cuda"); gen.manual_seed(500 + step)
        tg = pool[torch.randperm(pool.numel(), generator=gen, device="cuda")[:G * T]].reshape(G, T)
        seeds = [1000 * step + b for b in range(G)]
        probe = ctx.sample_many(tg.reshape(-1), offs, c["fanouts"], seeds, caps={"max_nodes_per_batch": 1 << 19})
        nodes, ents = probe.counts()
        caps = {"max_nodes_total": int(nodes.sum() * 1.4) + 1024, "max_entries_total": int(ents.sum() * 1.4) + 1024,
                "max_nodes_per_batch": int(nodes.sum(1).max() * 1.6) + 64,
                "max_inner_nodes_per_batch": int(nodes[:, :-1].sum(1).max() * 1.6) + 64}
        probe.free()
        d = ctx.sample_many(tg.reshape(-1), offs, c["fanouts"], seeds, caps=caps)
        out = torch.empty((G * T, c["hidden"]), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        view = O.GraphView(g_host[0], g_host[1], parts, resident)
        b = (17 * step + 5) % G
        ref = O.sample_dense(view, tg[b].tolist(), c["fanouts"], seeds[b])
        assert_dense_equal(d.view(b), ref)
        assert all(view.is_resident(u) for u in ref["node_ids"][::97])
        close(out[offs[b]:offs[b + 1]].cpu().numpy(), O.forward(ref, oracle_h0(ref["node_ids"]), np_layers), RTOL_TC)
        d.free()
        if step + 1 < len(states):
            ctx.commit_resident(120_000)


def test_config5_shaped_link_prediction_full_graph():
    """Config 5 as stated: R-MAT 86M nodes / 338M edges, 14,824 relations, embeddings of width 100 with std 0.001,
    16 partitions with 8 resident, a batch of 50,000 positive edges in 10 chunks of 1,000 shared negatives, one
    GraphSage layer with fanout 20 on the tensor cores, DistMult on the tensor cores -- the launch configuration of
    bench.py's link-prediction step.  Index arrays bit for bit; scores end to end against the fp64 oracle, and once
    more against the oracle fed the GPU's own H (which isolates the decoder's rounding)."""
    n, m, parts, cap, dim, nrel = 86_000_000, 338_000_000, 16, 8, 100, 14824
    g = inputs.rmat_graph(n, m, seed=5, device="cuda", n_relations=nrel)
    emb = inputs.normal_features(n, dim, seed=3, device="cuda", std=0.001)
    rel_emb = inputs.normal_features(nrel, dim, seed=9, device="cuda")
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets, g.nbrs)
    ctx.set_partitioning(parts)
    ctx.load_features(emb, capacity_parts=cap)
    resident = [0, 2, 3, 5, 8, 9, 12, 15]
    ctx.set_resident(resident)
    mask = inputs.resident_node_mask(n, parts, resident)
    n_edges, n_chunks, negs = 50_000, 10, 1000
    src, rel, dst = inputs.lp_edges(g, mask, n_edges, seed=1)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    del g
    lp = ctx.lp_prepare(src, rel, dst, n_chunks, negs, seed=2024)
    view = O.GraphView(g_host[0], g_host[1], parts, resident)
    prep = O.lp_prepare(view, src.tolist(), dst.tolist(), n_chunks, negs, 2024)
    got = lp.view()
    for key in ("targets", "src_idx", "dst_idx", "neg_ids", "neg_idx"):
        assert got[key].cpu().tolist() == prep[key], key
    layers = inputs.glorot_layers([dim, dim], seed=8)
    model = ctx.model(layers, mg.GEMM_TF32)
    d = ctx.sample(got["targets"], [20], seed=5)
    ref = O.sample_dense(view, prep["targets"], [20], 5)
    assert_dense_equal(d.view(0), ref)
    h = torch.empty((len(prep["targets"]), dim), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, h)
    ids = torch.as_tensor(ref["node_ids"], device="cuda")
    ref_h = O.forward(ref, emb[ids].cpu().numpy(), [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers])
    close(h.cpu().numpy(), ref_h, RTOL_TC)
    pos, nd, ns = ctx.distmult_score(lp, h, rel_emb)
    torch.cuda.synchronize()
    rel_h = rel_emb.cpu().numpy()
    # end to end: encoder and decoder both in TF32 on the GPU, both in fp64 in the oracle
    epos, end_, ens = O.distmult_scores(ref_h, rel_h, prep, rel.tolist(), n_chunks)
    close(pos.cpu().numpy(), epos, RTOL_TC)
    close(nd.cpu().numpy(), end_, RTOL_TC)
    close(ns.cpu().numpy(), ens, RTOL_TC)
    del epos, end_, ens
    # the decoder alone: the oracle fed the GPU's own H
    rpos, rnd, rns = O.distmult_scores(h.cpu().numpy(), rel_h, prep, rel.tolist(), n_chunks)
    close(pos.cpu().numpy(), rpos, RTOL_AGG)
    close(nd.cpu().numpy(), rnd, RTOL_TC)
    close(ns.cpu().numpy(), rns, RTOL_TC)


def test_async_host_output_equals_blocking_forward(tiny):
    g, feats = tiny
    ctx = make_ctx(g, feats)
    layers = inputs.random_bias_layers([16, 32, 8], seed=3)
    model = ctx.model(layers, mg.GEMM_TF32)
    outs_async = [torch.empty((300, 8), dtype=torch.float32).pin_memory() for _ in range(2)]
    want = []
    denses = []
    for i in range(2):
        targets = inputs.distinct_targets(10_000, 300, seed=20 + i)
        d = ctx.sample(targets, [6, 4], seed=i)
        ref = torch.empty((300, 8), dtype=torch.float32)
        ctx.forward(model, d, ref)
        want.append(ref)
        denses.append(d)
    for i in range(2):      # two copies in flight back to back, then one wait
        ctx.forward_host_async(model, denses[i], outs_async[i])
    ctx.wait_output()
    for i in range(2):
        assert torch.equal(outs_async[i], want[i])


@pytest.mark.parametrize("window", [1, 3, 16])
def test_windowed_layer_schedule_gives_the_same_output(tiny, window):
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [200, 0, 13, 200, 1, 300, 64, 128, 5]
    B = len(sizes)
    tg = [inputs.distinct_targets(10_000, s, seed=30 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    d = ctx.sample_many(torch.cat(tg), offs, [4, 3, 2], [500 + i for i in range(B)])
    layers = inputs.random_bias_layers([16, 32, 64, 8], seed=9)
    model = ctx.model(layers, mg.GEMM_TF32)
    want = torch.empty((int(offs[-1]), 8), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, want)
    ctx.set_layer_window(window)
    got = torch.full_like(want, float("nan"))
    ctx.forward(model, d, got)
    assert torch.equal(got, want)
    with pytest.raises(mg.MgError) as e:          # the windows do not keep H^1, H^2
        ctx.layer_output(model, d, 1, 0, 10)
    assert e.value.code == -2
    ctx.keep_layer_outputs(True)
    ctx.forward(model, d, got)
    assert torch.equal(got, want)
    nodes, _ = d.counts()
    assert ctx.layer_output(model, d, 1, 0, int(nodes[0, :3].sum())).shape[1] == 32


def test_sampling_overlapped_with_forward_matches_blocking_calls(tiny):
    """mg_sample_many_begin / _end: group i+1 is sampled on the sampling stream while group i runs its
    layers; results equal the blocking calls, and an unfinished sample cannot be used."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    layers = inputs.random_bias_layers([16, 32, 8], seed=3)
    model = ctx.model(layers, mg.GEMM_TF32)
    B, T, steps = 4, 150, 5
    offs = [T * i for i in range(B + 1)]
    tgs = [torch.cat([inputs.distinct_targets(10_000, T, seed=1000 * s + b) for b in range(B)]).cuda() for s in range(steps)]
    seeds = [[10 * s + b for b in range(B)] for s in range(steps)]
    want = []
    for s in range(steps):
        d = ctx.sample_many(tgs[s], offs, [6, 4], seeds[s])
        o = torch.empty((B * T, 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, o)
        want.append((o, d.view(B - 1).node_ids.clone()))
    denses = [None, None]
    denses[0] = ctx.sample_many_begin(tgs[0], offs, [6, 4], seeds[0])
    with pytest.raises(mg.MgError) as e:
        ctx.forward(model, denses[0], torch.empty((B * T, 8), dtype=torch.float32, device="cuda"))
    assert e.value.code == -2                       # still in flight
    outs = [torch.empty((B * T, 8), dtype=torch.float32, device="cuda") for _ in range(steps)]
    for s in range(steps):
        ctx.sample_many_end(denses[s & 1])
        if s + 1 < steps:
            denses[(s + 1) & 1] = ctx.sample_many_begin(tgs[s + 1], offs, [6, 4], seeds[s + 1], out=denses[(s + 1) & 1])
        ctx.forward(model, denses[s & 1], outs[s])
        assert torch.equal(denses[s & 1].view(B - 1).node_ids, want[s][1])
    for s in range(steps):
        assert torch.equal(outs[s], want[s][0])
    with pytest.raises(mg.MgError) as e:
        ctx.sample_many_end(denses[0])
    assert e.value.code == -2                       # nothing in flight
    # errors of an asynchronous sample surface at its end
    bad = ctx.sample_many_begin(torch.tensor([1, 1], dtype=torch.int32), [0, 2], [3], [0])
    with pytest.raises(mg.MgError) as e:
        ctx.sample_many_end(bad)
    assert e.value.code == -4


def test_extremes_largest_fanout_deepest_sample_all_nodes_empty_call():
    # a hub with 3000 in-neighbours and the largest supported fanout (1024): Floyd over a wide row
    n = 4000
    hub_src = torch.arange(1, 3001)
    src = torch.cat([hub_src, torch.randint(0, n, (20_000,), generator=torch.Generator().manual_seed(1))])
    dst = torch.cat([torch.zeros(3000, dtype=torch.int64), torch.randint(0, n, (20_000,), generator=torch.Generator().manual_seed(2))])
    g = inputs.build_csr(src, dst, n)
    ctx = make_ctx(g)
    view = oracle_view(g)
    t = torch.tensor([0, 5, 9], dtype=torch.int32)
    d = ctx.sample(t, [1024, 2], seed=3)
    ref = O.sample_dense(view, t.tolist(), [1024, 2], 3)
    assert_dense_equal(d.view(0), ref)
    assert np.diff(ref["nbr_offsets"])[-3] == 1024          # the hub keeps exactly the largest fanout
    with pytest.raises(mg.MgError) as e:
        ctx.sample(t, [1025], seed=3)
    assert e.value.code == -1
    # the deepest sample the library takes (8 hops), fanout 1 and 2
    d = ctx.sample(t, [2, 1, 2, 1, 2, 1, 2, 1], seed=4)
    assert_dense_equal(d.view(0), O.sample_dense(view, t.tolist(), [2, 1, 2, 1, 2, 1, 2, 1], 4))
    with pytest.raises(mg.MgError) as e:
        ctx.sample(t, [1] * 9, seed=4)
    assert e.value.code == -1
    # every node of the graph as a target: nothing new can be found, all deltas but the targets are empty
    allv = torch.arange(n, dtype=torch.int32)
    d = ctx.sample(allv, [3, 3], seed=5)
    ref = O.sample_dense(view, allv.tolist(), [3, 3], 5)
    assert_dense_equal(d.view(0), ref)
    assert ref["node_id_offsets"] == [0, 0, 0, n]
    # no targets at all
    d = ctx.sample(torch.empty(0, dtype=torch.int32), [3], seed=0)
    v = d.view(0)
    assert v.node_ids.numel() == 0 and v.nbrs.numel() == 0 and v.node_id_offsets.cpu().tolist() == [0, 0, 0]


def test_sample_handle_reuse_replays_and_recaptures(tiny):
    """The sampler's device work is captured in a CUDA graph per sample handle and replayed while the call's shape
    stays the same; targets, seeds and offsets of every call still take effect, and a new shape is captured anew."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    view = oracle_view(g)
    d = None
    for step, (fanouts, n) in enumerate([([6, 3], 200), ([6, 3], 200), ([6, 3], 200), ([4, 2, 2], 200), ([6, 3], 150)]):
        targets = inputs.distinct_targets(10_000, n, seed=40 + step)
        tg = targets.cuda() if step % 2 else targets
        offs = np.array([0, n // 2, n], dtype=np.int64)
        seeds = [7 * step + 1, 7 * step + 2]
        d = ctx.sample_many(tg, offs, fanouts, seeds, out=d)
        for b in range(2):
            ref = O.sample_dense(view, targets[offs[b]:offs[b + 1]].tolist(), fanouts, seeds[b])
            assert_dense_equal(d.view(b), ref)


def test_incoming_and_outgoing_sampling(tiny):
    """Section 4.1's second edge list: up to f incoming then up to f outgoing neighbours per node."""
    g, feats = tiny
    gt = inputs.transpose_csr(g)
    ctx = make_ctx(g, feats)
    with pytest.raises(mg.MgError) as e:
        ctx.set_sample_direction("inout")             # no outgoing list yet
    assert e.value.code == -2
    ctx.load_out_graph(gt.row_offsets.cuda(), gt.nbrs.cuda())
    ctx.set_sample_direction("inout")
    view = O.GraphView(g.row_offsets.numpy(), g.nbrs.numpy(), out_row_offsets=gt.row_offsets.numpy(), out_nbrs=gt.nbrs.numpy())
    layers = inputs.random_bias_layers([16, 16, 16, 8], seed=9)
    model = ctx.model(layers, mg.GEMM_FP32)
    sizes = [300, 1, 0, 257]
    tg = [inputs.distinct_targets(10_000, s, seed=40 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [77, 78, 79, 80]
    for fanouts in ([10, 5, 2], [40, 3, 1]):          # the second one takes the any-fanout pick kernel on the first hop
        d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
        out = torch.empty((int(offs[-1]), 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        for b in range(len(sizes)):
            ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b], direction="inout")
            assert_dense_equal(d.view(b), ref)
            if sizes[b]:
                ref_out = O.forward(ref, feats.numpy()[ref["node_ids"]], [(w.numpy(), n.numpy(), bb.numpy()) for w, n, bb in layers])
                close(out[offs[b]:offs[b + 1]].cpu().numpy(), ref_out, RTOL_AGG)
    # back to incoming-only sampling on the same context and handle
    ctx.set_sample_direction("in")
    d = ctx.sample_many(torch.cat(tg), offs, [10, 5, 2], seeds, out=d)
    assert_dense_equal(d.view(0), O.sample_dense(view, tg[0].tolist(), [10, 5, 2], seeds[0]))


def test_incoming_and_outgoing_sampling_under_the_buffer():
    n, parts = 6000, 6
    g = inputs.rmat_graph(n, 90_000, seed=4)
    gt = inputs.transpose_csr(g)
    feats = inputs.normal_features(n, 8, seed=2)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.load_out_graph(gt.row_offsets.to(torch.int32).cuda(), gt.nbrs.cuda())
    ctx.set_partitioning(parts)
    ctx.load_features(feats.cuda(), capacity_parts=parts)
    ctx.set_sample_direction("inout")
    for resident in ([0, 2, 5], [1, 2, 3, 4], list(range(parts))):
        ctx.set_resident(resident, async_=True)
        ctx.commit_resident(10_000)
        view = O.GraphView(g.row_offsets.numpy(), g.nbrs.numpy(), parts, resident, gt.row_offsets.numpy(), gt.nbrs.numpy())
        pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident)).flatten()
        targets = inputs.distinct_targets(pool, 100, seed=len(resident))
        d = ctx.sample(targets, [6, 4], seed=31)
        ref = O.sample_dense(view, targets.tolist(), [6, 4], 31, direction="inout")
        assert_dense_equal(d.view(0), ref)
        assert all(view.is_resident(u) for u in ref["node_ids"])


def test_sum_aggregator(tiny):
    """The neighbour term as a sum (Algorithm 3 as printed) instead of GraphSage's mean: fused TF32 layers, the
    unfused fp32 path, and identity weights = the printed additive layer."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    targets = inputs.distinct_targets(10_000, 300, seed=21)
    d = ctx.sample(targets, [7, 3], seed=5)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [7, 3], 5)
    h0 = feats.numpy()[ref["node_ids"]]
    layers = inputs.random_bias_layers([16, 32, 8], seed=3)
    np_layers = [(w.numpy(), n.numpy(), b.numpy()) for w, n, b in layers]
    want = O.forward(ref, h0, np_layers, aggregator="sum")
    want_mean = O.forward(ref, h0, np_layers)
    for prec, rtol in ((mg.GEMM_FP32, RTOL_AGG), (mg.GEMM_TF32, RTOL_TC)):
        model = ctx.model(layers, prec)
        out = torch.empty((300, 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, out)
        close(out.cpu().numpy(), want_mean, rtol)
        model.set_aggregator("sum")
        ctx.forward(model, d, out)
        close(out.cpu().numpy(), want, rtol)
        model.set_aggregator("mean")
        ctx.forward(model, d, out)
        close(out.cpu().numpy(), want_mean, rtol)
    eye = [(torch.eye(16), torch.eye(16), torch.zeros(16))]
    d1 = ctx.sample(targets, [7], seed=5)
    ref1 = O.sample_dense(oracle_view(g), targets.tolist(), [7], 5)
    model = ctx.model(eye, mg.GEMM_FP32)
    model.set_aggregator("sum")
    out = torch.empty((300, 16), dtype=torch.float32, device="cuda")
    ctx.forward(model, d1, out)
    close(out.cpu().numpy(), O.additive_layer(ref1, feats.numpy()[ref1["node_ids"]]), RTOL_AGG)


@pytest.mark.parametrize("cap_batch", [0, 60_000, 900_000])
def test_last_hop_deduplication_paths(tiny, cap_batch):
    """The last hop is deduplicated in shared memory when a mini-batch's node capacity fits a few table blocks
    (one block per mini-batch by default here, three buckets at 60,000) and through the global id table otherwise
    (900,000): the arrays are the oracle's either way."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [150, 0, 1, 400]
    tg = [inputs.distinct_targets(10_000, s, seed=60 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [5, 6, 7, 8]
    caps = {"max_nodes_per_batch": cap_batch} if cap_batch else None
    view = oracle_view(g)
    for fanouts in ([6], [5, 4], [3, 3, 3]):
        d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds, caps=caps)
        for b in range(len(sizes)):
            assert_dense_equal(d.view(b), O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]))
    # a repeated target is still refused on every path
    with pytest.raises(mg.MgError) as e:
        ctx.sample_many(torch.tensor([3, 9, 3], dtype=torch.int32), [0, 3], [2], [1], caps=caps)
    assert e.value.code == -4
    # a bound on the nodes that are sampled from (all but the farthest delta) shrinks the global id tables where the
    # last hop goes through shared memory: same arrays when the bound holds, a capacity error (nothing out of bounds)
    # when it does not
    if cap_batch != 900_000:
        fanouts = [5, 4, 3]
        refs = [O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]) for b in range(len(sizes))]
        inner = max(len(r["node_ids"]) - r["node_id_offsets"][1] for r in refs)
        tight = dict(caps or {"max_nodes_per_batch": 20_000}, max_inner_nodes_per_batch=inner)
        d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds, caps=tight)
        for b in range(len(sizes)):
            assert_dense_equal(d.view(b), refs[b])
        with pytest.raises(mg.MgError) as e:
            ctx.sample_many(torch.cat(tg), offs, fanouts, seeds, caps=dict(tight, max_inner_nodes_per_batch=inner // 3))
        assert e.value.code == -5


def test_comet_epoch_drives_the_partition_buffer():
    """One link-prediction epoch out of core under a COMET plan (Section 5.1): the plan's sets go through
    mg_set_resident / mg_commit_resident with host-backed embeddings, every set trains the edges of the buckets it
    was given, and every edge of the graph is trained exactly once; two of the sets are checked against the oracle
    end to end (negatives, target union, DENSE sample, layer, DistMult)."""
    n, p, l, c_l = 6000, 12, 6, 2
    g = inputs.rmat_graph(n, 40_000, seed=8, n_relations=11)
    emb = inputs.normal_features(n, 16, seed=4, std=0.01, pin=False).pin_memory()
    rel_emb = inputs.normal_features(11, 8, seed=6)
    plan = mg.comet_plan(p, l, c_l, seed=77)
    cap = c_l * (p // l)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(p)
    ctx.load_features(emb, capacity_parts=cap, backing=mg.BACKING_HOST)
    layers = inputs.random_bias_layers([16, 8], seed=2)
    model = ctx.model(layers, mg.GEMM_FP32)
    # every CSR slot is an edge dst <- src; its bucket is (partition of src, partition of dst)
    part_size = (n + p - 1) // p
    dst_all = torch.repeat_interleave(torch.arange(n), g.row_offsets[1:] - g.row_offsets[:-1])
    src_all = g.nbrs.long()
    set_of_edge = torch.as_tensor(plan["bucket_set"])[src_all // part_size, dst_all // part_size]
    trained = torch.zeros(g.n_edges, dtype=torch.int32)
    swaps = 0
    prev = None
    for k, resident in enumerate(plan["physical_sets"]):
        assert len(resident) == cap
        if prev is not None:
            swaps += len(set(resident) - set(prev))
        prev = resident
        ctx.set_resident(resident, async_=True)
        ctx.commit_resident(10_000)
        mine = torch.nonzero(set_of_edge == k).flatten()
        trained[mine] += 1
        if mine.numel() == 0:
            continue
        src, dst, rel = src_all[mine].int(), dst_all[mine].int(), g.edge_rel[mine]
        lp = ctx.lp_prepare(src, rel, dst, 2, 50, seed=900 + k)        # both endpoints resident by construction
        got = lp.view()
        d = ctx.sample(got["targets"], [8], seed=k)
        h = torch.empty((got["targets"].numel(), 8), dtype=torch.float32, device="cuda")
        ctx.forward(model, d, h)
        pos, nd, ns = ctx.distmult_score(lp, h, rel_emb.cuda(), precision=mg.GEMM_FP32)
        if k in (0, len(plan["physical_sets"]) - 1):
            view = oracle_view(g, p, resident)
            prep = O.lp_prepare(view, src.tolist(), dst.tolist(), 2, 50, 900 + k)
            assert got["targets"].cpu().tolist() == prep["targets"]
            ref = O.sample_dense(view, prep["targets"], [8], k)
            assert_dense_equal(d.view(0), ref)
            ref_h = O.forward(ref, emb.numpy()[ref["node_ids"]], [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers])
            close(h.cpu().numpy(), ref_h, RTOL_AGG)
            rpos, rnd, rns = O.distmult_scores(ref_h, rel_emb.numpy(), prep, rel.tolist(), 2)
            close(pos.cpu().numpy(), rpos, RTOL_AGG)
            close(nd.cpu().numpy(), rnd, RTOL_AGG)
            close(ns.cpu().numpy(), rns, RTOL_AGG)
    assert bool((trained == 1).all())                                   # an epoch trains every edge once
    assert swaps == (len(plan["physical_sets"]) - 1) * (p // l)         # one logical partition per step


def _gat_layers(dims, seed):
    g = torch.Generator().manual_seed(seed)
    out = []
    for di, dn in zip(dims[:-1], dims[1:]):
        bound = (6.0 / (di + dn)) ** 0.5
        w = (torch.rand((di, dn), generator=g) * 2 - 1) * bound
        a_s = torch.randn(dn, generator=g) * 0.5
        a_d = torch.randn(dn, generator=g) * 0.5
        b = torch.randn(dn, generator=g) * 0.1
        out.append((w, a_s, a_d, b))
    return out


@pytest.mark.parametrize("dims,fanouts", [([16, 8], [6]), ([16, 32, 12], [5, 3]), ([16, 260, 64, 4], [4, 3, 2])])
def test_graph_attention_forward(tiny, dims, fanouts):
    """The attention layers over DENSE against the oracle: fp32 GEMM and TF32 tensor-core GEMM, several mini-batches
    (one empty, one with a single target), in-only and incoming + outgoing samples."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [120, 0, 1, 300]
    tg = [inputs.distinct_targets(10_000, s, seed=70 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [11, 12, 13, 14]
    layers = _gat_layers(dims, seed=len(dims))
    np_layers = [tuple(t.numpy() for t in l) for l in layers]
    view = oracle_view(g)
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    refs = [O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]) for b in range(len(sizes))]
    wants = [O.gat_forward(r, feats.numpy()[r["node_ids"]], np_layers) if sizes[b] else None for b, r in enumerate(refs)]
    for prec, rtol in ((mg.GEMM_FP32, 2e-5), (mg.GEMM_TF32, RTOL_TC)):
        model = ctx.gat_model(layers, prec)
        out = torch.full((int(offs[-1]), dims[-1]), float("nan"), dtype=torch.float32, device="cuda")
        ctx.gat_forward(model, d, out)
        for b in range(len(sizes)):
            if sizes[b]:
                close(out[offs[b]:offs[b + 1]].cpu().numpy(), wants[b], rtol)
    # uniform attention (a = 0) is the mean over the node and its sampled neighbours of h W
    flat = [(w, torch.zeros_like(a), torch.zeros_like(a), b) for w, a, _, b in layers[:1]]
    if len(dims) == 2:
        model = ctx.gat_model(flat, mg.GEMM_FP32)
        out = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
        ctx.gat_forward(model, d, out)
        r = refs[3]
        h0 = feats.numpy()[r["node_ids"]].astype(np.float64)
        total = O.sage_layer(r, h0, flat[0][0].numpy(), flat[0][0].numpy(), np.zeros(dims[1]), relu=False, aggregator="sum")
        counts = np.diff(r["nbr_offsets"])[:sizes[3], None]
        close(out[offs[3]:offs[4]].cpu().numpy(), total / (counts + 1) + flat[0][3].numpy(), 2e-5)


@pytest.mark.parametrize("dims,heads", [([16, 24, 8], 2), ([16, 32, 32], 8), ([16, 100], 4), ([16, 264, 12], 3)])
def test_graph_attention_with_several_heads(tiny, dims, heads):
    """Multi-head attention: every head attends on its own column block; fp32 and tensor-core paths against the oracle,
    widths whose head blocks do and do not line up with the 32-column slices a lane owns."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [120, 1, 77]
    tg = [inputs.distinct_targets(10_000, s_, seed=50 + i) for i, s_ in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [21, 22, 23]
    fanouts = [5, 3][:len(dims) - 1]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    view = oracle_view(g)
    layers = _gat_layers(dims, seed=heads)
    np_layers = [tuple(t.numpy() for t in l) for l in layers]
    for prec, rtol in ((mg.GEMM_FP32, 5e-5), (mg.GEMM_TF32, RTOL_TC)):
        gm = ctx.gat_model(layers, prec)
        gm.set_heads(heads)
        out = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
        ctx.gat_forward(gm, d, out)
        for b in range(3):
            ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b])
            want = O.gat_forward(ref, feats.numpy()[ref["node_ids"]], np_layers, heads=heads)
            close(out[offs[b]:offs[b + 1]].cpu().numpy(), want, rtol)
    with pytest.raises(mg.MgError) as e:
        gm.set_heads(7)                              # no layer width here is a multiple of 7
    assert e.value.code == -1


def test_graph_attention_errors_and_fp16_features():
    n = 3000
    g = inputs.rmat_graph(n, 30_000, seed=3)
    feats16 = inputs.normal_features(n, 24, seed=2, dtype=torch.float16)
    ctx = make_ctx(g, feats16)
    layers = _gat_layers([24, 8], seed=1)
    targets = inputs.distinct_targets(n, 200, seed=5)
    d = ctx.sample(targets, [7], seed=3)
    ref = O.sample_dense(oracle_view(g), targets.tolist(), [7], 3)
    want = O.gat_forward(ref, feats16.float().numpy()[ref["node_ids"]], [tuple(t.numpy() for t in l) for l in layers])
    model = ctx.gat_model(layers, mg.GEMM_FP32)
    out = torch.empty((200, 8), dtype=torch.float32, device="cuda")
    ctx.gat_forward(model, d, out)
    close(out.cpu().numpy(), want, 2e-5)
    with pytest.raises(mg.MgError) as e:
        ctx.gat_model(_gat_layers([24, 516], seed=1))           # wider than an attention row may be
    assert e.value.code == -1
    with pytest.raises(mg.MgError) as e:
        ctx.gat_forward(ctx.gat_model(_gat_layers([24, 8, 8], seed=1)), d, out)     # two layers, one hop
    assert e.value.code == -2


@pytest.mark.parametrize("aggregator,prec,dims", [("mean", "fp32", [16, 24, 8]), ("sum", "fp32", [16, 24, 8]), ("mean", "tf32", [16, 24, 8]),
                                                  ("mean", "tf32", [16, 64, 32]), ("mean", "tf32", [16, 520, 36]),
                                                  ("sum", "fp32", [16, 300, 260])])
def test_backward_pass_and_sgd_step(tiny, aggregator, prec, dims):
    """Gradients of a scalar loss through the GraphSage layers against the oracle's chain rule (itself pinned by
    finite differences): weights, biases and the base representations' rows; then one SGD step."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    ctx.keep_layer_outputs(True)
    sizes = [150, 0, 1, 260]
    tg = [inputs.distinct_targets(10_000, s, seed=90 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [3, 4, 5, 6]
    fanouts = [5, 3]
    layers = inputs.random_bias_layers(dims, seed=12)
    np_layers = [(w.numpy(), n.numpy(), b.numpy()) for w, n, b in layers]
    precision = mg.GEMM_FP32 if prec == "fp32" else mg.GEMM_TF32
    # fp32: sums over thousands of rows, atomics in any order.  TF32: the tensor-core tolerance, with the oracle
    # differentiating the ReLU branch the GPU's TF32 forward pass took (a pre-activation within rounding of zero may
    # sit on the other side in fp64, which would change single gradient entries by O(1))
    rtol = 2e-4 if prec == "fp32" else RTOL_TC
    model = ctx.model(layers, precision)
    model.set_aggregator(aggregator)
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    out = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    gen = torch.Generator().manual_seed(5)
    g_out = torch.randn((int(offs[-1]), dims[-1]), generator=gen)
    grads, g_h0, ids = ctx.backward(model, d, g_out.cuda(), want_h0_grad=True)
    view = oracle_view(g)
    want = [[np.zeros_like(x, dtype=np.float64) for x in l] for l in np_layers]
    nodes, _ = d.counts()
    row0 = np.concatenate([[0], np.cumsum(nodes.sum(1).cpu().numpy())])
    ids_h, g_h0_h = ids.cpu().numpy(), g_h0.cpu().numpy()
    for b in range(len(sizes)):
        if not sizes[b]:
            continue
        ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b])
        masks = gpu_relu_branch(ctx, model, d, b, ref) if prec == "tf32" else None
        gr, d_h0 = O.backward(ref, feats.numpy()[ref["node_ids"]], np_layers, g_out[offs[b]:offs[b + 1]].numpy(), aggregator,
                              relu_masks=masks)
        for l in range(len(np_layers)):
            for p in range(3):
                want[l][p] += gr[l][p]
        # base-representation gradients: the library's packed rows carry their node ids
        lo, hi = int(row0[b]), int(row0[b + 1])
        assert sorted(ids_h[lo:hi].tolist()) == sorted(ref["node_ids"])
        where = {v: r for r, v in enumerate(ref["node_ids"])}
        close(g_h0_h[lo:hi], d_h0[[where[int(v)] for v in ids_h[lo:hi]]], rtol, per_row=True)
    for l in range(len(np_layers)):
        for p in range(3):
            close(grads[l][p].cpu().numpy(), want[l][p], rtol)
    # one SGD step: the next forward pass uses w - lr dw
    lr = 0.05
    ctx.sgd_step(model, lr)
    stepped = [tuple(torch.from_numpy(x - lr * gw).float() for x, gw in zip(np_layers[l], want[l])) for l in range(len(np_layers))]
    ctx.forward(model, d, out)
    ref3 = O.sample_dense(view, tg[3].tolist(), fanouts, seeds[3])
    want_out = O.forward(ref3, feats.numpy()[ref3["node_ids"]], [tuple(t.numpy() for t in l) for l in stepped], aggregator=aggregator)
    close(out[offs[3]:offs[4]].cpu().numpy(), want_out, 1e-3 if prec == "fp32" else RTOL_TC)   # (a TF32 forward pass again)
    # two Adagrad steps with the same gradients on a fresh copy of the weights
    if prec == "fp32":
        m2 = ctx.model(layers, precision)
        m2.set_aggregator(aggregator)
        ctx.forward(m2, d, out)
        ctx.backward(m2, d, g_out.cuda())
        ctx.adagrad_step(m2, 0.05, 1e-8)
        ctx.adagrad_step(m2, 0.05, 1e-8)
        ada = []
        for l in range(len(np_layers)):
            cur = []
            for x, gw in zip(np_layers[l], want[l]):
                w1, s1 = O.adagrad_step(x, gw, np.zeros_like(gw), 0.05, 1e-8)
                w2, _ = O.adagrad_step(w1, gw, s1, 0.05, 1e-8)
                cur.append(w2)
            ada.append(tuple(cur))
        ctx.forward(m2, d, out)
        close(out[offs[3]:offs[4]].cpu().numpy(), O.forward(ref3, feats.numpy()[ref3["node_ids"]], ada, aggregator=aggregator), 1e-3)
    # state errors
    ctx.keep_layer_outputs(False)
    other = ctx.model(layers, precision)
    with pytest.raises(mg.MgError) as e:
        ctx.backward(other, d, g_out.cuda())
    assert e.value.code == -2


def test_embedding_update_and_write_back_of_evicted_partitions():
    """A training step on the base representations out of core: gradients of H^0 from mg_backward, an SGD step on the
    rows in the partition buffer, and the updated partitions written back to the host table when they are evicted."""
    n, parts, cap = 6000, 6, 3
    g = inputs.rmat_graph(n, 60_000, seed=9)
    table = inputs.normal_features(n, 8, seed=3, pin=False).pin_memory()
    before = table.clone()
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(parts)
    ctx.load_features(table, capacity_parts=cap, backing=mg.BACKING_HOST)
    ctx.keep_layer_outputs(True)
    resident = [0, 2, 5]
    ctx.set_resident(resident, async_=True)
    ctx.commit_resident(10_000)
    layers = inputs.random_bias_layers([8, 8, 4], seed=1)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    model = ctx.model(layers, mg.GEMM_FP32)
    pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident)).flatten()
    sizes = [60, 80]
    tg = [inputs.distinct_targets(pool, s, seed=7 + i) for i, s in enumerate(sizes)]
    offs = [0, 60, 140]
    seeds = [1, 2]
    d = ctx.sample_many(torch.cat(tg), offs, [4, 3], seeds)
    out = torch.empty((140, 4), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    g_out = torch.randn((140, 4), generator=torch.Generator().manual_seed(3))
    _, g_h0, ids = ctx.backward(model, d, g_out.cuda(), want_h0_grad=True)
    lr = 0.1
    ctx.apply_embedding_sgd(d, g_h0, lr)
    # what the table must look like now: the oracle's gradient rows, summed per node over the two mini-batches
    view = oracle_view(g, parts, resident)
    want = before.numpy().astype(np.float64).copy()
    for b in range(2):
        ref = O.sample_dense(view, tg[b].tolist(), [4, 3], seeds[b])
        _, d_h0 = O.backward(ref, before.numpy()[ref["node_ids"]], np_layers, g_out[offs[b]:offs[b + 1]].numpy())
        np.subtract.at(want, np.asarray(ref["node_ids"]), lr * d_h0)
    # the buffer holds the update (read back through a fresh sample's H^0 rows); the host table does not yet
    probe = inputs.distinct_targets(pool, 300, seed=99)
    dp = ctx.sample(probe, [2], seed=5)
    refp = O.sample_dense(view, probe.tolist(), [2], 5)
    close(ctx.gather_h0(dp, 0, len(refp["node_ids"]), 8).cpu().numpy(), want[refp["node_ids"]], 2e-5)
    assert torch.equal(table, before)
    # evict everything that was updated: the rows go back to the host table before their slots are reused
    ctx.set_resident([1, 3, 4], async_=True)
    ctx.commit_resident(10_000)
    torch.cuda.synchronize()
    close(table.numpy(), want, 2e-5)
    changed = np.nonzero(np.abs(want - before.numpy()).sum(1))[0]
    assert len(changed) > 100 and all(int(v) // ((n + parts - 1) // parts) in resident for v in changed)
    # and come back from there when the partitions are loaded again
    ctx.set_resident(resident, async_=True)
    ctx.commit_resident(10_000)
    dp = ctx.sample(probe, [2], seed=5)
    close(ctx.gather_h0(dp, 0, len(refp["node_ids"]), 8).cpu().numpy(), want[refp["node_ids"]], 2e-5)


@pytest.mark.parametrize("case", range(24))
def test_randomised_small_configurations(case):
    """Seeded random shapes through the whole path against the oracle: graph size and kind, number and sizes of
    mini-batches (empty ones included), depth, fanouts, sampling direction, capacities (default, tight, large: the
    three deduplication paths), partitions with a partial resident set, aggregator, precision."""
    rng = np.random.default_rng(1000 + case)
    n = int(rng.integers(40, 2500))
    m = int(rng.integers(n, 12 * n))
    g = inputs.rmat_graph(n, m, seed=case) if case % 2 else inputs.erdos_renyi_graph(n, m, seed=case)
    dim = int(rng.choice([4, 8, 20, 36]))
    feats = inputs.normal_features(n, dim, seed=case + 1)
    parts = int(rng.choice([1, 1, 3, 5]))
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.to(torch.int32 if case % 3 == 0 else torch.int64).cuda(), g.nbrs.cuda())
    inout = bool(rng.integers(0, 2))
    gt = inputs.transpose_csr(g) if inout else None
    if inout:
        ctx.load_out_graph(gt.row_offsets.cuda(), gt.nbrs.cuda())
        ctx.set_sample_direction("inout")
    resident = None
    if parts > 1:
        ctx.set_partitioning(parts)
        ctx.load_features(feats.cuda(), capacity_parts=parts)
        resident = sorted(rng.choice(parts, size=int(rng.integers(1, parts + 1)), replace=False).tolist())
        ctx.set_resident(resident)
    else:
        ctx.load_features(feats.cuda())
    view = O.GraphView(g.row_offsets.numpy(), g.nbrs.numpy(), parts, resident,
                       gt.row_offsets.numpy() if inout else None, gt.nbrs.numpy() if inout else None)
    pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident if resident is not None else [0])).flatten()
    k = int(rng.integers(1, 5))
    fanouts = [int(rng.integers(1, 9)) if rng.random() < 0.8 else int(rng.integers(9, 41)) for _ in range(k)]
    B = int(rng.integers(1, 6))
    sizes = [int(rng.integers(0, min(40, pool.numel()) + 1)) for _ in range(B)]
    tg = [inputs.distinct_targets(pool, s, seed=50 * case + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    seeds = [int(rng.integers(0, 2**62)) for _ in range(B)]
    direction = "inout" if inout else "in"
    refs = [O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b], direction) for b in range(B)]
    most = max(len(r["node_ids"]) for r in refs)
    caps = [None, {"max_nodes_per_batch": most}, {"max_nodes_per_batch": 40_000}, {"max_nodes_per_batch": 1_200_000}][case % 4]
    all_targets = torch.cat(tg) if B else torch.empty(0, dtype=torch.int32)
    d = ctx.sample_many(all_targets.to(torch.int32), offs, fanouts, seeds, caps=caps)
    for b in range(B):
        assert_dense_equal(d.view(b), refs[b])
    dims = [dim] + [int(rng.choice([4, 8, 12, 32])) for _ in range(k)]
    layers = inputs.random_bias_layers(dims, seed=case + 3)
    np_layers = [(w.numpy(), nn.numpy(), bb.numpy()) for w, nn, bb in layers]
    aggregator = "sum" if case % 5 == 0 else "mean"
    prec, rtol = ((mg.GEMM_TF32, RTOL_TC) if case % 2 else (mg.GEMM_FP32, RTOL_AGG))
    if aggregator == "sum":
        rtol *= 4                       # sums of up to 2 x 40 rows per node and layer instead of means
    model = ctx.model(layers, prec)
    model.set_aggregator(aggregator)
    out = torch.full((int(offs[-1]), dims[-1]), float("nan"), dtype=torch.float32, device="cuda")
    if int(offs[-1]):
        ctx.forward(model, d, out)
    for b in range(B):
        if sizes[b]:
            want = O.forward(refs[b], feats.numpy()[refs[b]["node_ids"]], np_layers, aggregator=aggregator)
            close(out[offs[b]:offs[b + 1]].cpu().numpy(), want, rtol)


@pytest.mark.parametrize("case", range(10))
def test_randomised_backward_and_attention(case):
    """Seeded random shapes for the two widened model paths: gradients (fp32) and the attention layers (fp32)."""
    rng = np.random.default_rng(5000 + case)
    n = int(rng.integers(60, 1500))
    g = inputs.rmat_graph(n, int(rng.integers(2 * n, 10 * n)), seed=case)
    dim = int(rng.choice([4, 8, 16]))
    feats = inputs.normal_features(n, dim, seed=case + 1)
    ctx = make_ctx(g, feats)
    ctx.keep_layer_outputs(True)
    view = oracle_view(g)
    k = int(rng.integers(1, 4))
    fanouts = [int(rng.integers(1, 7)) for _ in range(k)]
    B = int(rng.integers(1, 4))
    sizes = [int(rng.integers(1, 30)) for _ in range(B)]
    tg = [inputs.distinct_targets(n, s, seed=70 * case + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    seeds = [int(rng.integers(0, 2**40)) for _ in range(B)]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    refs = [O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b]) for b in range(B)]
    dims = [dim] + [int(rng.choice([4, 8, 20])) for _ in range(k)]
    # gradients
    layers = inputs.random_bias_layers(dims, seed=case)
    np_layers = [(w.numpy(), nn.numpy(), bb.numpy()) for w, nn, bb in layers]
    aggregator = "sum" if case % 3 == 0 else "mean"
    model = ctx.model(layers, mg.GEMM_FP32)
    model.set_aggregator(aggregator)
    out = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
    ctx.forward(model, d, out)
    g_out = torch.randn((int(offs[-1]), dims[-1]), generator=torch.Generator().manual_seed(case))
    grads, g_h0, ids = ctx.backward(model, d, g_out.cuda(), want_h0_grad=True)
    want = [[np.zeros_like(x, dtype=np.float64) for x in l] for l in np_layers]
    nodes, _ = d.counts()
    row0 = np.concatenate([[0], np.cumsum(nodes.sum(1).cpu().numpy())])
    for b in range(B):
        gr, d_h0 = O.backward(refs[b], feats.numpy()[refs[b]["node_ids"]], np_layers, g_out[offs[b]:offs[b + 1]].numpy(), aggregator)
        for l in range(k):
            for p in range(3):
                want[l][p] += gr[l][p]
        lo, hi = int(row0[b]), int(row0[b + 1])
        where = {v: r for r, v in enumerate(refs[b]["node_ids"])}
        close(g_h0[lo:hi].cpu().numpy(), d_h0[[where[int(v)] for v in ids[lo:hi].cpu().numpy()]], 5e-4)
    for l in range(k):
        for p in range(3):
            close(grads[l][p].cpu().numpy(), want[l][p], 5e-4)
    # attention layers
    gat_layers = _gat_layers(dims, seed=case + 9)
    slope = float(rng.choice([0.0, 0.2, 0.5]))
    gm = ctx.gat_model(gat_layers, mg.GEMM_FP32, negative_slope=slope)
    ctx.gat_forward(gm, d, out)
    for b in range(B):
        want_out = O.gat_forward(refs[b], feats.numpy()[refs[b]["node_ids"]], [tuple(t.numpy() for t in l) for l in gat_layers], slope=slope)
        close(out[offs[b]:offs[b + 1]].cpu().numpy(), want_out, 5e-5)


@pytest.mark.parametrize("fanouts", [[22], [21, 3], [23, 2], [16, 2], [40, 2]])
def test_fused_layer_rows_around_the_entry_cache(tiny, fanouts):
    """Rows whose 32-row blocks hold about as many entries as the fused kernel caches in shared memory (22 per row on
    average): the graph's degrees spread around 20, so blocks fall on both sides of the limit, and a fanout of 40 puts
    every block past it.  Both aggregators, two mini-batches with a ragged last block."""
    g, feats = tiny
    ctx = make_ctx(g, feats)
    sizes = [301, 77]
    tg = [inputs.distinct_targets(10_000, s, seed=40 + i) for i, s in enumerate(sizes)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    seeds = [321, 322]
    d = ctx.sample_many(torch.cat(tg), offs, fanouts, seeds)
    dims = [16] + [32] * (len(fanouts) - 1) + [24]
    layers = inputs.random_bias_layers(dims, seed=12)
    model = ctx.model(layers, mg.GEMM_TF32)
    out = torch.empty((int(offs[-1]), dims[-1]), dtype=torch.float32, device="cuda")
    view = oracle_view(g)
    np_layers = [(w.numpy(), n.numpy(), b.numpy()) for w, n, b in layers]
    for aggregator in ("mean", "sum"):
        model.set_aggregator(aggregator)
        out.fill_(float("nan"))
        ctx.forward(model, d, out)
        for b in range(2):
            ref = O.sample_dense(view, tg[b].tolist(), fanouts, seeds[b])
            assert_dense_equal(d.view(b), ref)
            want = O.forward(ref, feats.numpy()[ref["node_ids"]], np_layers, aggregator=aggregator)
            close(out[offs[b]:offs[b + 1]].cpu().numpy(), want, RTOL_TC)
