"""mg_forward_noalloc: the forward pass for callers that may not allocate device memory while
they run (all device memory handed out at start-up, or an allocator-owning host framework, or a
loop that cannot take the synchronisation an allocation implies).  It must give what mg_forward
gives, call after call, although every call reuses the same built-in scratch array and finds the
previous call's values in it.  Collected last on purpose: a run that stops at the first failure
has then already run every other test."""
import numpy as np
import pytest
import torch

import paper_2202_02365_b200 as mg
from oracle import dense_oracle as O
from paper_2202_02365_b200 import inputs

pytestmark = pytest.mark.gpu

# The tolerances of the parity tests.  With MG_GEMM_FP32 both entry points run the same kernels (k_aggregate, then the
# fp32 GEMM), so 1e-5 holds between them as it does against the oracle.  With MG_GEMM_TF32 they do not: mg_forward runs
# the fused gather + tensor-core kernel, mg_forward_noalloc the separate aggregation kernel and the tensor-core GEMM;
# both round the same operands to TF32 but add the products up in a different order.
RTOL = {mg.GEMM_FP32: 1e-5, mg.GEMM_TF32: 5e-3}


def _close(got, ref, rtol):
    got = got.double().cpu().numpy() if torch.is_tensor(got) else np.asarray(got, dtype=np.float64)
    ref = ref.double().cpu().numpy() if torch.is_tensor(ref) else np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref ** 2))
    assert np.all(np.abs(got - ref) <= rtol * np.maximum(np.abs(ref), rms))


def _oracle_rows(g_host, feats_host, np_layers, targets, fanouts, seed, n_parts=1, resident=None):
    view = O.GraphView(g_host[0], g_host[1], n_parts, resident)
    ref = O.sample_dense(view, targets.tolist(), fanouts, seed)
    h0 = feats_host[torch.as_tensor(ref["node_ids"])].float().numpy()
    return O.forward(ref, h0, np_layers)


def test_noalloc_forward_matches_forward_twice_in_a_row():
    n = 20_000
    g = inputs.rmat_graph(n, 300_000, seed=31)
    feats = inputs.normal_features(n, 32, seed=32)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.load_features(feats.cuda())
    layers = inputs.random_bias_layers([32, 64, 16], seed=33)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    g_host = (g.row_offsets.numpy(), g.nbrs.numpy())
    for precision in (mg.GEMM_TF32, mg.GEMM_FP32):
        model = ctx.model(layers, precision)
        # two calls in a row on different samples: the second finds the first one's values in the scratch
        for call, (n_targets, seed) in enumerate([(700, 5), (333, 6)]):
            targets = inputs.distinct_targets(n, n_targets, seed=40 + call)
            d = ctx.sample_many(torch.cat([targets, targets[:50]]), [0, n_targets, n_targets + 50], [8, 4], [seed, seed + 100])
            want = torch.empty((n_targets + 50, 16), dtype=torch.float32, device="cuda")
            ctx.forward(model, d, want)
            got = torch.full_like(want, float("nan"))
            ctx.forward_noalloc(model, d, got)
            assert torch.isfinite(got).all()
            _close(got, want, RTOL[precision])
            # and on its own against the CPU oracle: the first mini-batch's rows
            _close(got[:n_targets], _oracle_rows(g_host, feats, np_layers, targets, [8, 4], seed), RTOL[precision])


def test_noalloc_forward_under_the_partition_buffer_with_fp16_rows():
    """The same with half-precision rows that live in host memory and reach the GPU through the partition buffer's
    slots (5 partitions, 3 resident, not in slot order): the aggregation kernel then widens fp16 rows and addresses
    them through the partition -> slot map."""
    n, parts, resident = 30_000, 5, [4, 1, 2]
    g = inputs.rmat_graph(n, 400_000, seed=51)
    feats = inputs.normal_features(n, 64, seed=52).half().pin_memory()
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.set_partitioning(parts)
    ctx.load_features(feats, capacity_parts=3, backing=mg.BACKING_HOST)
    ctx.set_resident(resident)
    layers = inputs.random_bias_layers([64, 32, 8], seed=53)
    np_layers = [(w.numpy(), nn.numpy(), b.numpy()) for w, nn, b in layers]
    g_host = (g.row_offsets.numpy(), g.nbrs.numpy())
    pool = torch.nonzero(inputs.resident_node_mask(n, parts, resident)).flatten()
    for precision in (mg.GEMM_FP32, mg.GEMM_TF32):
        model = ctx.model(layers, precision)
        for call, n_targets in enumerate([400, 90]):
            targets = inputs.distinct_targets(pool, n_targets, seed=60 + call)
            d = ctx.sample(targets, [6, 3], seed=9 + call)
            want = torch.empty((n_targets, 8), dtype=torch.float32, device="cuda")
            ctx.forward(model, d, want)
            got = torch.full_like(want, float("nan"))
            ctx.forward_noalloc(model, d, got)
            _close(got, want, RTOL[precision])
            _close(got, _oracle_rows(g_host, feats, np_layers, targets, [6, 3], 9 + call, parts, resident), RTOL[precision])


def test_noalloc_forward_rejects_what_does_not_fit():
    n = 50_000
    g = inputs.rmat_graph(n, 1_000_000, seed=34)
    feats = inputs.normal_features(n, 16, seed=35)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.load_features(feats.cuda())
    model = ctx.model(inputs.glorot_layers([16, 1024, 16], seed=36), mg.GEMM_FP32)
    targets = inputs.distinct_targets(n, 4000, seed=37)
    d = ctx.sample(targets, [10, 10], seed=1)
    nodes, _ = d.counts()
    assert int(nodes[0, :2].sum()) * 1024 * 4 > 12 << 20          # H^1 alone exceeds the 12 MiB limit
    out = torch.empty((4000, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(mg.MgError) as e:
        ctx.forward_noalloc(model, d, out)
    assert e.value.code == -5 and "scratch" in str(e.value)
    ctx.forward(model, d, out)                                      # the allocating entry point still serves it
