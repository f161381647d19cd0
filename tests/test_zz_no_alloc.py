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
from paper_2202_02365_b200 import inputs

pytestmark = pytest.mark.gpu

RTOL = 1e-5   # the tolerance of the fp32 parity tests; both entry points run the same kernels


def _close(got, ref, rtol):
    got, ref = got.double().cpu().numpy(), ref.double().cpu().numpy()
    rms = np.sqrt(np.mean(ref ** 2))
    assert np.all(np.abs(got - ref) <= rtol * np.maximum(np.abs(ref), rms))


def test_noalloc_forward_matches_forward_twice_in_a_row():
    n = 20_000
    g = inputs.rmat_graph(n, 300_000, seed=31)
    feats = inputs.normal_features(n, 32, seed=32)
    ctx = mg.Context(0)
    ctx.load_graph(g.row_offsets.cuda(), g.nbrs.cuda())
    ctx.load_features(feats.cuda())
    layers = inputs.random_bias_layers([32, 64, 16], seed=33)
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
            _close(got, want, RTOL)


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
