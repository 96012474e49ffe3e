"""gto_build_tree_noalloc against gto_build_tree.

The no-allocation call exists for hosts that cannot let a library call cudaMalloc (a trainer
whose allocator must own every device byte, a fixed memory budget, a thread that cannot take
the stall of an allocation).  It keeps its scratch in a fixed device array inside the library,
shared by all calls, so this file checks the two things that could go wrong with that: the
results must equal the context-based call's, and a second call must not see anything stale
from the first.  Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import pytest
import torch

from paper_2509_22134_b200 import synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
INT_FIELDS = ("node_token", "node_parent", "node_depth", "node_ctx_row", "node_slot", "node_pool",
              "node_mask")
FLOAT_FIELDS = ("node_logp", "node_score", "row_lse")


def _trees_equal(a, b):
    for name in INT_FIELDS:
        assert torch.equal(a[name], b[name]), name
    for name in FLOAT_FIELDS:      # same kernels, same inputs: well inside the parity tolerance
        assert torch.allclose(a[name].double(), b[name].double(), rtol=0, atol=1e-6), name


def _matches_the_oracle(w, data, tree, positions):
    """The no-allocation call's own output against the oracle's tree, node by node."""
    import numpy as np
    from oracle import gto_oracle as orc
    for b in positions:
        for t in range(w.G):
            want = orc.build_tree(data["draft"][t, b].float().cpu().numpy().astype(np.float64), w.D, w.k, w.g)
            for name, attr in (("node_token", "token"), ("node_parent", "parent"), ("node_depth", "depth"),
                               ("node_ctx_row", "ctx_row"), ("node_slot", "slot"), ("node_pool", "pool")):
                assert np.array_equal(tree[name][t, b].cpu().numpy(), getattr(want, attr)), (name, t, b)
            assert np.max(np.abs(tree["node_score"][t, b].cpu().numpy() - want.score)) <= 1e-5
            assert np.max(np.abs(tree["row_lse"][t, b].cpu().numpy() - want.row_lse)) <= 2e-6


def test_two_calls_in_a_row_match_the_context_call():
    from paper_2509_22134_b200 import binding as gto
    # two different shapes back to back, the larger first, so stale scratch would show
    shapes = [dict(B=64, V_draft=4104, V_target=4104, D=4, k=5, g=30, dtype="bf16", seed=11),
              dict(B=16, V_draft=1000, V_target=1000, D=3, k=4, g=12, dtype="f32", seed=12)]
    torch.cuda.set_device(0)
    for kw in shapes:
        w = synth.Workload("noalloc", **kw)
        data = synth.generate(w, DEV)
        cfg = gto.make_config(w.B, w.D, w.k, w.g, w.m, w.V_draft, w.V_target, w.dtype)
        ctx = gto.gto_create(cfg, 0)
        want = gto.alloc_tree(cfg, DEV)
        got = gto.alloc_tree(cfg, DEV)
        for t in got.values():
            t.view(torch.uint8).fill_(0xA5)          # poison: every element must be written
        gto.gto_build_tree(ctx, data["draft"], want)
        gto.gto_build_tree_noalloc(cfg, 0, data["draft"], got)
        torch.cuda.synchronize()
        _trees_equal(got, want)
        gto.gto_destroy(ctx)
        _matches_the_oracle(w, data, got, positions=(0, w.B - 1))


def test_a_batch_beyond_the_fixed_scratch_is_refused():
    from paper_2509_22134_b200 import binding as gto
    w = synth.WORKLOADS[2]                            # 124 928 rows x 10 > 2^20 entries
    assert w.G * w.B * w.R * w.k > gto.GTO_NOALLOC_MAX_ENTRIES
    cfg = gto.make_config(w.B, w.D, w.k, w.g, w.m, w.V_draft, w.V_target, w.dtype)
    tree = gto.alloc_tree(cfg, DEV)
    draft = torch.empty(16, dtype=torch.bfloat16, device=DEV)   # never read: refused first
    with pytest.raises(gto.GtoError) as e:
        gto.gto_build_tree_noalloc(cfg, 0, draft, tree)
    assert e.value.code == 7
