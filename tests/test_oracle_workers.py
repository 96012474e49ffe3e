"""The worker pool that runs the oracle on every host core: results come back in order, a
failure in a worker surfaces in the parent, logits survive the trip bit for bit."""
import numpy as np
import pytest
import torch

from oracle import parallel as opar


def test_logits_round_trip_exactly():
    g = torch.Generator().manual_seed(0)
    x = torch.randn(3, 257, generator=g) * 7
    for dt in (torch.bfloat16, torch.float16, torch.float32):
        raw, tag = opar.encode_logits(x.to(dt))
        assert np.array_equal(opar.decode_logits(raw, tag), x.to(dt).float().numpy())


def test_pool_runs_oracle_functions_in_order_and_reports_failures():
    from oracle import gto_oracle as orc
    rows = [np.random.default_rng(i).normal(size=50) for i in range(5)]
    with opar.OracleWorkers(2) as pool:
        out, wall = pool.run("oracle.gto_oracle", "lse_and_topk", [dict(z=r) for r in rows], common=dict(k=3))
        for r, (lse, ids, lp) in zip(rows, out):
            want = orc.lse_and_topk(r, 3)
            assert lse == want[0] and np.array_equal(ids, want[1])
        assert wall > 0
        with pytest.raises(AssertionError, match="oracle worker"):
            pool.run("oracle.gto_oracle", "build_tree", [dict(draft=np.zeros((2, 2, 4)), D=2, k=2, g=99)])
        out, _ = pool.run("oracle.gto_oracle", "argmax_low", [dict(z=[1, 3, 3])])    # still usable
        assert out == [1]
