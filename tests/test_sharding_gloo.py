"""The N > 1 path on CPU (gloo): positions shard over ranks in whole groups with no
data-path collective.  Checked here: (a) shard_positions covers the batch exactly once, in
whole groups, also when the groups do not divide by the world size; (b) a rank's shard of
the synthetic batch is bit-identical to the same positions of the full batch (the generators
are keyed by absolute position); (c) the oracle's pass over one rank's groups needs nothing
from another rank: the group results gathered from all ranks equal a single-process pass over
the full batch; (d) the benchmark's max-over-ranks reduction returns the slowest rank's time
on every rank.  The hardware path itself is not shown on more than one GPU by this file."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GROUPS = 4          # groups in the global batch: not a multiple of 3


def _old_fn_at(w, first):
    from paper_2509_22134_b200 import synth

    def f(path_logp, path_row, path_token, path_len):
        out = np.zeros_like(path_logp)
        for i in range(path_logp.shape[0]):
            out[i] = synth.old_logp_from_path(w, path_logp[i:i + 1], path_row[i:i + 1],
                                              path_token[i:i + 1], path_len[i:i + 1], b0=first + i)[0]
        return out
    return f


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import gto_oracle as orc
    from paper_2509_22134_b200 import synth
    from paper_2509_22134_b200.sharding import shard_positions
    w0 = synth.WORKLOADS[0]                       # m = 8
    B = GROUPS * w0.m
    first, count = shard_positions(B, w0.m, world)[rank]
    assert count % w0.m == 0
    full = synth.generate(w0.with_B(B), "cpu")
    mine = []
    if count:
        w = w0.with_B(count)
        data = synth.generate(w, "cpu", b0=first)
        sl = slice(first, first + count)
        assert torch.equal(data["draft"][:, :, 0, 0], full["draft"][:, sl, 0, 0])
        assert torch.equal(data["draft"][:, :, 1:], full["draft"][:, sl, 1:])
        assert torch.equal(data["target"], full["target"][:, sl])
        for g0 in range(0, count, w.m):            # this rank's groups, from its own shard only
            out = orc.group_pass(data["draft"][:, g0:g0 + w.m].numpy(), data["target"][:, g0:g0 + w.m].numpy(),
                                 w.D, w.k, w.g, w.m, _old_fn_at(w, first + g0))
            mine.append((first + g0, out["A"], out["sur"]["loss"], out["grad"]))
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)         # test plumbing only: the pass itself sent nothing
    if rank == 0:
        seen = sorted(x for part in gathered for x in part)
        assert [x[0] for x in seen] == [g * w0.m for g in range(GROUPS)]
        for b0, A, loss, grad in seen:             # one process over the full batch agrees
            ref = orc.group_pass(full["draft"][:, b0:b0 + w0.m].numpy(), full["target"][:, b0:b0 + w0.m].numpy(),
                                 w0.D, w0.k, w0.g, w0.m, _old_fn_at(w0, b0))
            assert np.array_equal(A, ref["A"]) and np.array_equal(loss, ref["sur"]["loss"])
            assert np.array_equal(grad, ref["grad"])
        assert len({float(x[1].sum() + x[3].sum()) for x in seen}) == GROUPS   # different positions
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], world, "cpu")
    assert got == [10.0 + world - 1, 5.0], got
    assert bench.shard_first_position(rank, w0.B) == shard_positions(world * w0.B, w0.m, world)[rank][0]
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(out_dir, f"ok{rank}"), "w").close()


@pytest.mark.parametrize("world", [2, 3])
def test_ranks_shard_whole_groups_without_a_collective(tmp_path, world):
    port = 29500 + (os.getpid() * 7 + world) % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))


def test_shard_positions_covers_the_batch_once_in_whole_groups():
    from paper_2509_22134_b200.sharding import shard_positions
    for B, m, world in [(1024, 8, 8), (32, 8, 3), (8, 8, 4), (0, 4, 2), (40, 1, 7), (2048, 8, 5)]:
        parts = shard_positions(B, m, world)
        assert len(parts) == world
        assert parts[0][0] == 0 and sum(n for _, n in parts) == B
        for (a, n), (b, _) in zip(parts, parts[1:]):
            assert a + n == b
        assert all(a % m == 0 and n % m == 0 for a, n in parts)          # no group straddles ranks
        sizes = [n // m for _, n in parts]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    for bad in [(10, 4, 2), (8, 0, 1), (8, 8, 0)]:
        with pytest.raises(ValueError):
            shard_positions(*bad)
