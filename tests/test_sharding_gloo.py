"""The N > 1 path on CPU (gloo, world size 2): positions shard over ranks in whole groups
with no data-path collective, so (a) a rank's shard of the synthetic batch is bit-identical
to the same positions of the full batch, (b) the oracle's pass over a shard equals its pass
over those positions of the full batch (groups never straddle ranks), and (c) the benchmark's
max-over-ranks reduction returns the slowest rank's time on every rank."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import gto_oracle as orc
    from paper_2509_22134_b200 import synth
    w = synth.WORKLOADS[0]                       # B = 8 per rank, one group each
    b0 = bench.shard_first_position(rank, w.B)
    data = synth.generate(w, "cpu", b0=b0)
    full = synth.generate(w.with_B(w.B * world), "cpu")
    sl = slice(b0, b0 + w.B)
    assert torch.equal(data["draft"][:, :, 0, 0], full["draft"][:, sl, 0, 0])
    assert torch.equal(data["draft"][:, :, 1:], full["draft"][:, sl, 1:])
    assert torch.equal(data["target"], full["target"][:, sl])

    def old_fn_at(first):
        def f(path_logp, path_row, path_token, path_len):
            out = np.zeros_like(path_logp)
            for i in range(path_logp.shape[0]):
                out[i] = synth.old_logp_from_path(w, path_logp[i:i + 1], path_row[i:i + 1],
                                                  path_token[i:i + 1], path_len[i:i + 1], b0=first + i)[0]
            return out
        return f
    mine = orc.group_pass(data["draft"].numpy(), data["target"].numpy(), w.D, w.k, w.g, w.m, old_fn_at(b0))
    ref = orc.group_pass(full["draft"][:, sl].numpy(), full["target"][:, sl].numpy(), w.D, w.k, w.g, w.m,
                         old_fn_at(b0))
    assert np.array_equal(mine["A"], ref["A"]) and np.array_equal(mine["grad"], ref["grad"])
    # the two ranks really hold different positions
    gathered = [None] * world
    dist.all_gather_object(gathered, float(mine["R"].sum()))
    assert gathered[0] != gathered[1]

    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], world, "cpu")
    assert got == [10.0 + world - 1, 5.0], got
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(out_dir, f"ok{rank}"), "w").close()


def test_two_ranks_shard_positions_without_a_collective(tmp_path):
    world = 2
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))
