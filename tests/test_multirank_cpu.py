"""World-size-2 check (gloo, CPU) of the host logic bench.py uses when it runs on several GPUs:
every rank draws its own shard, times are reduced with MAX and token counts with SUM."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2512_06547_b200 import workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.make_workload("1p5b", "cpu", with_operands=False, seed=bench.rank_seed("1p5b", rank))
    n_valid = int(wl.mask.sum())
    (t_step, t_e2e), (valid, rows) = bench.reduce_over_ranks([10.0 + rank, 30.0 - rank], [n_valid, wl.N], "cpu")
    np.save(os.path.join(out_dir, f"rank{rank}.npy"),
            np.array([t_step, t_e2e, valid, rows, n_valid, wl.valid_len.sum(), wl.targets[:64].sum()], dtype=np.float64))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"rank{r}.npy") for r in range(world))
    # every rank sees the same whole-job figures
    assert np.array_equal(r0[:4], r1[:4])
    assert r0[0] == 11.0 and r0[1] == 30.0                      # MAX over ranks
    assert r0[2] == r0[4] + r1[4] and r0[3] == 2 * 16384        # SUM over ranks
    # the shards differ (different draws), with the same shapes
    assert r0[5] != r1[5] and r0[6] != r1[6]


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert not dist.is_initialized()
    (t,), (c,) = bench.reduce_over_ranks([3.5], [7], "cpu")
    assert t == 3.5 and c == 7.0
