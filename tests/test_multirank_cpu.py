"""World-size-2 checks (gloo, CPU) of the host logic that runs on several GPUs:
  * bench.py: every rank draws its own shard, times are reduced with MAX and token counts with SUM;
  * the data-parallel step: the reduction logic of DataParallelStep (M all-reduced first, per-rank weights
    M_r / M, grad_w and the weighted loss summed) with the fp64 oracle standing in for the GPU kernels gives
    the loss and the gradients of the oracle on the concatenated batch."""
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


# ------------------------------------------------------------------------------------ data-parallel step
def _dp_problem():
    """One batch of 6 sequences, split 4 / 2 over two ranks (unequal M_r on purpose)."""
    sys.path.insert(0, ROOT)
    from paper_2512_06547_b200 import workloads
    wl = workloads.make_workload("tiny", "cpu", n_prompts=3, group=2, row_len=40, len_lo=7, len_hi=40)
    cut = int(wl.cu_seqlens[4])
    return wl, cut


def _oracle_step(wl, rows, scale):
    """What a3po_train_step computes on the rows `rows`, in the oracle, with the upstream gradient times `scale`."""
    from oracle import a3po_oracle as orc
    from paper_2512_06547_b200 import workloads
    hn, wn = wl.hidden[rows].double().numpy(), wl.w.double().numpy()
    logp, _ = orc.token_logprobs_fwd(hn, wn, wl.targets[rows], row_mask=wl.mask[rows])
    behav = workloads.behav_logp_from(np.where(wl.mask[rows] != 0, logp, -1.0), wl.behav_noise[rows])
    args = (logp, behav, wl.versions[rows], wl.current_version, wl.adv[rows], wl.mask[rows], wl.clip_eps)
    loss, _ = orc.loss_fwd(*args)
    g = orc.loss_bwd(*args, grad_loss=scale)
    gh, gw = orc.token_logprobs_bwd(hn, wn, wl.targets[rows], g)
    return loss, g, gh, gw


def _dp_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from paper_2512_06547_b200.data_parallel import DataParallelStep
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl, cut = _dp_problem()
    rows = slice(0, cut) if rank == 0 else slice(cut, wl.N)

    def count_fn(mask):
        return torch.tensor([int(np.count_nonzero(mask))], dtype=torch.int64)

    def scale_fn(m_local, m_global, loss_local):
        scale = (m_local.double() / m_global.double().clamp_min(1)).float()
        return scale, (None if loss_local is None else (scale.double() * loss_local.double()))

    def step_fn(batch, scale):
        loss, g, gh, gw = _oracle_step(wl, rows, float(scale.item()))
        return {"loss": torch.tensor([loss], dtype=torch.float64), "grad_w": torch.from_numpy(gw),
                "grad_hidden": torch.from_numpy(gh), "grad_logp": torch.from_numpy(g)}

    out = DataParallelStep(count_fn, scale_fn, step_fn)({"mask": wl.mask[rows]})
    np.savez(os.path.join(out_dir, f"dp{rank}.npz"), loss=out["loss"].numpy(), grad_w=out["grad_w"].numpy(),
             grad_hidden=out["grad_hidden"].numpy(), grad_logp=out["grad_logp"].numpy(),
             m=np.array([int(out["m_local"]), int(out["m_global"])]))
    dist.barrier()
    dist.destroy_process_group()


def test_data_parallel_step_equals_whole_batch(tmp_path):
    world = 2
    mp.spawn(_dp_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl, cut = _dp_problem()
    r = [np.load(tmp_path / f"dp{k}.npz") for k in range(world)]
    loss, g, gh, gw = _oracle_step(wl, slice(0, wl.N), 1.0)          # the whole batch on one rank
    m0, m1 = int(wl.mask[:cut].sum()), int(wl.mask[cut:].sum())
    assert m0 != m1 and list(r[0]["m"]) == [m0, m0 + m1] and list(r[1]["m"]) == [m1, m0 + m1]
    for k in range(world):                                            # both ranks hold the whole-job loss and grad_w
        assert abs(float(r[k]["loss"][0]) - loss) <= 1e-6 * max(abs(loss), 1e-3)   # the weight crosses as fp32
        np.testing.assert_allclose(r[k]["grad_w"], gw, rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(np.concatenate([r[0]["grad_logp"], r[1]["grad_logp"]]), g, rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([r[0]["grad_hidden"], r[1]["grad_hidden"]]), gh, rtol=1e-6, atol=1e-9)
