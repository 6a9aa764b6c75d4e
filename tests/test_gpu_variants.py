"""GPU parity of the widened rows: explicit-anchor decoupled loss ("recompute" / coupled baselines), GRPO
advantages, and the bounded-wait self-test."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from oracle import a3po_oracle as orc
from paper_2512_06547_b200 import workloads
from tests.helpers import BOUNDARY_REL, LOSS_RTOL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("n,anchor", [(0, "noisy"), (5, "noisy"), (100_003, "noisy"), (1 << 20, "noisy"),
                                      (50_000, "behaviour")])
def test_decoupled_loss_matches_oracle(n, anchor):
    inp = workloads.loss_sweep(n, seed=300 + n % 97, correlated=True)
    rng = np.random.default_rng(n + 1)
    if anchor == "behaviour":
        prox = inp["behav_logp"].copy()                      # Eq. 1: coupled PPO-clip
    else:
        prox = np.minimum(inp["logp"] + 0.1 * rng.standard_normal(n).astype(np.float32), 0).astype(np.float32)
    ws = a3po.new_workspace(a3po.a3po_loss_workspace_bytes(n))
    loss = torch.full((1,), 5.0, device=DEV)
    stats = a3po.new_stats()
    grad = torch.full((n,), 5.0, device=DEV)
    a3po.a3po_decoupled_loss_fwd_bwd(_dev(inp["logp"]), _dev(inp["behav_logp"]), _dev(prox), _dev(inp["adv"]),
                                     _dev(inp["mask"]), inp["clip_eps"], loss, ws, grad_logp=grad, stats=stats)
    torch.cuda.synchronize()
    ref_loss, ref_stats, ref_grad, terms = orc.decoupled_loss(inp["logp"], inp["behav_logp"], prox, inp["adv"],
                                                              inp["mask"], inp["clip_eps"])
    got = a3po.read_stats(stats)
    assert abs(float(loss.item()) - ref_loss) <= LOSS_RTOL * ref_stats["abs_obj_mean"] + 1e-30
    assert got["n_valid"] == ref_stats["n_valid"]
    ambiguous = terms["valid"] & (terms["margin"] < BOUNDARY_REL * terms["r"])
    assert abs(got["n_clipped"] - ref_stats["n_clipped"]) <= int(ambiguous.sum())
    m = max(ref_stats["n_valid"], 1)
    g = grad.cpu().numpy().astype(np.float64)
    ok = (np.abs(g - ref_grad) <= 1e-5 * np.abs(ref_grad) + 1e-7 / m) | ambiguous
    assert ok.all() and not g[inp["mask"] == 0].any()
    # forward-only form
    loss2 = torch.zeros(1, device=DEV)
    a3po.a3po_decoupled_loss_fwd_bwd(_dev(inp["logp"]), _dev(inp["behav_logp"]), _dev(prox), _dev(inp["adv"]),
                                     _dev(inp["mask"]), inp["clip_eps"], loss2, ws)
    torch.cuda.synchronize()
    assert abs(float(loss2.item()) - ref_loss) <= LOSS_RTOL * ref_stats["abs_obj_mean"] + 1e-30


@pytest.mark.parametrize("packed", [False, True])
def test_grpo_advantages_match_oracle(packed):
    name = "8b_packed" if packed else "1p5b"
    kw = dict(n_prompts=5, group=8, len_lo=3, len_hi=400) if packed else dict(n_prompts=3, group=4, row_len=64,
                                                                              len_lo=10, len_hi=64)
    wl = workloads.make_workload(name, with_operands=False, **kw)
    rng = np.random.default_rng(7)
    group = kw["group"]
    rewards = (rng.random(wl.B) < 0.4).astype(np.float32)
    rewards[:group] = 1.0                                      # an all-equal group: advantages are exactly zero
    rewards[group:2 * group] = rng.standard_normal(group)      # real-valued rewards
    adv = torch.full((wl.N,), 9.0, device=DEV)
    ws = a3po.new_workspace(a3po.a3po_grpo_workspace_bytes(wl.B))
    a3po.a3po_grpo_advantages(_dev(rewards), group, _dev(wl.cu_seqlens), adv, ws)
    torch.cuda.synchronize()
    ref = orc.expand_per_sequence(orc.grpo_advantages(rewards, group), wl.cu_seqlens, wl.N)
    got = adv.cpu().numpy()
    assert np.max(np.abs(got - ref)) <= 1e-5 * max(1.0, np.abs(ref).max())
    assert not got[: wl.cu_seqlens[group]].any()
    with pytest.raises(a3po.A3poError):
        a3po.a3po_grpo_advantages(_dev(rewards), group + 1, _dev(wl.cu_seqlens), adv, ws)   # B % group != 0


def test_bounded_wait_gives_up_and_reports():
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    a3po.a3po_selftest_wait_timeout(status, timeout_ms=40)
    stop.record()
    torch.cuda.synchronize()
    assert int(status.item()) == a3po.STATUS_WAIT_TIMEOUT
    assert 30.0 <= start.elapsed_time(stop) <= 500.0
    # the context is still usable afterwards
    assert float(torch.ones(8, device=DEV).sum().item()) == 8.0
