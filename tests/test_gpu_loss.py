"""GPU parity: A-3PO loss kernels (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from paper_2512_06547_b200 import workloads
from tests.helpers import check_loss_outputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dev(inp, offset=0):
    """Device copies; offset > 0 shifts every array by `offset` elements to break 16-byte alignment."""
    out = {}
    for k in ("logp", "behav_logp", "versions", "adv", "mask"):
        a = torch.from_numpy(np.ascontiguousarray(inp[k]))
        if offset:
            buf = torch.empty(a.numel() + offset, dtype=a.dtype, device=DEV)
            buf[offset:].copy_(a)
            out[k] = buf[offset:]
        else:
            out[k] = a.to(DEV)
    return out


def _run_all(inp, detach=True, offset=0, per_seq=None):
    d = _dev(inp, offset)
    n = inp["N"]
    ws = a3po.new_workspace(a3po.a3po_loss_workspace_bytes(n))
    loss = torch.full((1,), 7.0, device=DEV)
    stats = a3po.new_stats()
    versions, cu = d["versions"], None
    if per_seq is not None:
        versions = torch.from_numpy(per_seq[0]).to(DEV)
        cu = torch.from_numpy(per_seq[1]).to(DEV)
    common = (d["logp"], d["behav_logp"], versions, inp["current_version"], d["adv"], d["mask"], inp["clip_eps"])
    a3po.a3po_loss_fwd(*common, loss, ws, stats=stats, cu_seqlens=cu)
    torch.cuda.synchronize()
    loss_fwd = float(loss.item())
    stats_fwd = a3po.read_stats(stats)
    check_loss_outputs(inp, loss_fwd, stats_fwd, None)

    gbuf = torch.full((n + offset,), 9.0, device=DEV)
    g1 = gbuf[offset:]
    a3po.a3po_loss_bwd(*common, g1, ws, detach_prox=detach, fwd_stats=stats, cu_seqlens=cu)
    torch.cuda.synchronize()
    check_loss_outputs(inp, None, None, g1.cpu().numpy(), detach=detach)

    g2 = torch.full((n + offset,), 9.0, device=DEV)[offset:]
    gl = torch.tensor([1.7], device=DEV)
    a3po.a3po_loss_bwd(*common, g2, ws, detach_prox=detach, grad_loss=gl, cu_seqlens=cu)  # counts the mask itself
    torch.cuda.synchronize()
    check_loss_outputs(inp, None, None, g2.cpu().numpy(), detach=detach, grad_loss=float(np.float32(1.7)))

    g3 = torch.full((n + offset,), 9.0, device=DEV)[offset:]
    loss.fill_(7.0)
    stats3 = a3po.new_stats()
    a3po.a3po_loss_fwd_bwd(*common, loss, g3, ws, detach_prox=detach, stats=stats3, cu_seqlens=cu)
    torch.cuda.synchronize()
    check_loss_outputs(inp, float(loss.item()), a3po.read_stats(stats3), g3.cpu().numpy(), detach=detach)
    assert a3po.read_stats(stats3)["n_valid"] == stats_fwd["n_valid"]
    return loss_fwd, stats_fwd, g1


@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 1023, 4096, 1_000_003, 1 << 20])
@pytest.mark.parametrize("correlated", [False, True])
def test_loss_matches_oracle(n, correlated):
    inp = workloads.loss_sweep(n, seed=1234 + n, correlated=correlated)
    _run_all(inp, detach=True)


@pytest.mark.parametrize("detach", [True, False])
def test_both_gradient_readings(detach):
    inp = workloads.loss_sweep(50_001, seed=77, correlated=True)
    _run_all(inp, detach=detach)


@pytest.mark.parametrize("offset", [1, 3])
def test_misaligned_arrays_take_the_scalar_path(offset):
    inp = workloads.loss_sweep(10_007, seed=5, correlated=True)
    _run_all(inp, offset=offset)


def test_masked_tokens_may_hold_nan():
    inp = workloads.loss_sweep(20_000, seed=6, correlated=True)
    clean_loss, clean_stats, clean_g = _run_all(inp)
    dirty = dict(inp)
    for k in ("logp", "behav_logp", "adv"):
        a = inp[k].copy()
        a[inp["mask"] == 0] = np.nan
        dirty[k] = a
    dirty["logp"][np.flatnonzero(inp["mask"] == 0)[:3]] = np.inf
    loss, stats, g = _run_all(dirty)
    assert loss == clean_loss and stats == clean_stats and torch.equal(g, clean_g)


def test_all_masked_and_run_to_run_determinism():
    inp = workloads.loss_sweep(9999, seed=8)
    inp["mask"] = np.zeros_like(inp["mask"])
    loss, stats, g = _run_all(inp)
    assert loss == 0.0 and stats["n_valid"] == 0 and not g.any()
    inp = workloads.loss_sweep(3_000_001, seed=9, correlated=True)
    a = _run_all(inp)
    b = _run_all(inp)
    assert a[0] == b[0] and a[1] == b[1] and torch.equal(a[2], b[2])


def test_versions_per_sequence_with_cu_seqlens():
    wl = workloads.make_workload("8b_packed", with_operands=False, n_prompts=3, group=4, len_lo=5, len_hi=700)
    rng = np.random.default_rng(3)
    logp = (-rng.standard_exponential(wl.N)).astype(np.float32)
    inp = dict(logp=logp, behav_logp=workloads.behav_logp_from(logp, wl.behav_noise), versions=wl.versions,
               current_version=wl.current_version, adv=wl.adv, mask=wl.mask, clip_eps=wl.clip_eps, N=wl.N)
    assert len(set(wl.versions_per_seq.tolist())) > 1
    _run_all(inp, per_seq=(wl.versions_per_seq, wl.cu_seqlens))


def test_staleness_edge_cases():
    """d < 0, d = 0, d = 1 and a huge d, on identical tokens (alpha = 1, 1, 1, ~0)."""
    n = 4096
    inp = workloads.loss_sweep(n, seed=10, correlated=True)
    cur = inp["current_version"]
    inp["versions"] = np.resize(np.array([cur + 5, cur, cur - 1, cur - 2, cur - 1_000_000, -2**31 + 7], np.int32), n)
    _run_all(inp)


def test_workspace_too_small_is_an_error():
    inp = workloads.loss_sweep(1000, seed=11)
    d = _dev(inp)
    loss = torch.zeros(1, device=DEV)
    with pytest.raises(a3po.A3poError) as e:
        a3po.a3po_loss_fwd(d["logp"], d["behav_logp"], d["versions"], 1, d["adv"], d["mask"], 0.2, loss,
                           a3po.new_workspace(256))
    assert e.value.code == -3
