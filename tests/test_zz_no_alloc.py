"""a3po_loss_fwd_static: the loss forward for callers that cannot hand the library a workspace.

Some users of this library run where no device memory can be obtained at call time: a callback
inside a framework that keeps its allocator to itself, a loop that must not stall on an
allocation, a process whose GPU memory was handed out in full beforehand.  For them the library
carries its own fixed scratch array.  This file checks, through the C ABI, that the variant gives
the same answer as a3po_loss_fwd with a caller workspace, on two calls in a row that share the
array (the second with different data, so leftovers of the first would show), and that a batch
beyond the stated maximum is refused on the host.  It is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from oracle import a3po_oracle as orc
from paper_2512_06547_b200 import workloads
from paper_2512_06547_b200.binding import LOSS_FWD_STATIC_MAX_TOKENS
from tests.helpers import LOSS_RTOL

DEV = "cuda"


def _both_ways(inp, per_seq=None, warmed_up=True):
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    logp, behav, versions, adv, mask = (to_dev(inp[k]) for k in ("logp", "behav_logp", "versions", "adv", "mask"))
    cu = None
    if per_seq is not None:
        versions, cu = to_dev(per_seq[0]), to_dev(per_seq[1])
    args = (logp, behav, versions, inp["current_version"], adv, mask, inp["clip_eps"])
    loss_ws, loss_st = torch.full((1,), 3.0, device=DEV), torch.full((1,), 4.0, device=DEV)
    stats_ws, stats_st = a3po.new_stats(), a3po.new_stats()
    ws = a3po.new_workspace(a3po.a3po_loss_workspace_bytes(inp["N"]))
    a3po.a3po_loss_fwd(*args, loss_ws, ws, stats=stats_ws, cu_seqlens=cu)
    torch.cuda.synchronize()
    # the entry exists for callers that cannot obtain device memory: it must not obtain any itself
    # (the driver reports the device's free memory; torch's caching allocator is not involved in the call)
    free_before, _ = torch.cuda.mem_get_info()
    a3po.a3po_loss_fwd_static(*args, loss_st, stats=stats_st, cu_seqlens=cu)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    if warmed_up:
        assert free_after == free_before, (free_before, free_after)
    loss_ref, ref = orc.loss_fwd(inp["logp"], inp["behav_logp"], inp["versions"], inp["current_version"], inp["adv"],
                                 inp["mask"], inp["clip_eps"])
    assert abs(float(loss_st.item()) - float(loss_ws.item())) <= LOSS_RTOL * ref["abs_obj_mean"]
    assert abs(float(loss_st.item()) - loss_ref) <= LOSS_RTOL * ref["abs_obj_mean"]      # and against the oracle
    s_ws, s_st = a3po.read_stats(stats_ws), a3po.read_stats(stats_st)
    assert s_st["n_valid"] == s_ws["n_valid"] == ref["n_valid"]
    assert s_st["n_clipped"] == s_ws["n_clipped"]
    assert s_st["iw_max"] == pytest.approx(s_ws["iw_max"], rel=1e-5)
    assert s_st["iw_min"] == pytest.approx(s_ws["iw_min"], rel=1e-5)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_twice_in_a_row():
    first = workloads.loss_sweep(300_007, seed=901, correlated=True)
    # the very first launch of a kernel in a process may make the driver load its code (lazy module loading),
    # which is not the call allocating: the free-memory check applies from the second call on
    _both_ways(first, warmed_up=False)
    _both_ways(first)
    second = workloads.loss_sweep(41_003, seed=902, correlated=False)     # smaller: most of the array keeps call 1's data
    _both_ways(second)
    # per-sequence versions use the part of the array that holds the expanded per-token versions
    wl = workloads.make_workload("8b_packed", with_operands=False, n_prompts=2, group=4, len_lo=9, len_hi=900)
    logp = (-np.random.default_rng(5).standard_exponential(wl.N)).astype(np.float32)
    third = dict(logp=logp, behav_logp=workloads.behav_logp_from(logp, wl.behav_noise), versions=wl.versions,
                 current_version=wl.current_version, adv=wl.adv, mask=wl.mask, clip_eps=wl.clip_eps, N=wl.N)
    _both_ways(third, per_seq=(wl.versions_per_seq, wl.cu_seqlens))
    _both_ways(workloads.loss_sweep(LOSS_FWD_STATIC_MAX_TOKENS, seed=903, correlated=True))   # exactly the maximum


@pytest.mark.gpu
def test_batch_beyond_the_maximum_is_refused():
    lib = a3po.load_library()
    small = torch.zeros(16, device=DEV)
    before = small.clone()
    p = ctypes.c_void_p(small.data_ptr())
    rc = lib.a3po_loss_fwd_static(p, p, p, 0, None, 0, 1, p, p, LOSS_FWD_STATIC_MAX_TOKENS + 1, 0.2, p, None, None)
    assert rc == -6 and b"A3PO_LOSS_FWD_STATIC_MAX_TOKENS" in lib.a3po_status_string(rc)
    torch.cuda.synchronize()
    assert torch.equal(small, before)                    # refused before anything ran
