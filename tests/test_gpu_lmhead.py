"""GPU parity: LM-head log-prob forward/backward (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from oracle import a3po_oracle as orc
from paper_2512_06547_b200 import workloads
from tests.helpers import GRAD_FRO_RTOL, LOGP_TOL_BF16, LOGP_TOL_F32, rel_fro, row_rel_err, to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def gpu_fwd(hidden, w, targets, row_mask=None, want_entropy=False, inv_t=1.0):
    n, h = hidden.shape
    v = w.shape[0]
    dt = a3po.A3PO_F32 if hidden.dtype == torch.float32 else a3po.A3PO_BF16
    ws = a3po.new_workspace(a3po.a3po_token_logprobs_workspace_bytes(n, h, v, dt, 0))
    logp = torch.full((n,), 5.0, device=DEV)
    lse = torch.full((n,), 5.0, device=DEV)
    ent = torch.full((n,), 5.0, device=DEV) if want_entropy else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    a3po.a3po_token_logprobs_fwd(hidden, w, targets, logp, lse, ws, row_mask=row_mask, entropy=ent,
                                 inv_temperature=inv_t, status=status)
    torch.cuda.synchronize()
    return logp, lse, ent, int(status.item())


def gpu_bwd(hidden, w, targets, lse, grad_logp, grad_w=None, accumulate=False, inv_t=1.0, ws_bytes=None):
    n, h = hidden.shape
    v = w.shape[0]
    dt = a3po.A3PO_F32 if hidden.dtype == torch.float32 else a3po.A3PO_BF16
    if ws_bytes is None:
        ws_bytes = a3po.a3po_token_logprobs_workspace_bytes(n, h, v, dt, 1)
    ws = a3po.new_workspace(ws_bytes)
    gh = torch.full_like(hidden, 3.0)
    if grad_w is None:
        grad_w = torch.full((v, h), 3.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    a3po.a3po_token_logprobs_bwd(hidden, w, targets, lse, grad_logp, gh, grad_w, ws, accumulate_grad_w=accumulate,
                                 inv_temperature=inv_t, status=status)
    torch.cuda.synchronize()
    return gh, grad_w, int(status.item())


def _problem(n, h, v, dtype, seed):
    hidden, w = workloads.lm_head_operands(n, h, v, dtype, seed, DEV)
    rng = np.random.default_rng(seed)
    targets = torch.from_numpy(rng.integers(0, v, size=n).astype(np.int32)).to(DEV)
    g = rng.standard_normal(n).astype(np.float32) / max(n, 1)
    g[rng.random(n) < 0.2] = 0.0
    return hidden, w, targets, torch.from_numpy(g).to(DEV)


def _check_fwd_bwd(n, h, v, dtype, seed, inv_t=1.0, want_entropy=True):
    hidden, w, targets, g = _problem(n, h, v, dtype, seed)
    tol = LOGP_TOL_F32 if dtype == "f32" else LOGP_TOL_BF16
    logp, lse, ent, status = gpu_fwd(hidden, w, targets, want_entropy=want_entropy, inv_t=inv_t)
    assert status == 0
    hn, wn, tn = to_np64(hidden), to_np64(w), targets.cpu().numpy()
    logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, tn, inv_temperature=inv_t)
    scale = np.maximum(1.0, np.abs(lse_ref)) if dtype == "f32" else 1.0
    assert np.max(np.abs(logp.cpu().numpy() - logp_ref) / scale) <= tol
    assert np.max(np.abs(lse.cpu().numpy() - lse_ref) / scale) <= tol
    if want_entropy:
        ent_ref = orc.token_entropy(hn, wn, inv_temperature=inv_t)
        assert np.max(np.abs(ent.cpu().numpy() - ent_ref)) <= (1e-4 if dtype == "f32" else 5e-3)
    gh, gw, status = gpu_bwd(hidden, w, targets, lse, g, inv_t=inv_t)
    assert status == 0
    gh_ref, gw_ref = orc.token_logprobs_bwd(hn, wn, tn, to_np64(g), inv_temperature=inv_t)
    bound = 1e-4 if dtype == "f32" else GRAD_FRO_RTOL
    assert rel_fro(to_np64(gh), gh_ref) <= bound
    assert rel_fro(to_np64(gw), gw_ref) <= bound
    zero_rows = (g == 0).cpu().numpy()
    assert not to_np64(gh)[zero_rows].any()
    return hidden, w, targets, g, lse, gw, gw_ref


def test_tiny_config_fp32_full_compare():
    """Config 'tiny': H=64, V=1000, N=512, fp32 (rows, columns and K all have ragged tiles)."""
    wl = workloads.make_workload("tiny", DEV)
    targets = torch.from_numpy(wl.targets).to(DEV)
    mask = torch.from_numpy(wl.mask).to(DEV)
    logp, lse, ent, status = gpu_fwd(wl.hidden, wl.w, targets, row_mask=mask, want_entropy=True)
    assert status == 0
    logp_ref, lse_ref = orc.token_logprobs_fwd(to_np64(wl.hidden), to_np64(wl.w), wl.targets, row_mask=wl.mask)
    assert np.max(np.abs(logp.cpu().numpy() - logp_ref)) <= LOGP_TOL_F32 * 10   # |lse| ~ 7
    assert np.max(np.abs(lse.cpu().numpy() - lse_ref)) <= LOGP_TOL_F32 * 10
    assert not logp.cpu().numpy()[wl.mask == 0].any()


@pytest.mark.parametrize("n,h,v", [(1, 8, 5), (63, 24, 64), (65, 40, 129), (200, 64, 1000), (130, 72, 333)])
def test_fp32_shapes(n, h, v):
    _check_fwd_bwd(n, h, v, "f32", seed=100 + n, inv_t=0.9)


@pytest.mark.parametrize("n,h,v", [(515, 1536, 4096 + 37), (131, 256, 777), (128, 64, 256), (300, 4096, 2048 + 8),
                                   (257, 72, 1000), (64, 8, 9), (1, 200, 300), (33, 12, 50)])
def test_bf16_shrunken_shapes(n, h, v):
    """Same H as the 1.5B / 8B heads, shrunken V and N with ragged row and vocabulary tails; also hidden sizes
    that are not a multiple of the 64-wide K block (72, 8, 200: the K tail is zero-filled by the TMA loads), a
    vocabulary smaller than one column tile, a single row, and a hidden size (12) whose rows are not 16-byte
    multiples, which the tensor-core path rejects and the FP32-pipe kernels take."""
    _check_fwd_bwd(n, h, v, "bf16", seed=200 + n)


def test_bf16_temperature_and_entropy():
    _check_fwd_bwd(260, 512, 3000, "bf16", seed=31, inv_t=1.0 / 0.7)


def test_grad_w_accumulates_and_chunks_agree():
    """accumulate_grad_w adds into the existing buffer; a workspace that forces several row chunks
    gives the same gradients as one chunk."""
    n, h, v = 400, 128, 1500
    hidden, w, targets, g, lse, gw, gw_ref = _check_fwd_bwd(n, h, v, "bf16", seed=41, want_entropy=False)
    base = torch.randn(v, h, device=DEV)
    _, acc, _ = gpu_bwd(hidden, w, targets, lse, g, grad_w=base.clone(), accumulate=True)
    assert rel_fro(to_np64(acc - base), gw_ref) <= GRAD_FRO_RTOL
    small = a3po.a3po_token_logprobs_min_workspace_bytes(n, h, v, a3po.A3PO_BF16, 1)
    gh_small, gw_small, _ = gpu_bwd(hidden, w, targets, lse, g, ws_bytes=small)
    assert rel_fro(to_np64(gw_small), gw_ref) <= GRAD_FRO_RTOL
    with pytest.raises(a3po.A3poError):
        gpu_bwd(hidden, w, targets, lse, g, ws_bytes=small // 4)


def test_out_of_range_target_is_flagged_not_dereferenced():
    hidden, w, targets, g = _problem(100, 64, 300, "bf16", 51)
    bad = targets.clone()
    bad[7] = 300
    bad[9] = -4
    logp, lse, _, status = gpu_fwd(hidden, w, bad)
    assert status & a3po.STATUS_TARGET_OUT_OF_RANGE
    good, lse_good, _, status = gpu_fwd(hidden, w, targets)
    assert status == 0
    keep = torch.ones(100, dtype=torch.bool, device=DEV)
    keep[7] = keep[9] = False
    assert torch.equal(logp[keep], good[keep]) and torch.equal(lse, lse_good)
    assert torch.isfinite(logp).all()


def test_empty_batch():
    hidden, w, targets, g = _problem(0, 64, 300, "bf16", 52)
    logp, lse, _, status = gpu_fwd(hidden, w, targets)
    gh, gw, _ = gpu_bwd(hidden, w, targets, lse, g)
    assert not gw.any()


def test_full_vocab_sub_batch_1p5b():
    """Full-size V and H of the 1.5B-shaped config on a sub-batch of rows (all outputs)."""
    _check_fwd_bwd(384, 1536, workloads.QWEN_VOCAB, "bf16", seed=61, want_entropy=False)


def test_masked_and_zero_gradient_rows_are_skipped_consistently():
    """Row compaction: any pattern of masked rows (forward) or zero upstream gradients (backward), including
    none and all of them, gives the same numbers as the oracle; grad_w is exactly zero / untouched when no row
    takes part."""
    n, h, v = 700, 256, 2000
    hidden, w, targets, g = _problem(n, h, v, "bf16", 71)
    hn, wn, tn = to_np64(hidden), to_np64(w), targets.cpu().numpy()
    rng = np.random.default_rng(72)
    for keep_frac in (0.0, 0.03, 0.5, 1.0):
        mask_np = (rng.random(n) < keep_frac).astype(np.uint8)
        mask = torch.from_numpy(mask_np).to(DEV)
        logp, lse, _, status = gpu_fwd(hidden, w, targets, row_mask=mask)
        assert status == 0
        logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, tn, row_mask=mask_np)
        assert np.max(np.abs(logp.cpu().numpy() - logp_ref), initial=0.0) <= LOGP_TOL_BF16
        assert np.max(np.abs(lse.cpu().numpy() - lse_ref), initial=0.0) <= LOGP_TOL_BF16
        assert not logp.cpu().numpy()[mask_np == 0].any()
        # backward with the upstream gradient restricted to the kept rows
        g_np = g.cpu().numpy() * mask_np
        full_lse = torch.from_numpy(orc.token_logprobs_fwd(hn, wn, tn)[1].astype(np.float32)).to(DEV)
        gh, gw, status = gpu_bwd(hidden, w, targets, full_lse, torch.from_numpy(g_np).to(DEV))
        assert status == 0
        gh_ref, gw_ref = orc.token_logprobs_bwd(hn, wn, tn, g_np.astype(np.float64))
        if g_np.any():
            assert rel_fro(to_np64(gh), gh_ref) <= GRAD_FRO_RTOL and rel_fro(to_np64(gw), gw_ref) <= GRAD_FRO_RTOL
        else:
            assert not gh.float().abs().sum().item() and not gw.abs().sum().item()     # overwritten with zeros
            base = torch.randn(v, h, device=DEV)
            _, acc, _ = gpu_bwd(hidden, w, targets, full_lse, torch.zeros(n, device=DEV), grad_w=base.clone(),
                                accumulate=True)
            assert torch.equal(acc, base)                                              # accumulate: untouched
        assert not to_np64(gh)[g_np == 0].any()


def _keep_pair(hidden, w, targets, g, mask=None, want_entropy=False):
    n, h = hidden.shape
    v = w.shape[0]
    kept = a3po.new_workspace(a3po.a3po_kept_bytes(n, v))
    ws = a3po.new_workspace(max(a3po.a3po_token_logprobs_fwd_keep_workspace_bytes(n, h, v),
                                a3po.a3po_token_logprobs_bwd_kept_workspace_bytes(n, h, v)))
    logp, lse = torch.full((n,), 5.0, device=DEV), torch.full((n,), 5.0, device=DEV)
    ent = torch.full((n,), 5.0, device=DEV) if want_entropy else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    a3po.a3po_token_logprobs_fwd_keep(hidden, w, targets, logp, lse, kept, ws, row_mask=mask, entropy=ent,
                                      status=status)
    ws.fill_(0xAB)                                              # the backward must not depend on the forward's scratch
    gh = torch.full_like(hidden, 3.0)
    gw = torch.full((v, h), 3.0, dtype=torch.float32, device=DEV)
    a3po.a3po_token_logprobs_bwd_kept(hidden, w, targets, lse, g, kept, gh, gw, ws, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return logp, lse, ent, gh, gw, kept, ws


@pytest.mark.parametrize("n,h,v", [(600, 512, 8192 + 24), (300, 1536, 4096 + 40)])
def test_peaked_rows_both_backward_paths(n, h, v):
    """Confident rows, as in an RL fine-tuning batch: target probability between 0.3 and 0.999, half of the
    targets in the last eighth of the vocabulary (late column tiles, last split).  dz at the target is
    g (1 - p_y), a cancellation; the recomputing pair and the keeping pair must both hold the gradient
    tolerance row by row, not only over the whole matrix."""
    hidden, w, _, g = _problem(n, h, v, "bf16", 300 + n)
    targets_np = workloads.peak_targets(hidden, w, np.random.default_rng(17 + n))
    targets = torch.from_numpy(targets_np).to(DEV)
    hn, wn = to_np64(hidden), to_np64(w)
    logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, targets_np)
    p_y = np.exp(logp_ref)
    assert p_y.min() < 0.45 and p_y.max() > 0.995 and np.median(p_y) > 0.8          # the rows really are peaked
    gh_ref, gw_ref = orc.token_logprobs_bwd(hn, wn, targets_np, to_np64(g))
    ent_ref = orc.token_entropy(hn, wn)
    live = to_np64(g) != 0

    logp, lse, ent, status = gpu_fwd(hidden, w, targets, want_entropy=True)
    assert status == 0
    gh, gw, status = gpu_bwd(hidden, w, targets, lse, g)
    assert status == 0
    k_logp, k_lse, k_ent, k_gh, k_gw, _, _ = _keep_pair(hidden, w, targets, g, want_entropy=True)
    for tag, (lp, ls, en, a, b) in {"recomputing pair": (logp, lse, ent, gh, gw),
                                    "keeping pair": (k_logp, k_lse, k_ent, k_gh, k_gw)}.items():
        e_lp = np.max(np.abs(lp.cpu().numpy() - logp_ref))
        e_ls = np.max(np.abs(ls.cpu().numpy() - lse_ref))
        e_en = np.max(np.abs(en.cpu().numpy() - ent_ref))
        e_row = row_rel_err(to_np64(a)[live], gh_ref[live])
        e_gw = rel_fro(to_np64(b), gw_ref)
        print(f"[peaked {tag} n={n} h={h} v={v}] logp {e_lp:.2e} lse {e_ls:.2e} entropy {e_en:.2e} "
              f"grad_hidden rows: median {np.median(e_row):.2e} worst {e_row.max():.2e}  grad_w fro {e_gw:.2e}")
        assert e_lp <= LOGP_TOL_BF16 and e_ls <= LOGP_TOL_BF16 and e_en <= 5e-3
        assert e_row.max() <= GRAD_FRO_RTOL and e_gw <= GRAD_FRO_RTOL
        assert not to_np64(a)[~live].any()


def test_forward_keep_backward_kept_pair_matches_oracle_and_plain_pair():
    """The forward that keeps its softmax and the backward that uses it, as two separate calls with the
    upstream gradient computed in between (as under an autograd engine)."""
    n, h, v = 700, 512, 5000 + 24
    hidden, w, targets, g = _problem(n, h, v, "bf16", 91)
    rng = np.random.default_rng(92)
    mask_np = (rng.random(n) < 0.7).astype(np.uint8)
    mask = torch.from_numpy(mask_np).to(DEV)
    g = g * mask                                                # skipped rows carry no gradient
    logp, lse, _, gh, gw, kept, ws = _keep_pair(hidden, w, targets, g, mask=mask)
    hn, wn, tn = to_np64(hidden), to_np64(w), targets.cpu().numpy()
    logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, tn, row_mask=mask_np)
    assert np.max(np.abs(logp.cpu().numpy() - logp_ref)) <= LOGP_TOL_BF16
    assert np.max(np.abs(lse.cpu().numpy() - lse_ref)) <= LOGP_TOL_BF16
    gh_ref, gw_ref = orc.token_logprobs_bwd(hn, wn, tn, to_np64(g))
    assert rel_fro(to_np64(gh), gh_ref) <= GRAD_FRO_RTOL and rel_fro(to_np64(gw), gw_ref) <= GRAD_FRO_RTOL
    assert not to_np64(gh)[to_np64(g) == 0].any()
    # the plain pair gives the same gradients within the tolerance, and accumulation works on the kept pair too
    gh2, gw2, _ = gpu_bwd(hidden, w, targets, lse, g)
    assert rel_fro(to_np64(gw), to_np64(gw2)) <= GRAD_FRO_RTOL and rel_fro(to_np64(gh), to_np64(gh2)) <= GRAD_FRO_RTOL
    base = torch.randn(v, h, device=DEV)
    acc = base.clone()
    a3po.a3po_token_logprobs_bwd_kept(hidden, w, targets, lse, g, kept, gh, acc, ws, accumulate_grad_w=True)
    torch.cuda.synchronize()
    assert rel_fro(to_np64(acc - base), gw_ref) <= GRAD_FRO_RTOL
    # a row the forward skipped has nothing kept: whatever upstream gradient it carries is ignored (never used as
    # an index), so the result is the one for g * mask
    g_stray = g.clone()
    g_stray[mask == 0] = 1.0
    gh3 = torch.full_like(hidden, 3.0)
    gw3 = torch.full((v, h), 3.0, dtype=torch.float32, device=DEV)
    a3po.a3po_token_logprobs_bwd_kept(hidden, w, targets, lse, g_stray, kept, gh3, gw3, ws)
    torch.cuda.synchronize()
    assert torch.equal(gw3, gw) and torch.equal(gh3, gh)
    # shapes outside the tensor-core path are refused, not silently computed another way
    h_odd, w_odd, t_odd, g_odd = _problem(16, 12, 40, "bf16", 93)
    with pytest.raises(a3po.A3poError) as e:
        a3po.a3po_token_logprobs_fwd_keep(h_odd, w_odd, t_odd, torch.empty(16, device=DEV), torch.empty(16, device=DEV),
                                          a3po.new_workspace(a3po.a3po_kept_bytes(16, 40)),
                                          a3po.new_workspace(a3po.a3po_token_logprobs_fwd_keep_workspace_bytes(16, 12, 40)))
    assert e.value.code == -2
