"""Shared comparators for the GPU parity tests (tolerances are stated here, once)."""
import numpy as np
import torch

from oracle import a3po_oracle as orc

# Tolerances (floating point):
#   per-token logp / lse: bf16 inputs with fp32 accumulation |err| <= 2e-3; fp32 inputs 1e-5 * max(1, |lse|)
#   loss: |L_gpu - L_ref| <= 1e-5 * mean_valid |obj|          (relative to the L1 scale of the mean)
#   dL/dlogp: |dg_t| <= 1e-5 |g_ref,t| + 1e-7 / M, except tokens whose ratio sits within 1e-5 (relative) of a
#             clip bound, where fp32 and fp64 may legitimately pick different branches: either value is accepted
#   grad_hidden / grad_w: relative Frobenius error <= 1e-2
LOGP_TOL_BF16 = 2e-3
LOGP_TOL_F32 = 1e-5
LOSS_RTOL = 1e-5
GRAD_FRO_RTOL = 1e-2
BOUNDARY_REL = 1e-5


def to_np64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a (bf16 / fp32 / int) tensor to a float64 or integer numpy array."""
    t = t.detach().cpu()
    if t.dtype in (torch.bfloat16, torch.float16, torch.float32):
        return t.to(torch.float64).numpy()
    return t.numpy()


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def row_rel_err(a, b):
    """Per-row relative error ||a_t - b_t|| / ||b_t|| of two [N, H] arrays (rows with b_t = 0 report ||a_t||)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    num = np.linalg.norm(a - b, axis=1)
    den = np.linalg.norm(b, axis=1)
    return np.where(den > 0, num / np.where(den > 0, den, 1.0), num)


def chained_loss_tol(terms, logp_tol):
    """Bound on |L_gpu - L_ref| when the loss stage consumes log-probs that are off by at most `logp_tol`:
    the loss value depends on l_theta through iw = w^(1-alpha) and r = w^alpha, so
    |dL| <= logp_tol * mean_valid |(1 - alpha) obj + alpha iw A r act|  (+ the loss kernel's own 1e-5 mean|obj|)."""
    valid = terms["valid"]
    m = max(int(valid.sum()), 1)
    through = terms["iw"] * terms["adv"] * terms["r"] * terms["act"]
    dobj = (1.0 - terms["alpha"]) * terms["obj"] + terms["alpha"] * through
    return (logp_tol * float(np.abs(dobj[valid]).sum()) + LOSS_RTOL * float(np.abs(terms["obj"][valid]).sum())) / m


def check_loss_outputs(inp, loss_gpu, stats_gpu, grad_gpu, detach=True, grad_loss=1.0):
    """inp: dict of numpy arrays (logp, behav_logp, versions [per token], current_version, adv, mask, clip_eps)."""
    args = (inp["logp"], inp["behav_logp"], inp["versions"], inp["current_version"], inp["adv"], inp["mask"],
            inp["clip_eps"])
    terms = orc.loss_terms(*args)
    loss_ref, stats_ref = orc.loss_fwd(*args)
    valid = terms["valid"]
    m = max(stats_ref["n_valid"], 1)
    ambiguous = valid & (terms["margin"] < BOUNDARY_REL * terms["r"])
    n_amb = int(ambiguous.sum())
    if loss_gpu is not None:
        assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * stats_ref["abs_obj_mean"] + 1e-30, (loss_gpu, loss_ref)
    if stats_gpu is not None:
        assert stats_gpu["n_valid"] == stats_ref["n_valid"]
        assert abs(stats_gpu["n_clipped"] - stats_ref["n_clipped"]) <= n_amb
        if stats_ref["n_valid"]:
            assert abs(stats_gpu["iw_max"] - stats_ref["iw_max"]) <= 1e-5 * stats_ref["iw_max"]
            assert abs(stats_gpu["iw_min"] - stats_ref["iw_min"]) <= 1e-5 * stats_ref["iw_min"]
        else:
            assert stats_gpu["iw_max"] == 0.0 and stats_gpu["iw_min"] == 0.0
    if grad_gpu is not None:
        g_ref = orc.loss_bwd(*args, detach_prox=detach, grad_loss=grad_loss)
        g = np.asarray(grad_gpu, dtype=np.float64)
        assert np.all(g[~valid] == 0.0)
        ok = np.abs(g - g_ref) <= 1e-5 * np.abs(g_ref) + 1e-7 / m
        if n_amb:
            # on a clip bound either branch is a correct answer: compare with the other branch too
            flipped = dict(terms)
            through = terms["iw"] * terms["adv"] * terms["r"] * (~terms["act"])
            if detach:
                alt = through
            else:
                alt = (1.0 - terms["alpha"]) * terms["obj"] + terms["alpha"] * through
            alt = np.where(valid, -(grad_loss / m) * alt, 0.0)
            ok |= ambiguous & (np.abs(g - alt) <= 1e-5 * np.abs(alt) + 1e-7 / m)
        bad = np.flatnonzero(~ok)
        assert bad.size == 0, (bad[:5], g[bad[:5]], g_ref[bad[:5]])
    return loss_ref, stats_ref


def check_loss_outputs_sliced(inp, loss_gpu, stats_gpu, grad_gpu, slice_tokens=1 << 22):
    """check_loss_outputs for token counts whose fp64 intermediates would not fit in memory at once: the oracle's
    per-token terms are evaluated slice by slice (tokens only interact through the mean, whose numerator, M and
    diagnostics are accumulated here in the order of the slices); default reading (anchor detached)."""
    n = int(inp["N"])
    tot_obj = tot_abs = 0.0
    m = n_clip = n_amb = 0
    iw_max, iw_min = 0.0, np.inf
    for lo in range(0, n, slice_tokens):          # pass 1: M and the forward quantities
        sl = slice(lo, min(lo + slice_tokens, n))
        t = orc.loss_terms(inp["logp"][sl], inp["behav_logp"][sl], inp["versions"][sl], inp["current_version"],
                           inp["adv"][sl], inp["mask"][sl], inp["clip_eps"])
        v = t["valid"]
        m += int(v.sum())
        tot_obj += float(t["obj"][v].sum())
        tot_abs += float(np.abs(t["obj"][v]).sum())
        n_clip += int((v & ~t["act"]).sum())
        n_amb += int((v & (t["margin"] < BOUNDARY_REL * t["r"])).sum())
        if v.any():
            iw_max, iw_min = max(iw_max, float(t["iw"][v].max())), min(iw_min, float(t["iw"][v].min()))
    loss_ref = -tot_obj / max(m, 1)
    assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * tot_abs / max(m, 1) + 1e-30, (loss_gpu, loss_ref)
    assert stats_gpu["n_valid"] == m and abs(stats_gpu["n_clipped"] - n_clip) <= n_amb
    assert abs(stats_gpu["iw_max"] - iw_max) <= 1e-5 * iw_max and abs(stats_gpu["iw_min"] - iw_min) <= 1e-5 * iw_min
    for lo in range(0, n, slice_tokens):          # pass 2: every token's gradient, with the global M
        sl = slice(lo, min(lo + slice_tokens, n))
        t = orc.loss_terms(inp["logp"][sl], inp["behav_logp"][sl], inp["versions"][sl], inp["current_version"],
                           inp["adv"][sl], inp["mask"][sl], inp["clip_eps"])
        v = t["valid"]
        g = np.asarray(grad_gpu[sl], dtype=np.float64)
        through = t["iw"] * t["adv"] * t["r"]
        g_ref = np.where(v, -(1.0 / m) * through * t["act"], 0.0)
        g_alt = np.where(v, -(1.0 / m) * through * (~t["act"]), 0.0)
        amb = v & (t["margin"] < BOUNDARY_REL * t["r"])
        ok = np.abs(g - g_ref) <= 1e-5 * np.abs(g_ref) + 1e-7 / m
        ok |= amb & (np.abs(g - g_alt) <= 1e-5 * np.abs(g_alt) + 1e-7 / m)
        assert np.all(g[~v] == 0.0)
        bad = np.flatnonzero(~ok)
        assert bad.size == 0, (lo, bad[:5], g[bad[:5]], g_ref[bad[:5]])
    return loss_ref
