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
