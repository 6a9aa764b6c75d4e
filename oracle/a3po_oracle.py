"""fp64 CPU oracle for the A-3PO log-prob + loss path.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain definition of what the CUDA library computes.  It exists so
that tests, the smoke check and the CPU-baseline leg of the benchmark can compare against it.
The product path never imports it, and it imports nothing from the product package: the two
share no code, tables or helpers.

Everything is numpy in float64.  Inputs of lower precision (bf16 / fp32 arrays that the GPU
reads) are widened exactly to float64 before any arithmetic; `clip_eps` is taken as the fp32
value that crosses the C ABI, widened.  No blocking, fusion or reordering beyond processing
token rows in independent slabs (rows never interact before the final mean), so each function
can be checked against the paper by eye.

Notation follows the paper: l_theta = log pi_theta(a_t|s_t) (current policy), l_behav =
log pi_behav, l_prox = log pi_prox, d = staleness, alpha = interpolation coefficient,
w = pi_theta/pi_behav, r = pi_theta/pi_prox, iw = pi_prox/pi_behav, A = advantage, eps = clip.

Pins (tests/test_oracle_*.py) — every function below is pinned to something other than
itself: softmax normalisation, W=0 closed form, brute-force scalar loops, scipy's logsumexp,
finite differences, the sandwich / closed-form / contraction statements of the theorem, the
d=0 reduction to coupled PPO (Eq. 1) and a hand-derived worked example.  Nothing here is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "lm_head_logits",
    "token_logprobs_fwd",
    "token_entropy",
    "token_logprobs_bwd",
    "expand_per_sequence",
    "staleness",
    "staleness_alpha",
    "prox_logp",
    "loss_terms",
    "loss_fwd",
    "loss_bwd",
    "decoupled_loss",
    "grpo_advantages",
]

_ROW_SLAB = 256  # rows handled per slab; rows are independent, this only bounds memory


def _f64(x):
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------------------
# LM head -> per-token log-probabilities  (policy forward, last stage; Sec. 2.2 "forward
# pass", Sec. 3 "token log-probabilities", Sec. 4.1 sampling temperature 1.0)
# --------------------------------------------------------------------------------------
def lm_head_logits(hidden, w, inv_temperature=1.0):
    """z[t, v] = inv_T * sum_k hidden[t, k] * W[v, k]   (hidden [N,H], W [V,H], both row-major)."""
    return (_f64(hidden) @ _f64(w).T) * float(inv_temperature)


def token_logprobs_fwd(hidden, w, targets, inv_temperature=1.0, row_mask=None):
    """Per-token log pi_theta(y_t | s_t) = z[t, y_t] - logsumexp_v z[t, v].

    Returns (logp [N], lse [N]) in float64.  Rows whose `row_mask` entry is 0 are not part of
    the batch: they return logp = 0 and lse = 0.
    """
    hidden = _f64(hidden)
    w = _f64(w)
    targets = np.asarray(targets, dtype=np.int64)
    n = hidden.shape[0]
    v = w.shape[0]
    if n and (targets.min() < 0 or targets.max() >= v):
        raise ValueError("target index outside [0, V)")
    logp = np.zeros(n)
    lse = np.zeros(n)
    for lo in range(0, n, _ROW_SLAB):
        hi = min(lo + _ROW_SLAB, n)
        z = lm_head_logits(hidden[lo:hi], w, inv_temperature)
        mx = z.max(axis=1)
        s = np.exp(z - mx[:, None]).sum(axis=1)
        lse[lo:hi] = mx + np.log(s)
        logp[lo:hi] = z[np.arange(hi - lo), targets[lo:hi]] - lse[lo:hi]
    if row_mask is not None:
        keep = np.asarray(row_mask) != 0
        logp = np.where(keep, logp, 0.0)
        lse = np.where(keep, lse, 0.0)
    return logp, lse


def token_entropy(hidden, w, inv_temperature=1.0):
    """Policy entropy per row, H_t = -sum_v p_v log p_v (the stability diagnostic of Fig. 4)."""
    hidden = _f64(hidden)
    w = _f64(w)
    n = hidden.shape[0]
    ent = np.zeros(n)
    for lo in range(0, n, _ROW_SLAB):
        hi = min(lo + _ROW_SLAB, n)
        z = lm_head_logits(hidden[lo:hi], w, inv_temperature)
        mx = z.max(axis=1, keepdims=True)
        lse = mx + np.log(np.exp(z - mx).sum(axis=1, keepdims=True))
        logp_all = z - lse
        ent[lo:hi] = -(np.exp(logp_all) * logp_all).sum(axis=1)
    return ent


def token_logprobs_bwd(hidden, w, targets, grad_logp, inv_temperature=1.0):
    """Gradients of sum_t grad_logp[t] * logp[t] w.r.t. hidden and W.

    dz[t, v] = grad_logp[t] * (1[v == y_t] - softmax(z[t])[v]) * inv_T
    grad_hidden[t, :] = sum_v dz[t, v] * W[v, :]
    grad_w[v, :]      = sum_t dz[t, v] * hidden[t, :]
    Returns (grad_hidden [N,H], grad_w [V,H]) in float64.
    """
    hidden = _f64(hidden)
    w = _f64(w)
    g = _f64(grad_logp)
    targets = np.asarray(targets, dtype=np.int64)
    n, h = hidden.shape
    v = w.shape[0]
    grad_hidden = np.zeros((n, h))
    grad_w = np.zeros((v, h))
    for lo in range(0, n, _ROW_SLAB):
        hi = min(lo + _ROW_SLAB, n)
        z = lm_head_logits(hidden[lo:hi], w, inv_temperature)
        mx = z.max(axis=1, keepdims=True)
        lse = mx + np.log(np.exp(z - mx).sum(axis=1, keepdims=True))
        p = np.exp(z - lse)
        onehot_minus_p = -p
        onehot_minus_p[np.arange(hi - lo), targets[lo:hi]] += 1.0
        dz = g[lo:hi, None] * onehot_minus_p * float(inv_temperature)
        grad_hidden[lo:hi] = dz @ w
        grad_w += dz.T @ hidden[lo:hi]
    return grad_hidden, grad_w


# --------------------------------------------------------------------------------------
# A-3PO decoupled loss  (Eq. 2, Eq. 3, Eq. 4; Listing 1 for the d < 1 convention)
# --------------------------------------------------------------------------------------
def expand_per_sequence(values_per_seq, cu_seqlens, n):
    """Broadcast one value per sequence to every token of a packed batch (cu_seqlens [B+1])."""
    values_per_seq = np.asarray(values_per_seq)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    out = np.zeros(n, dtype=values_per_seq.dtype)
    for b in range(len(cu) - 1):
        out[cu[b]:cu[b + 1]] = values_per_seq[b]
    return out


def staleness(versions, current_version):
    """d = v(pi_theta) - v(pi_behav), an integer per token (Eq. 4)."""
    return np.int64(current_version) - np.asarray(versions, dtype=np.int64)


def staleness_alpha(versions, current_version):
    """alpha = 1/d for d >= 1, else 1 (Eq. 4; d < 0 follows Listing 1's `where`: alpha = 1)."""
    d = staleness(versions, current_version)
    safe_d = np.where(d >= 1, d, 1).astype(np.float64)
    return np.where(d >= 1, 1.0 / safe_d, 1.0)


def prox_logp(logp, behav_logp, alpha):
    """log pi_prox = alpha * log pi_behav + (1 - alpha) * log pi_theta (Eq. 3), literally."""
    return alpha * _f64(behav_logp) + (1.0 - alpha) * _f64(logp)


def loss_terms(logp, behav_logp, versions, current_version, adv, mask, clip_eps):
    """Every per-token quantity of Eq. 2 with the interpolated anchor of Eq. 3-4.

    Returns a dict of float64 arrays [N]: alpha, l_prox, iw, r, s1 (= r*A), s2 (= clip(r)*A),
    obj (= iw * min(s1, s2)), act (1 where the unclipped branch is the minimum, ties included),
    margin (distance of r to the nearer clip bound), valid (mask != 0).
    Masked-out tokens have their inputs replaced by harmless values first, so garbage / NaN
    under the mask never propagates (select semantics).
    """
    valid = np.asarray(mask) != 0
    l_theta = np.where(valid, _f64(logp), 0.0)
    l_behav = np.where(valid, _f64(behav_logp), 0.0)
    a = np.where(valid, _f64(adv), 0.0)
    eps = np.float64(np.float32(clip_eps))
    alpha = staleness_alpha(versions, current_version)
    l_prox = prox_logp(l_theta, l_behav, alpha)
    iw = np.exp(l_prox - l_behav)          # pi_prox / pi_behav  (importance weight)
    r = np.exp(l_theta - l_prox)           # pi_theta / pi_prox  (trust-region ratio)
    s1 = r * a
    s2 = np.minimum(np.maximum(r, 1.0 - eps), 1.0 + eps) * a
    obj = iw * np.minimum(s1, s2)
    act = (s1 <= s2)
    margin = np.minimum(np.abs(r - (1.0 - eps)), np.abs(r - (1.0 + eps)))
    return dict(alpha=alpha, l_prox=l_prox, iw=iw, r=r, s1=s1, s2=s2, obj=obj, act=act,
                margin=margin, valid=valid, adv=a)


def loss_fwd(logp, behav_logp, versions, current_version, adv, mask, clip_eps):
    """L = -(sum_t m_t * obj_t) / max(M, 1), M = sum_t m_t  (Eq. 2's E_t as a masked token mean).

    Returns (loss, stats) with stats = dict(n_valid, n_clipped, iw_max, iw_min, abs_obj_mean).
    n_clipped counts valid tokens whose clipped term is the strict minimum (zero gradient).
    iw_max / iw_min are over valid tokens (0 when there are none).
    """
    t = loss_terms(logp, behav_logp, versions, current_version, adv, mask, clip_eps)
    valid = t["valid"]
    m = int(valid.sum())
    total = float(np.sum(np.where(valid, t["obj"], 0.0)))
    loss = -total / max(m, 1)
    stats = dict(
        n_valid=m,
        n_clipped=int(np.sum(valid & ~t["act"])),
        iw_max=float(t["iw"][valid].max()) if m else 0.0,
        iw_min=float(t["iw"][valid].min()) if m else 0.0,
        abs_obj_mean=float(np.sum(np.where(valid, np.abs(t["obj"]), 0.0))) / max(m, 1),
    )
    return loss, stats


def loss_bwd(logp, behav_logp, versions, current_version, adv, mask, clip_eps,
             detach_prox=True, grad_loss=1.0):
    """g_t = dL/d l_theta_t.

    detach_prox=True (the anchor is a constant, as the recomputed anchor of Sec. 2.2 is):
        g_t = -(grad_loss * m_t / M) * iw * A * r * act
    detach_prox=False (differentiate through Eq. 3 as well):
        g_t = -(grad_loss * m_t / M) * ((1 - alpha) * obj + alpha * iw * A * r * act)
    """
    t = loss_terms(logp, behav_logp, versions, current_version, adv, mask, clip_eps)
    valid = t["valid"]
    m = int(valid.sum())
    if m == 0:
        return np.zeros(valid.shape[0])
    through_ratio = t["iw"] * t["adv"] * t["r"] * t["act"]
    if detach_prox:
        dobj = through_ratio
    else:
        dobj = (1.0 - t["alpha"]) * t["obj"] + t["alpha"] * through_ratio
    return np.where(valid, -(float(grad_loss) / m) * dobj, 0.0)


def decoupled_loss(logp, behav_logp, prox_logp, adv, mask, clip_eps, grad_loss=1.0):
    """Eq. 2 with an explicit, frozen proximal policy (the "recompute" baseline of Sec. 2.2).

    iw = exp(l_prox - l_behav), r = exp(l_theta - l_prox), obj = iw * min(r A, clip(r) A),
    L = -sum m obj / max(M, 1);  dL/dl_theta = -(grad_loss m / M) iw A r act  (anchor constant).
    Returns (loss, stats, grad_logp, terms).
    """
    valid = np.asarray(mask) != 0
    l_theta = np.where(valid, _f64(logp), 0.0)
    l_behav = np.where(valid, _f64(behav_logp), 0.0)
    l_prox = np.where(valid, _f64(prox_logp), 0.0)
    a = np.where(valid, _f64(adv), 0.0)
    eps = np.float64(np.float32(clip_eps))
    iw = np.exp(l_prox - l_behav)
    r = np.exp(l_theta - l_prox)
    s1 = r * a
    s2 = np.minimum(np.maximum(r, 1.0 - eps), 1.0 + eps) * a
    obj = iw * np.minimum(s1, s2)
    act = s1 <= s2
    m = int(valid.sum())
    loss = -float(np.sum(np.where(valid, obj, 0.0))) / max(m, 1)
    stats = dict(
        n_valid=m,
        n_clipped=int(np.sum(valid & ~act)),
        iw_max=float(iw[valid].max()) if m else 0.0,
        iw_min=float(iw[valid].min()) if m else 0.0,
        abs_obj_mean=float(np.sum(np.where(valid, np.abs(obj), 0.0))) / max(m, 1),
    )
    grad = np.where(valid, -(float(grad_loss) / max(m, 1)) * iw * a * r * act, 0.0)
    margin = np.minimum(np.abs(r - (1.0 - eps)), np.abs(r - (1.0 + eps)))
    return loss, stats, grad, dict(r=r, iw=iw, act=act, margin=margin, valid=valid)


# --------------------------------------------------------------------------------------
# GRPO advantages (Sec. 4.1 "group reward normalization"; the paper gives no formula, the
# usual one is taken: population standard deviation, 1e-6 added to the denominator)
# --------------------------------------------------------------------------------------
def grpo_advantages(rewards, group_size, norm_eps=1e-6):
    """A_i = (R_i - mean_group) / (std_group + norm_eps), one value per sequence."""
    r = _f64(rewards).reshape(-1, group_size)
    mean = r.mean(axis=1, keepdims=True)
    std = np.sqrt(((r - mean) ** 2).mean(axis=1, keepdims=True))
    return ((r - mean) / (std + norm_eps)).reshape(-1)
