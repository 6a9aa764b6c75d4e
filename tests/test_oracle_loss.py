"""Pins for the oracle's A-3PO loss forward/backward (CPU only).

The paper fixes: Eq. 4's d -> alpha table, the sandwich property, the closed form r = w^alpha,
the contraction |w^alpha - 1| <= |w - 1|, the limit r -> 1 for large staleness, and that d = 0
recovers coupled PPO (Eq. 1).  The tests also use closed forms (behaviour == current), a
hand-derived example (tests/golden) and central finite differences.
"""
import math
import os

import numpy as np
import pytest

from oracle import a3po_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "a3po_hand_example.txt")


def _batch(n, seed, max_d=6, noise=0.3):
    rng = np.random.default_rng(seed)
    logp = -rng.standard_exponential(n)
    behav = np.minimum(logp + noise * rng.standard_normal(n), 0.0)
    cur = 20
    versions = cur - rng.integers(0, max_d + 1, size=n)
    adv = rng.standard_normal(n)
    mask = (rng.random(n) < 0.85).astype(np.uint8)
    return logp, behav, versions, cur, adv, mask


def test_alpha_table():
    cur = 1_000_010
    d = np.array([-3, 0, 1, 2, 4, 1_000_000])
    alpha = orc.staleness_alpha(cur - d, cur)
    np.testing.assert_array_equal(alpha, [1.0, 1.0, 1.0, 0.5, 0.25, 1e-6])
    np.testing.assert_array_equal(orc.staleness(cur - d, cur), d)


def test_sandwich_property():
    logp, behav, versions, cur, adv, mask = _batch(4000, 1, max_d=12, noise=2.0)
    t = orc.loss_terms(logp, behav, versions, cur, adv, np.ones_like(mask), 0.2)
    lo = np.minimum(logp, behav)
    hi = np.maximum(logp, behav)
    assert np.all(t["l_prox"] >= lo - 1e-15) and np.all(t["l_prox"] <= hi + 1e-15)


def test_fresh_samples_anchor_on_behaviour():
    """d = 0 and d = 1 both give alpha = 1: the anchor is exactly the behaviour policy."""
    logp, behav, _, cur, adv, mask = _batch(500, 2)
    for d in (0, 1):
        t = orc.loss_terms(logp, behav, np.full(500, cur - d), cur, adv, np.ones(500), 0.2)
        np.testing.assert_array_equal(t["l_prox"], behav)
        np.testing.assert_array_equal(t["iw"], 1.0)


def test_closed_form_ratio_and_contraction():
    logp, behav, versions, cur, adv, mask = _batch(3000, 3, max_d=9, noise=1.0)
    ones = np.ones(3000)
    t = orc.loss_terms(logp, behav, versions, cur, adv, ones, 0.2)
    delta = logp - behav
    w = np.exp(delta)
    np.testing.assert_allclose(t["r"], w ** t["alpha"], rtol=1e-13)
    np.testing.assert_allclose(t["iw"], np.exp((1 - t["alpha"]) * delta), rtol=1e-13)
    np.testing.assert_allclose(t["iw"] * t["r"], w, rtol=1e-13)
    assert np.all(np.abs(t["r"] - 1) <= np.abs(w - 1) + 1e-15)


def test_large_staleness_limit():
    logp, behav, _, _, adv, _ = _batch(200, 4, noise=1.0)
    cur = 2_000_000
    t = orc.loss_terms(logp, behav, np.full(200, cur - 1_000_000), cur, adv, np.ones(200), 0.2)
    np.testing.assert_allclose(t["r"], 1.0, atol=1e-5)
    np.testing.assert_allclose(t["obj"], np.exp(logp - behav) * adv, rtol=2e-5, atol=1e-12)


def _coupled_ppo_clip_loss(logp, old_logp, adv, mask, eps):
    """Eq. 1 written independently with scalar loops: -mean_t min(r A, clip(r) A)."""
    total, count = 0.0, 0
    for lt, lo, a, m in zip(logp, old_logp, adv, mask):
        if not m:
            continue
        r = math.exp(lt - lo)
        clipped = min(max(r, 1 - eps), 1 + eps)
        total += min(r * a, clipped * a)
        count += 1
    return -total / max(count, 1)


def test_zero_staleness_recovers_coupled_ppo():
    logp, behav, _, cur, adv, mask = _batch(2000, 5, noise=0.4)
    eps32 = float(np.float32(0.2))
    loss, stats = orc.loss_fwd(logp, behav, np.full(2000, cur), cur, adv, mask, 0.2)
    assert loss == pytest.approx(_coupled_ppo_clip_loss(logp, behav, adv, mask, eps32), rel=1e-13)
    assert stats["n_valid"] == int(mask.sum())


def test_on_policy_closed_form():
    """behaviour == current: every ratio is 1, L = -sum(m A)/M and g_t = -m_t A_t / M."""
    logp, _, versions, cur, adv, mask = _batch(777, 6)
    loss, stats = orc.loss_fwd(logp, logp, versions, cur, adv, mask, 0.2)
    m = mask.sum()
    assert loss == pytest.approx(-(adv * mask).sum() / m, rel=1e-14)
    assert stats["n_clipped"] == 0
    # Eq. 3 is evaluated literally (alpha*l + (1-alpha)*l), which rounds: 1e-14, not exact
    assert stats["iw_max"] == pytest.approx(1.0, abs=1e-14) and stats["iw_min"] == pytest.approx(1.0, abs=1e-14)
    for detach in (True, False):
        g = orc.loss_bwd(logp, logp, versions, cur, adv, mask, 0.2, detach_prox=detach)
        np.testing.assert_allclose(g, -(mask * adv) / m, rtol=1e-14)


def test_hand_example_from_golden_file():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for row in rows:
        p_theta, p_behav, d, eps, adv, alpha, iw, r, obj, clipped, g_det, g_thr = map(float, row)
        args = (np.array([math.log(p_theta)]), np.array([math.log(p_behav)]),
                np.array([10 - int(d)]), 10, np.array([adv]), np.array([1]), eps)
        t = orc.loss_terms(*args)
        loss, stats = orc.loss_fwd(*args)
        # eps crosses the ABI as fp32 (0.2f = 0.2 + 3e-9), hence 1e-8 not 1e-15
        assert t["alpha"][0] == alpha
        assert t["iw"][0] == pytest.approx(iw, rel=1e-14)
        assert t["r"][0] == pytest.approx(r, rel=1e-14)
        assert t["obj"][0] == pytest.approx(obj, rel=1e-8)
        assert loss == pytest.approx(-obj, rel=1e-8)
        assert stats["n_clipped"] == int(clipped)
        assert orc.loss_bwd(*args, detach_prox=True)[0] == pytest.approx(g_det, rel=1e-8, abs=1e-15)
        assert orc.loss_bwd(*args, detach_prox=False)[0] == pytest.approx(g_thr, rel=1e-8)


def test_clipped_count_brute_force():
    logp, behav, versions, cur, adv, mask = _batch(1500, 7, noise=0.6)
    _, stats = orc.loss_fwd(logp, behav, versions, cur, adv, mask, 0.2)
    eps = float(np.float32(0.2))
    count = 0
    iw_all = []
    for lt, lb, ver, a, m in zip(logp, behav, versions, adv, mask):
        if not m:
            continue
        d = cur - ver
        alpha = 1.0 / d if d >= 1 else 1.0
        r = math.exp(alpha * (lt - lb))          # closed form, Theorem item 2
        iw_all.append(math.exp((1 - alpha) * (lt - lb)))
        if (r > 1 + eps and a > 0) or (r < 1 - eps and a < 0):
            count += 1
    assert 0 < count < mask.sum()
    assert stats["n_clipped"] == count
    assert stats["iw_max"] == pytest.approx(max(iw_all), rel=1e-13)
    assert stats["iw_min"] == pytest.approx(min(iw_all), rel=1e-13)


def test_masked_tokens_are_selected_out():
    logp, behav, versions, cur, adv, mask = _batch(300, 8)
    base_loss, base_stats = orc.loss_fwd(logp, behav, versions, cur, adv, mask, 0.2)
    base_g = orc.loss_bwd(logp, behav, versions, cur, adv, mask, 0.2)
    dirty = [x.copy() for x in (logp, behav, adv)]
    for arr in dirty:
        arr[mask == 0] = np.nan
    dirty[0][np.flatnonzero(mask == 0)[:2]] = np.inf
    loss, stats = orc.loss_fwd(dirty[0], dirty[1], versions, cur, dirty[2], mask, 0.2)
    assert loss == base_loss and stats == base_stats
    g = orc.loss_bwd(dirty[0], dirty[1], versions, cur, dirty[2], mask, 0.2)
    np.testing.assert_array_equal(g, base_g)
    assert np.all(g[mask == 0] == 0.0)
    # removing the masked tokens altogether gives the same loss
    keep = mask == 1
    loss2, _ = orc.loss_fwd(logp[keep], behav[keep], versions[keep], cur, adv[keep], mask[keep], 0.2)
    assert loss2 == pytest.approx(base_loss, rel=1e-14)


def test_empty_and_fully_masked():
    z = np.zeros(0)
    loss, stats = orc.loss_fwd(z, z, z.astype(np.int32), 3, z, z.astype(np.uint8), 0.2)
    assert loss == 0.0 and stats["n_valid"] == 0 and stats["iw_max"] == 0.0
    logp, behav, versions, cur, adv, _ = _batch(10, 9)
    loss, stats = orc.loss_fwd(logp, behav, versions, cur, adv, np.zeros(10, np.uint8), 0.2)
    assert loss == 0.0 and stats["n_valid"] == 0
    assert np.all(orc.loss_bwd(logp, behav, versions, cur, adv, np.zeros(10, np.uint8), 0.2) == 0)


def _loss_with_frozen_anchor(logp, l_prox, behav, adv, mask, eps):
    """Eq. 2 with an explicit, constant anchor (scalar loops) — for the detach-reading FD."""
    total, count = 0.0, 0
    for lt, lp, lb, a, m in zip(logp, l_prox, behav, adv, mask):
        if not m:
            continue
        iw = math.exp(lp - lb)
        r = math.exp(lt - lp)
        total += iw * min(r * a, min(max(r, 1 - eps), 1 + eps) * a)
        count += 1
    return -total / max(count, 1)


@pytest.mark.parametrize("detach", [True, False])
def test_gradient_matches_finite_differences(detach):
    n = 40
    logp, behav, versions, cur, adv, mask = _batch(n, 10, noise=0.5)
    eps = float(np.float32(0.2))
    t = orc.loss_terms(logp, behav, versions, cur, adv, mask, 0.2)
    far = t["margin"] > 1e-3           # keep finite differences away from the clip kinks
    assert far.sum() > 30 and (~t["act"] & t["valid"]).any() and (t["act"] & t["valid"]).any()
    g = orc.loss_bwd(logp, behav, versions, cur, adv, mask, 0.2, detach_prox=detach, grad_loss=1.7)
    step = 1e-6
    for i in np.flatnonzero(far):
        lp_, lm_ = logp.copy(), logp.copy()
        lp_[i] += step
        lm_[i] -= step
        if detach:
            f_p = _loss_with_frozen_anchor(lp_, t["l_prox"], behav, adv, mask, eps)
            f_m = _loss_with_frozen_anchor(lm_, t["l_prox"], behav, adv, mask, eps)
        else:
            f_p, _ = orc.loss_fwd(lp_, behav, versions, cur, adv, mask, 0.2)
            f_m, _ = orc.loss_fwd(lm_, behav, versions, cur, adv, mask, 0.2)
        assert g[i] == pytest.approx(1.7 * (f_p - f_m) / (2 * step), abs=1e-8)


def test_frozen_anchor_formulation_agrees_on_forward():
    logp, behav, versions, cur, adv, mask = _batch(200, 11)
    t = orc.loss_terms(logp, behav, versions, cur, adv, mask, 0.2)
    loss, _ = orc.loss_fwd(logp, behav, versions, cur, adv, mask, 0.2)
    ref = _loss_with_frozen_anchor(logp, t["l_prox"], behav, adv, mask, float(np.float32(0.2)))
    assert loss == pytest.approx(ref, rel=1e-13)


def test_per_sequence_expansion():
    cu = np.array([0, 3, 3, 7])
    out = orc.expand_per_sequence(np.array([5, 6, 7], dtype=np.int32), cu, 7)
    np.testing.assert_array_equal(out, [5, 5, 5, 7, 7, 7, 7])


def test_grpo_advantages():
    adv = orc.grpo_advantages([1, 0, 0, 1, 1, 1, 1, 1], 4)
    np.testing.assert_allclose(adv[:4], np.array([1, -1, -1, 1]) / (1 + 2e-6) * 1.0, rtol=1e-5)
    np.testing.assert_array_equal(adv[4:], 0.0)
    assert abs(adv[:4].sum()) < 1e-12


# ---------------------------------------------------------------------------- explicit anchor (Eq. 2 as it stands)
def test_decoupled_loss_with_behaviour_anchor_is_coupled_ppo():
    """prox = behav turns Eq. 2 into Eq. 1 (independent scalar implementation above)."""
    logp, behav, _, _, adv, mask = _batch(1500, 21, noise=0.4)
    loss, stats, grad, _ = orc.decoupled_loss(logp, behav, behav, adv, mask, 0.2)
    assert loss == pytest.approx(_coupled_ppo_clip_loss(logp, behav, adv, mask, float(np.float32(0.2))), rel=1e-13)
    assert stats["iw_max"] == 1.0 and stats["iw_min"] == 1.0


def test_decoupled_loss_with_interpolated_anchor_is_a3po():
    """Feeding the anchor of Eq. 3-4 explicitly reproduces the A-3PO loss and its detached gradient."""
    logp, behav, versions, cur, adv, mask = _batch(1200, 22, noise=0.5)
    prox = orc.prox_logp(logp, behav, orc.staleness_alpha(versions, cur))
    loss, stats, grad, _ = orc.decoupled_loss(logp, behav, prox, adv, mask, 0.2, grad_loss=1.3)
    ref_loss, ref_stats = orc.loss_fwd(logp, behav, versions, cur, adv, mask, 0.2)
    assert loss == pytest.approx(ref_loss, rel=1e-13)
    assert stats["n_clipped"] == ref_stats["n_clipped"] and stats["n_valid"] == ref_stats["n_valid"]
    np.testing.assert_allclose(grad, orc.loss_bwd(logp, behav, versions, cur, adv, mask, 0.2, grad_loss=1.3),
                               rtol=1e-12, atol=1e-18)


def test_decoupled_loss_scalar_brute_force_and_finite_differences():
    n = 30
    rng = np.random.default_rng(23)
    logp = -rng.standard_exponential(n)
    behav = np.minimum(logp + 0.3 * rng.standard_normal(n), 0)
    prox = np.minimum(logp + 0.2 * rng.standard_normal(n), 0)
    adv = rng.standard_normal(n)
    mask = (rng.random(n) < 0.8).astype(np.uint8)
    eps = float(np.float32(0.2))
    loss, stats, grad, terms = orc.decoupled_loss(logp, behav, prox, adv, mask, 0.2)
    assert loss == pytest.approx(_loss_with_frozen_anchor(logp, prox, behav, adv, mask, eps), rel=1e-13)
    step = 1e-6
    for i in np.flatnonzero(terms["margin"] > 1e-3):
        lp_, lm_ = logp.copy(), logp.copy()
        lp_[i] += step
        lm_[i] -= step
        fd = (_loss_with_frozen_anchor(lp_, prox, behav, adv, mask, eps)
              - _loss_with_frozen_anchor(lm_, prox, behav, adv, mask, eps)) / (2 * step)
        assert grad[i] == pytest.approx(fd, abs=1e-8)
