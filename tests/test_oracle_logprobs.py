"""Pins for the oracle's LM-head log-prob forward/backward (CPU only).

Each test compares the oracle with something that is not the oracle: a normalisation identity,
a closed form, scalar brute force written from the textbook softmax, scipy's logsumexp, or
central finite differences.
"""
import math

import numpy as np
import pytest
from scipy.special import logsumexp

from oracle import a3po_oracle as orc


def _problem(n, h, v, seed):
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((n, h))
    w = rng.standard_normal((v, h)) / math.sqrt(h)
    targets = rng.integers(0, v, size=n)
    return hidden, w, targets


def test_softmax_normalisation():
    hidden, w, _ = _problem(6, 8, 23, 1)
    total = np.zeros(6)
    for y in range(23):
        logp, _ = orc.token_logprobs_fwd(hidden, w, np.full(6, y))
        assert np.all(logp <= 0.0)
        total += np.exp(logp)
    np.testing.assert_allclose(total, 1.0, rtol=0, atol=1e-12)


def test_zero_weights_give_uniform():
    hidden, _, targets = _problem(5, 8, 37, 2)
    logp, lse = orc.token_logprobs_fwd(hidden, np.zeros((37, 8)), targets)
    np.testing.assert_allclose(logp, -math.log(37), rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse, math.log(37), rtol=0, atol=1e-15)


def test_brute_force_scalar_softmax():
    """Textbook p_v = e^{z_v} / sum e^{z_u} with scalar loops (no max subtraction), non-square
    H != V so a transposed operand cannot pass."""
    n, h, v = 3, 4, 7
    hidden, w, targets = _problem(n, h, v, 3)
    inv_t = 0.7
    logp, lse = orc.token_logprobs_fwd(hidden, w, targets, inv_temperature=inv_t)
    for t in range(n):
        z = [inv_t * sum(hidden[t, k] * w[u, k] for k in range(h)) for u in range(v)]
        denom = sum(math.exp(zu) for zu in z)
        assert logp[t] == pytest.approx(math.log(math.exp(z[targets[t]]) / denom), abs=1e-13)
        assert lse[t] == pytest.approx(math.log(denom), abs=1e-13)


def test_matches_scipy_logsumexp_with_large_logits():
    """Library routine as the pin, at logit magnitudes where a naive exp would overflow."""
    hidden, w, targets = _problem(9, 16, 41, 4)
    hidden *= 300.0
    z = hidden @ w.T
    assert np.abs(z).max() > 800
    logp, lse = orc.token_logprobs_fwd(hidden, w, targets)
    np.testing.assert_allclose(lse, logsumexp(z, axis=1), rtol=1e-14)
    np.testing.assert_allclose(logp, z[np.arange(9), targets] - logsumexp(z, axis=1), rtol=1e-12, atol=1e-10)


def test_shift_and_permutation_invariance():
    n, h, v = 7, 8, 19
    hidden, w, targets = _problem(n, h, v, 5)
    base, _ = orc.token_logprobs_fwd(hidden, w, targets)
    # adding the same vector u to every row of W adds hidden.u to every logit of a row
    u = np.random.default_rng(6).standard_normal(h)
    shifted, _ = orc.token_logprobs_fwd(hidden, w + u[None, :], targets)
    np.testing.assert_allclose(shifted, base, atol=1e-12)
    # relabelling the vocabulary
    perm = np.random.default_rng(7).permutation(v)
    inv = np.empty(v, dtype=np.int64)
    inv[perm] = np.arange(v)
    permuted, _ = orc.token_logprobs_fwd(hidden, w[perm], inv[targets])
    np.testing.assert_allclose(permuted, base, atol=1e-13)


def test_temperature_is_a_logit_scale():
    hidden, w, targets = _problem(5, 8, 13, 8)
    a, _ = orc.token_logprobs_fwd(hidden, w, targets, inv_temperature=0.5)
    b, _ = orc.token_logprobs_fwd(hidden * 0.5, w, targets, inv_temperature=1.0)
    np.testing.assert_allclose(a, b, atol=1e-13)


def test_row_mask_and_slabs():
    # more rows than one slab; masked rows report zeros, others are unaffected
    n = orc._ROW_SLAB + 37
    hidden, w, targets = _problem(n, 4, 11, 9)
    mask = (np.arange(n) % 3 != 0).astype(np.uint8)
    logp, lse = orc.token_logprobs_fwd(hidden, w, targets, row_mask=mask)
    full, full_lse = orc.token_logprobs_fwd(hidden, w, targets)
    assert np.all(logp[mask == 0] == 0) and np.all(lse[mask == 0] == 0)
    np.testing.assert_array_equal(logp[mask == 1], full[mask == 1])
    z = hidden @ w.T
    np.testing.assert_allclose(full_lse, logsumexp(z, axis=1), rtol=1e-14)


def test_out_of_range_target_rejected():
    hidden, w, targets = _problem(3, 4, 5, 10)
    targets[1] = 5
    with pytest.raises(ValueError):
        orc.token_logprobs_fwd(hidden, w, targets)


def test_entropy_pins():
    hidden, w, _ = _problem(4, 8, 29, 11)
    ent = orc.token_entropy(hidden, np.zeros_like(w))
    np.testing.assert_allclose(ent, math.log(29), atol=1e-13)
    ent = orc.token_entropy(hidden, w, inv_temperature=1.3)
    for t in range(4):
        z = 1.3 * (w @ hidden[t])
        p = np.exp(z) / np.exp(z).sum()
        assert ent[t] == pytest.approx(-(p * np.log(p)).sum(), abs=1e-13)


# ---------------------------------------------------------------------------- backward
def _scalar_objective(hidden, w, targets, coeff, inv_t):
    logp, _ = orc.token_logprobs_fwd(hidden, w, targets, inv_temperature=inv_t)
    return float(np.dot(coeff, logp))


@pytest.mark.parametrize("peaked", [False, True])
def test_backward_matches_finite_differences(peaked):
    n, h, v = 5, 8, 17
    hidden, w, targets = _problem(n, h, v, 12)
    if peaked:
        # confident rows: the target's weight row is moved along the row's hidden state until the target holds
        # most of the probability mass (p_y up to 0.999), where dz at the target, g (1 - p_y), is a cancellation
        targets = np.arange(n) * 3 % v
        for t, lift in enumerate([4.0, 6.0, 8.0, 10.0, 12.0]):
            w[targets[t]] += lift * hidden[t] / np.dot(hidden[t], hidden[t])
        p_y = np.exp(orc.token_logprobs_fwd(hidden, w, targets, inv_temperature=0.8)[0])
        assert p_y.max() > 0.99 and np.median(p_y) > 0.5
    coeff = np.random.default_rng(13).standard_normal(n)
    inv_t = 0.8
    gh, gw = orc.token_logprobs_bwd(hidden, w, targets, coeff, inv_temperature=inv_t)
    step = 1e-6
    fd_h = np.zeros_like(hidden)
    for idx in np.ndindex(*hidden.shape):
        hp = hidden.copy(); hp[idx] += step
        hm = hidden.copy(); hm[idx] -= step
        fd_h[idx] = (_scalar_objective(hp, w, targets, coeff, inv_t)
                     - _scalar_objective(hm, w, targets, coeff, inv_t)) / (2 * step)
    fd_w = np.zeros_like(w)
    for idx in np.ndindex(*w.shape):
        wp = w.copy(); wp[idx] += step
        wm = w.copy(); wm[idx] -= step
        fd_w[idx] = (_scalar_objective(hidden, wp, targets, coeff, inv_t)
                     - _scalar_objective(hidden, wm, targets, coeff, inv_t)) / (2 * step)
    np.testing.assert_allclose(gh, fd_h, atol=2e-8)
    np.testing.assert_allclose(gw, fd_w, atol=2e-8)


def test_backward_structure():
    n, h, v = 6, 5, 13
    hidden, w, targets = _problem(n, h, v, 14)
    g = np.random.default_rng(15).standard_normal(n)
    gh, gw = orc.token_logprobs_bwd(hidden, w, targets, g)
    # each row of dz sums to zero, hence the vocab-sum of grad_w vanishes
    np.testing.assert_allclose(gw.sum(axis=0), 0.0, atol=1e-13)
    # linear in the upstream gradient
    gh2, gw2 = orc.token_logprobs_bwd(hidden, w, targets, -2.5 * g)
    np.testing.assert_allclose(gh2, -2.5 * gh, atol=1e-13)
    np.testing.assert_allclose(gw2, -2.5 * gw, atol=1e-13)
    # rows with zero upstream gradient get zero grad_hidden and do not touch grad_w
    g0 = g.copy(); g0[2] = 0.0
    gh0, gw0 = orc.token_logprobs_bwd(hidden, w, targets, g0)
    assert np.all(gh0[2] == 0.0)
    keep = np.arange(n) != 2
    _, gw_sub = orc.token_logprobs_bwd(hidden[keep], w, targets[keep], g[keep])
    np.testing.assert_allclose(gw0, gw_sub, atol=1e-13)
    # slab additivity (more rows than one slab)
    n_big = orc._ROW_SLAB + 9
    hidden, w, targets = _problem(n_big, 4, 7, 16)
    g = np.random.default_rng(17).standard_normal(n_big)
    _, gw_all = orc.token_logprobs_bwd(hidden, w, targets, g)
    _, gw_a = orc.token_logprobs_bwd(hidden[:100], w, targets[:100], g[:100])
    _, gw_b = orc.token_logprobs_bwd(hidden[100:], w, targets[100:], g[100:])
    np.testing.assert_allclose(gw_all, gw_a + gw_b, atol=1e-12)
