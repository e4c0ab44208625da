"""Pins for the oracle's Eq. 7 statistics and the penalty-weight feedback loop (Algorithm 1)."""
import numpy as np

from oracle import lte_oracle as orc


def test_stats_closed_forms():
    # z = logit(r): r is known exactly; one head above the threshold everywhere, one below, one mixed
    r = np.array([[[0.9, 0.9, 0.9, 0.9], [0.1, 0.2, 0.3, 0.4], [0.75, 0.25, 0.5, 1.0 - 1e-12]]])
    z = np.log(r) - np.log1p(-r)
    count, pen = orc.sparsity_stats(z, lam=[1.0, 1.0, 1.0])
    np.testing.assert_array_equal(count, [4, 0, 2])                        # r = 0.5 is not above the threshold (strict)
    np.testing.assert_allclose(pen, 4 * 0.4 + 0.0 + 0.25 + 0.5, atol=1e-9)
    # the weights multiply per head; unscored positions (-inf) count for nothing; counts average over the batch
    z2 = np.concatenate([z, np.full_like(z, -np.inf)], axis=0)
    count2, pen2 = orc.sparsity_stats(z2, lam=[2.0, 5.0, 0.0])
    np.testing.assert_allclose(count2, [2, 0, 1])
    np.testing.assert_allclose(pen2, 2.0 * 1.6, atol=1e-9)


def test_moving_average_has_its_closed_form():
    # constant count c from cbar = 0: cbar_k = c (1 - (1 - a)^k), a = 2 / (1 + u / 2)
    u, c = 32, 700.0
    a = 2.0 / (1.0 + u / 2.0)
    lam, cbar = np.array([1e-9]), np.array([0.0])
    for k in range(1, 50):
        lam, cbar = orc.lambda_update(lam, cbar, np.array([c]), step=k, u=u)
        np.testing.assert_allclose(cbar, c * (1.0 - (1.0 - a) ** k), rtol=1e-12)


def test_feedback_directions_clamp_floor_and_re_enable():
    u = 4
    # a head far above the cap: every u-th step multiplies by alpha, up to the clamp at 1
    lam, cbar = np.array([0.5]), np.array([1000.0])
    seen = []
    for step in range(1, 13):
        lam, cbar = orc.lambda_update(lam, cbar, np.array([1000.0]), step, u=u, cap=512, alpha=1.5)
        seen.append(lam[0])
    assert seen[:3] == [0.5, 0.5, 0.5] and seen[3] == 0.75 and seen[7] == 1.0 and seen[11] == 1.0
    # a head below the band: divided by alpha; once below the floor it is switched off, and stays off inside the band
    lam, cbar = np.array([2e-9]), np.array([100.0])
    lam, cbar = orc.lambda_update(lam, cbar, np.array([100.0]), 4, u=u, cap=512, alpha=1.5)
    np.testing.assert_allclose(lam, [2e-9 / 1.5])
    lam, cbar = orc.lambda_update(lam, cbar, np.array([100.0]), 8, u=u, cap=512, alpha=1.5)
    assert lam[0] == 0.0
    lam, cbar = orc.lambda_update(lam, np.array([500.0]), np.array([500.0]), 12, u=u, cap=512, alpha=1.5)
    assert lam[0] == 0.0                                                   # between 0.95 cap and cap: unchanged
    # above the cap with the weight at zero: re-enabled at the floor
    lam, cbar = orc.lambda_update(lam, np.array([600.0]), np.array([600.0]), 16, u=u, cap=512, alpha=1.5)
    assert lam[0] == 1e-9
    # not a multiple of u: only the average moves
    lam2, cbar2 = orc.lambda_update(np.array([0.3]), np.array([900.0]), np.array([900.0]), 17, u=u, cap=512, alpha=1.5)
    assert lam2[0] == 0.3
