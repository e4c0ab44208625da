"""GPU parity: lte_sparsity_stats (Eq. 7 penalty value and the retention counts Algorithm 1 steers) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,T,tau,with_lam", [(3, 5, 1000, 0.5, True), (1, 2, 37, 0.5, False), (8, 16, 2048, 0.7, True), (2, 3, 4099, 0.3, True)])
def test_stats_match_oracle(B, H, T, tau, with_lam):
    rng = np.random.default_rng(B * 100 + H)
    z = (rng.standard_normal((B, H, T)) * 1.5).astype(np.float32)
    z[:, :, -3:] = -np.inf                                                 # the unscored tail
    z[np.abs(z - orc.logit(tau)) < 1e-4] += 1e-3                           # keep clear of the threshold (fp32 vs fp64 compare)
    lam = rng.uniform(0, 1, H).astype(np.float32) if with_lam else None
    s = lte.shape(B, H, T, 64, 16, 8, lte.BF16, tau=tau)
    count, pen = lte.lte_sparsity_stats(s, torch.from_numpy(z).cuda(), None if lam is None else torch.from_numpy(lam).cuda())
    torch.cuda.synchronize()
    c64, p64 = orc.sparsity_stats(z, lam, tau)
    np.testing.assert_allclose(count.cpu().numpy(), c64, rtol=1e-6)
    assert abs(float(pen.cpu()) - p64) <= 1e-4 * max(1.0, abs(p64))
    # twice the same bits: fixed summation order
    count2, pen2 = lte.lte_sparsity_stats(s, torch.from_numpy(z).cuda(), None if lam is None else torch.from_numpy(lam).cuda())
    assert torch.equal(count, count2) and torch.equal(pen, pen2)
