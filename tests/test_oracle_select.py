"""Pins for the oracle's one-shot selection (Eq. 5 + capped capacity) and its streaming twin."""
import os

import numpy as np
import pytest

from oracle import lte_oracle as orc
from tests.bruteforce import topr_bruteforce

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _sel1(z, W, R, sink=0, tau=0.5):
    idx, cnt, nc = orc.select(np.asarray(z, float)[None, None], W, R, sink, tau)
    return list(idx[0, 0, :cnt[0, 0]]), int(cnt[0, 0]), int(nc[0, 0]), idx[0, 0]


def test_hand_made_orders():
    T, W, R = 20, 4, 3
    inc = np.arange(1, T + 1, dtype=float)
    assert _sel1(inc, W, R)[0] == [13, 14, 15]            # last R eligible (j <= T-1-W = 15)
    assert _sel1(-inc + 100, W, R)[0] == [0, 1, 2]         # decreasing: first R
    assert _sel1(np.ones(T), W, R)[0] == [0, 1, 2]         # ties -> older token wins
    got, cnt, nc, raw = _sel1(-np.ones(T), W, R)
    assert got == [] and cnt == 0 and nc == 0 and list(raw) == [-1, -1, -1]
    assert _sel1(np.zeros(T), W, R)[1] == 0                # threshold is strict: r = 0.5 is dropped


def test_sink_ranks_first_and_counts_against_budget():
    T, W = 16, 4
    z = np.full(T, -3.0); z[5] = 9.0; z[7] = 8.0; z[9] = 7.0
    assert _sel1(z, W, 4, sink=2)[0] == [0, 1, 5, 7]
    assert _sel1(z, W, 2, sink=2)[0] == [0, 1]
    assert _sel1(z, W, 1, sink=2)[0] == [0]
    assert _sel1(z, W, 8, sink=2)[0] == [0, 1, 5, 7, 9]


def test_short_prompt_has_no_candidates():
    assert _sel1(np.ones(5), 8, 4)[1] == 0
    assert _sel1(np.ones(8), 8, 4)[1] == 0
    assert _sel1(np.ones(9), 8, 4)[0] == [0]


def test_worked_example_fixture():
    # tests/golden/select_worked_example.txt: a case small enough to rank by hand.
    lines = [l for l in open(os.path.join(GOLD, "select_worked_example.txt")) if not l.startswith("#")]
    kv = dict(l.strip().split("=", 1) for l in lines if "=" in l)
    z = [float(x) for x in kv["z"].split()]
    want = [int(x) for x in kv["idx"].split()]
    got, cnt, nc, _ = _sel1(z, int(kv["W"]), int(kv["R"]), int(kv["sink"]))
    assert got == want and nc == int(kv["ncand"])


@pytest.mark.parametrize("seed", range(6))
def test_bruteforce_random_with_ties(seed):
    rng = np.random.default_rng(seed)
    B, H, T = 2, 3, 50
    W, R, sink = int(rng.integers(1, 12)), int(rng.integers(0, 10)), int(rng.integers(0, 4))
    z = np.round(rng.standard_normal((B, H, T)) * 2) / 2          # many exact ties
    idx, cnt, nc = orc.select(z, W, R, sink, 0.5)
    for b in range(B):
        for h in range(H):
            want, n = topr_bruteforce(z[b, h], W, R, sink, 0.0)
            assert list(idx[b, h, :cnt[b, h]]) == want and nc[b, h] == n
            assert np.all(idx[b, h, cnt[b, h]:] == -1)
            assert cnt[b, h] <= R and all(j <= T - 1 - W for j in want)


@pytest.mark.parametrize("seed", range(6))
def test_streaming_pool_equals_one_shot(seed):
    # Section 3.1.3 describes the capped pool twice (top-b at prefill; replace-the-lowest while
    # decoding): with one total order both must end with the same pool.
    rng = np.random.default_rng(100 + seed)
    B, H, T, d = 1, 4, 70, 2
    W, R, sink = int(rng.integers(3, 10)), int(rng.integers(1, 9)), int(rng.integers(0, 3))
    z = np.round(rng.standard_normal((B, H, T)) * 3) / 3
    z[:, :, T - 2:] = -np.inf
    x = rng.standard_normal((B, H, T, d))
    _, _, pidx, pcnt = orc.stream(x, x, x, z, W, R, sink)
    idx, cnt, _ = orc.select(z, W, R, sink)
    assert np.array_equal(pidx, idx) and np.array_equal(pcnt, cnt)
