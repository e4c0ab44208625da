"""Pins for the oracle's prefill attention and streaming decode (Section 3.1.3)."""
import os

import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import synth
from tests.bruteforce import dense_attention, dense_mask

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _case(seed, B=2, H=2, T=40, d=8, W=6, R=5, K=5, sink=0):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, T, d)) for _ in range(3))
    w = rng.standard_normal((H, K, 2 * d)) * 0.2
    z = orc.scores(k, v, w)
    idx, cnt, _ = orc.select(z, W, R, sink)
    return q, k, v, w, z, idx, cnt


@pytest.mark.parametrize("seed,W,R,sink", [(0, 6, 5, 0), (1, 1, 3, 0), (2, 9, 40, 2), (3, 4, 0, 0), (4, 64, 4, 0)])
def test_dense_bruteforce(seed, W, R, sink):
    q, k, v, w, z, idx, cnt = _case(seed, W=W, R=R, sink=sink)
    B, H, T, d = q.shape
    scale = 0.37
    o, lse = orc.attn_prefill(q, k, v, idx, cnt, W, scale)
    for b in range(B):
        for h in range(H):
            M = dense_mask(T, W, idx[b, h, :cnt[b, h]])
            oref, lref, _ = dense_attention(q[b, h], k[b, h], v[b, h], M, scale)
            np.testing.assert_allclose(o[b, h], oref, atol=1e-12)
            np.testing.assert_allclose(lse[b, h], lref, atol=1e-12)


def test_config1_every_output_against_dense_bruteforce():
    cfg = synth.CONFIGS["C1"]
    x = synth.make(cfg, seed=0)
    z = orc.scores(x["k"], x["v"], x["w"])
    idx, cnt, ncand = orc.select(z, cfg.W, cfg.R)
    assert np.all(cnt <= cfg.R) and np.all(ncand >= cnt)
    o, lse = orc.attn_prefill(x["q"], x["k"], x["v"], idx, cnt, cfg.W)
    scale = 1.0 / np.sqrt(cfg.d)
    for h in range(cfg.H):
        M = dense_mask(cfg.T, cfg.W, idx[0, h, :cnt[0, h]])
        oref, lref, _ = dense_attention(*(x[t][0, h].astype(np.float64) for t in "qkv"), M, scale)
        np.testing.assert_allclose(o[0, h], oref, atol=1e-12)
        np.testing.assert_allclose(lse[0, h], lref, atol=1e-12)


def test_budget_zero_is_sliding_window_and_wide_window_is_causal():
    q, k, v, w, z, idx, cnt = _case(5, T=48, W=7, R=0)
    B, H, T, d = q.shape
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    i = torch.arange(T)[:, None]; j = torch.arange(T)[None, :]
    band = (j <= i) & (j > i - 7)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=band)
    o, _ = orc.attn_prefill(q, k, v, idx, cnt, 7)
    np.testing.assert_allclose(o, ref.numpy(), atol=1e-10)
    # W >= T: full causal attention whatever the retained list says
    idx2, cnt2, _ = orc.select(z, T, 4)
    assert np.all(cnt2 == 0)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    o, lse = orc.attn_prefill(q, k, v, idx2, cnt2, T)
    np.testing.assert_allclose(o, ref.numpy(), atol=1e-10)
    s = torch.einsum("bhid,bhjd->bhij", tq, tk) / np.sqrt(d)
    s = s.masked_fill(j > i, -np.inf)
    np.testing.assert_allclose(lse, torch.logsumexp(s, -1).numpy(), atol=1e-10)


def test_threshold_off_and_large_budget_is_full_causal():
    # With the threshold disabled every scored out-of-window token is retained, so R >= T gives
    # dense causal attention for every query whose far keys are all scored.
    q, k, v, w, z, _, _ = _case(6, T=32, W=5, R=0, K=1)     # K = 1: every position has a score
    idx, cnt, _ = orc.select(z, 5, 32, 0, tau=0.0)
    assert np.all(cnt == 32 - 5)
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    o, _ = orc.attn_prefill(q, k, v, idx, cnt, 5)
    np.testing.assert_allclose(o, ref.numpy(), atol=1e-10)


def test_closed_forms_zero_query_and_constant_value():
    q, k, v, w, z, idx, cnt = _case(7, T=60, W=8, R=6)
    B, H, T, d = q.shape
    o, lse = orc.attn_prefill(np.zeros_like(q), k, v, idx, cnt, 8)
    for b in range(B):
        for h in range(H):
            kept = idx[b, h, :cnt[b, h]]
            for i in range(T):
                nvis = int(np.sum(kept <= i - 8))
                size = min(i + 1, 8) + nvis
                assert abs(lse[b, h, i] - np.log(size)) < 1e-12      # pins |A_i| exactly
                members = list(kept[kept <= i - 8]) + list(range(max(0, i - 7), i + 1))
                np.testing.assert_allclose(o[b, h, i], v[b, h, members].mean(0), atol=1e-12)
    c = np.random.default_rng(0).standard_normal(d)
    o, _ = orc.attn_prefill(q, k, np.broadcast_to(c, v.shape).copy(), idx, cnt, 8)
    np.testing.assert_allclose(o, np.broadcast_to(c, o.shape), atol=1e-12)


def test_query_subset_and_pool_permutation():
    q, k, v, w, z, idx, cnt = _case(8, T=50, W=6, R=7)
    o, lse = orc.attn_prefill(q, k, v, idx, cnt, 6)
    qpos = np.stack([np.stack([np.sort(np.random.default_rng(h).choice(50, 9, replace=False))
                               for h in range(2)]) for _ in range(2)]).astype(np.int32)
    os_, ls_ = orc.attn_prefill(q, k, v, idx, cnt, 6, qpos=qpos)
    for b in range(2):
        for h in range(2):
            np.testing.assert_allclose(os_[b, h], o[b, h, qpos[b, h]], atol=0)
            np.testing.assert_allclose(ls_[b, h], lse[b, h, qpos[b, h]], atol=0)
    idx_perm = idx.copy()
    for b in range(2):
        for h in range(2):
            n = cnt[b, h]
            idx_perm[b, h, :n] = idx[b, h, :n][::-1]
    o2, _ = orc.attn_prefill(q, k, v, idx_perm, cnt, 6)
    np.testing.assert_allclose(o2, o, atol=1e-12)


def test_worked_example_set_sizes():
    # tests/golden/attn_set_sizes.txt: |A_i| counted by hand for the worked selection example.
    lines = [l for l in open(os.path.join(GOLD, "attn_set_sizes.txt")) if not l.startswith("#")]
    kv = dict(l.strip().split("=", 1) for l in lines if "=" in l)
    T, W = int(kv["T"]), int(kv["W"])
    idx = np.array([int(x) for x in kv["idx"].split()], np.int32)[None, None]
    cnt = np.array([[idx.shape[2]]], np.int32)
    sizes = [int(x) for x in kv["sizes"].split()]
    rng = np.random.default_rng(0)
    k, v = rng.standard_normal((1, 1, T, 4)), rng.standard_normal((1, 1, T, 4))
    _, lse = orc.attn_prefill(np.zeros((1, 1, T, 4)), k, v, idx, cnt, W)
    np.testing.assert_allclose(np.exp(lse[0, 0]), sizes, atol=1e-9)


# ---- streaming decode -------------------------------------------------------
@pytest.mark.parametrize("seed,W,R,sink", [(0, 6, 4, 0), (1, 5, 3, 2), (2, 8, 0, 0), (3, 3, 50, 0)])
def test_stream_step_equals_last_row_of_one_shot_prefill(seed, W, R, sink):
    q, k, v, w, z, _, _ = _case(10 + seed, B=1, H=3, T=45, W=W, R=R, K=5, sink=sink)
    B, H, T, d = q.shape
    o, lse, pidx, pcnt = orc.stream(q, k, v, z, W, R, sink)
    for n in range(T):
        zz = z[:, :, :n + 1]
        idx, cnt, _ = orc.select(zz, W, R, sink)       # candidates j <= n-W are all scored already
        qpos = np.full((B, H, 1), n, np.int32)
        o1, l1 = orc.attn_prefill(q[:, :, :n + 1], k[:, :, :n + 1], v[:, :, :n + 1], idx, cnt, W, qpos=qpos)
        np.testing.assert_allclose(o[:, :, n], o1[:, :, 0], atol=1e-12)
        np.testing.assert_allclose(lse[:, :, n], l1[:, :, 0], atol=1e-12)
    idx, cnt, _ = orc.select(z, W, R, sink)
    assert np.array_equal(pidx, idx) and np.array_equal(pcnt, cnt)


def test_stream_n_from_is_a_suffix():
    q, k, v, w, z, _, _ = _case(20, B=1, H=2, T=40, W=5, R=4)
    o, lse, pi, pc = orc.stream(q, k, v, z, 5, 4)
    o2, lse2, pi2, pc2 = orc.stream(q, k, v, z, 5, 4, n_from=25)
    assert np.array_equal(o[:, :, 25:], o2) and np.array_equal(lse[:, :, 25:], lse2)
    assert np.array_equal(pi, pi2) and np.array_equal(pc, pc2)
