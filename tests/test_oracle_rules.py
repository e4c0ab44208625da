"""Pins for the training-free selection rules of the ablation (Section 4): uniform stride + window, and ranking by
accumulated attention."""
import os

import numpy as np

from oracle import lte_oracle as orc
from tests.bruteforce import dense_attention, dense_mask

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or "=" not in line:
            continue
        k, v = line.strip().split("=")
        out[k] = [int(x) for x in v.split()]
    return out


def test_uniform_stride_hand_worked_example():
    g = _gold("uniform_stride_worked_example.txt")
    T, W, sink = g["T"][0], g["W"][0], g["sink"][0]
    idx, cnt = orc.select_uniform(2, 3, T, W, g["R"][0], sink)
    assert np.all(cnt == len(g["idx"]))
    assert idx.shape == (2, 3, g["R"][0]) and np.all(idx[:, :, :len(g["idx"])] == g["idx"]) and np.all(idx[:, :, len(g["idx"]):] == -1)
    idx2, cnt2 = orc.select_uniform(1, 1, T, W, g["R2"][0], sink)
    assert cnt2[0, 0] == g["cnt2"][0] and list(idx2[0, 0, :cnt2[0, 0]]) == list(range(g["cnt2"][0]))
    idx3, cnt3 = orc.select_uniform(1, 1, T, W, g["R3"][0], sink)
    assert list(idx3[0, 0, :cnt3[0, 0]]) == g["idx3"]


def test_uniform_stride_invariants():
    rng = np.random.default_rng(0)
    for _ in range(200):
        T, W, R, sink = int(rng.integers(1, 300)), int(rng.integers(1, 80)), int(rng.integers(0, 60)), int(rng.integers(0, 5))
        idx, cnt = orc.select_uniform(1, 1, T, W, R, sink)
        kept = idx[0, 0, :cnt[0, 0]]
        E = max(T - W, 0)
        assert cnt[0, 0] <= R and np.all(np.diff(kept) > 0) and (len(kept) == 0 or kept[-1] <= E - 1)
        ns = min(sink, E, R)
        assert list(kept[:ns]) == list(range(ns))                        # the sink comes first
        rest = kept[ns:]
        if len(rest) > 1:
            assert len(set(np.diff(rest))) == 1                          # one stride
        if R - ns > 0 and E - min(sink, E) > 0:
            stride = rest[1] - rest[0] if len(rest) > 1 else None
            assert rest[0] == sink
            if stride is not None and stride > 1:                        # the smallest stride that fits: one less would overflow
                assert len(range(sink, E, stride - 1)) > R - ns
            assert E - 1 - rest[-1] < (stride or E)                      # the stride runs through to the end


def test_accumulated_attention_against_dense_mask_and_row_sums():
    rng = np.random.default_rng(1)
    B, H, T, d, W = 1, 2, 40, 8, 6
    q, k = rng.standard_normal((B, H, T, d)), rng.standard_normal((B, H, T, d))
    idx = np.full((B, H, 5), -1, np.int32); cnt = np.zeros((B, H), np.int32)
    idx[0, 0, :4] = [0, 3, 11, 20]; cnt[0, 0] = 4
    idx[0, 1, :2] = [7, 30]; cnt[0, 1] = 2
    a = orc.attn_colsum(q, k, idx, cnt, W)
    for h in range(H):
        m = dense_mask(T, W, idx[0, h, :cnt[0, h]])
        _, _, p = dense_attention(q[0, h], k[0, h], k[0, h], m, 1.0 / np.sqrt(d))
        np.testing.assert_allclose(a[0, h], p.sum(axis=0), atol=1e-12)     # column sums of the dense masked softmax
        assert abs(a[0, h].sum() - T) < 1e-9                                # every query's weights sum to one
    # q = 0: uniform weights 1 / |A_i|: a closed form that pins which queries see which key
    a0 = orc.attn_colsum(np.zeros_like(q), k, idx, cnt, W)
    for h in range(H):
        kept = idx[0, h, :cnt[0, h]]
        size = np.array([min(i + 1, W) + np.sum(kept <= i - W) for i in range(T)], float)
        want = np.zeros(T)
        for j in range(T):
            seen = [i for i in range(j, min(j + W, T))] + ([i for i in range(j + W, T)] if j in kept else [])
            want[j] = sum(1.0 / size[i] for i in seen)
        np.testing.assert_allclose(a0[0, h], want, atol=1e-12)


def test_accumulated_attention_rule_is_top_r_without_a_threshold():
    a = np.array([[[0.2, 3.0, 0.0, 1.5, 1.5, 0.1, 9.0, 9.0, 9.0, 9.0]]])    # T = 10, W = 4 -> eligible 0..5
    idx, cnt = orc.select_rule(orc.RULE_ACCUM_ATTN, a, 10, 4, 3)
    assert list(idx[0, 0, :cnt[0, 0]]) == [1, 3, 4]                          # 3.0, then the tie at 1.5 (older first)
    idx, cnt = orc.select_rule(orc.RULE_ACCUM_ATTN, a, 10, 4, 10)
    assert list(idx[0, 0, :cnt[0, 0]]) == [0, 1, 2, 3, 4, 5]                 # a zero score is still a candidate
    idx, cnt = orc.select_rule(orc.RULE_ACCUM_ATTN, a, 10, 4, 2, sink=1)
    assert list(idx[0, 0, :cnt[0, 0]]) == [0, 1]                             # sink first, counted against the budget
