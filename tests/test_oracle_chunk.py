"""Pins for the oracle's chunked (continued) prefill on top of a cache (Section 3.1.3, cached prefilling).

The chunk-end reading: the pool a cache holds after n0 tokens competes with the tokens that leave the window while
the chunk [n0, n1) arrives; the chunk's queries see their window and the entries of the resulting list that are older
than their window.  Pinned against (a) a worked example ranked by hand, (b) the composition property of a top-R
selection (top-R of [top-R of a prefix, plus the rest] = top-R of everything, so a chunk on top of a one-shot prefill
must reproduce the one-shot prefill of the longer prompt), (c) the token-by-token simulation where the cap never
binds, and (d) the dense masked attention of tests/bruteforce.py.
"""
import numpy as np
import pytest

from oracle import lte_oracle as orc
from tests.bruteforce import dense_attention, dense_mask


def _seq(seed, B=2, H=2, T=60, d=8, K=5):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, T, d)) for _ in range(3))
    w = rng.standard_normal((H, K, 2 * d)) * 0.2
    return q, k, v, orc.scores(k, v, w)


def test_worked_example_ranked_by_hand():
    # one head, W = 2, R = 3, tau = 0.5 (keep iff z > 0).  The cache holds n0 = 6 tokens: its pool is {1, 3} (logits 0.5
    # and 2.0), positions 4, 5 sit in the window.  The chunk brings tokens 6..9, so positions 4..7 leave the window:
    #   z4 = 1.0 (candidate), z5 = -1.0 (dropped), z6 = 0.7 (candidate), z7 = 3.0 (candidate).
    # Ranking of {1: 0.5, 3: 2.0, 4: 1.0, 6: 0.7, 7: 3.0}: 7, 3, 4 | 6, 1  ->  the list is [3, 4, 7].
    z = np.array([[[9., 0.5, -3., 2.0, 1.0, -1.0, 0.7, 3.0, 0.1, 0.2]]])
    pool = np.array([[[1, 3, -1]]], np.int32)
    idx, cnt = orc.chunk_select(z, 6, 10, 2, 3, pool, np.array([[2]], np.int32))
    assert cnt[0, 0] == 3 and idx[0, 0].tolist() == [3, 4, 7]
    # with a sink of two tokens position 1 ranks first whatever its logit: 1, 7, 3
    idx, cnt = orc.chunk_select(z, 6, 10, 2, 3, pool, np.array([[2]], np.int32), sink=2)
    assert idx[0, 0].tolist() == [1, 3, 7]
    # room for everybody: pool and the three candidates, ascending
    idx, cnt = orc.chunk_select(z, 6, 10, 2, 8, np.array([[[1, 3, -1, -1, -1, -1, -1, -1]]], np.int32), np.array([[2]], np.int32))
    assert cnt[0, 0] == 5 and idx[0, 0, :5].tolist() == [1, 3, 4, 6, 7]


@pytest.mark.parametrize("seed,n0,W,R,sink", [(0, 25, 6, 5, 0), (1, 40, 3, 4, 2), (2, 7, 9, 3, 0), (3, 0, 5, 6, 0),
                                               (4, 59, 8, 2, 1), (5, 30, 6, 100, 0)])
def test_chunk_on_a_one_shot_prefix_equals_the_one_shot_prefill(seed, n0, W, R, sink):
    q, k, v, z = _seq(seed)
    B, H, T, d = q.shape
    if n0 > 0:
        p_idx, p_cnt, _ = orc.select(z[:, :, :n0], W, R, sink)      # only positions <= n0-1-W enter: all scored by then
    else:
        p_idx, p_cnt = np.full((B, H, R), -1, np.int32), np.zeros((B, H), np.int32)
    o, lse, idx, cnt = orc.prefill_chunk(q, k, v, z, n0, W, R, p_idx, p_cnt, sink, scale=0.4)
    f_idx, f_cnt, _ = orc.select(z, W, R, sink)
    np.testing.assert_array_equal(idx, f_idx)
    np.testing.assert_array_equal(cnt, f_cnt)
    o_full, lse_full = orc.attn_prefill(q, k, v, f_idx, f_cnt, W, 0.4)
    np.testing.assert_allclose(o, o_full[:, :, n0:], atol=1e-13)
    np.testing.assert_allclose(lse, lse_full[:, :, n0:], atol=1e-13)


def test_two_chunks_compose():
    q, k, v, z = _seq(7)
    B, H, T, d = q.shape
    W, R = 5, 4
    p_idx, p_cnt, _ = orc.select(z[:, :, :20], W, R)
    _, _, i1, c1 = orc.prefill_chunk(q[:, :, :41], k[:, :, :41], v[:, :, :41], z, 20, W, R, p_idx, p_cnt)
    o2, lse2, i2, c2 = orc.prefill_chunk(q, k, v, z, 41, W, R, i1, c1)
    f_idx, f_cnt, _ = orc.select(z, W, R)
    np.testing.assert_array_equal(i2, f_idx)
    o_full, _ = orc.attn_prefill(q, k, v, f_idx, f_cnt, W)
    np.testing.assert_allclose(o2, o_full[:, :, 41:], atol=1e-13)


def test_without_a_binding_cap_the_chunk_is_the_token_by_token_simulation():
    q, k, v, z = _seq(11)
    B, H, T, d = q.shape
    W, R, n0 = 6, 64, 22                                            # R above any candidate count: nothing is ever evicted
    o_s, lse_s, p_s, c_s = orc.stream(q, k, v, z, W, R, n_from=n0)
    p_idx, p_cnt, _ = orc.select(z[:, :, :n0], W, R)
    o, lse, idx, cnt = orc.prefill_chunk(q, k, v, z, n0, W, R, p_idx, p_cnt)
    np.testing.assert_allclose(o, o_s, atol=1e-12)
    np.testing.assert_allclose(lse, lse_s, atol=1e-12)
    np.testing.assert_array_equal(cnt, c_s)
    for b in range(B):
        for h in range(H):
            assert sorted(idx[b, h, :cnt[b, h]].tolist()) == sorted(p_s[b, h, :c_s[b, h]].tolist())


def test_arbitrary_pool_against_dense_masked_attention():
    # a pool that is not the top-R of its prefix (as a cache restored from elsewhere might hold)
    q, k, v, z = _seq(13, B=1, H=2, T=36)
    W, R, n0 = 4, 5, 20
    pool = np.array([[[2, 9, 11, -1, -1], [0, 1, 15, 14, -1]]], np.int32)
    pcnt = np.array([[3, 4]], np.int32)
    pool[0, 1, :4] = np.sort(pool[0, 1, :4])
    o, lse, idx, cnt = orc.prefill_chunk(q, k, v, z, n0, W, R, pool, pcnt, scale=0.3)
    for h in range(2):
        cand = set(pool[0, h, :pcnt[0, h]].tolist()) | {j for j in range(n0 - W, 36 - W) if z[0, h, j] > 0}
        best = sorted(sorted(cand, key=lambda j: (-z[0, h, j], j))[:R])
        assert idx[0, h, :cnt[0, h]].tolist() == best
        M = dense_mask(36, W, np.array(best, np.int32))
        oref, lref, _ = dense_attention(q[0, h], k[0, h], v[0, h], M, 0.3)
        np.testing.assert_allclose(o[0, h], oref[n0:], atol=1e-12)
        np.testing.assert_allclose(lse[0, h], lref[n0:], atol=1e-12)


def test_streaming_intervals_reproduce_the_token_by_token_pool_with_a_binding_cap():
    """The streaming reading of a chunk, written as visibility intervals [enter, leave) per entry (the form the GPU path
    consumes), against the token-by-token simulation: at every query of the chunk the entries whose interval contains
    it are exactly the simulation's pool at that step (read off as the final pool of the simulation stopped there).
    The cap binds (R far below the number of candidates), so entries do leave inside the chunk."""
    rng = np.random.default_rng(5)
    T, d, W, R, sink, n0 = 90, 4, 6, 5, 1, 40
    q, k, v = (rng.standard_normal((1, 1, T, d)) for _ in range(3))
    z = rng.standard_normal((1, 1, T)); z[0, 0, 50] = z[0, 0, 44]                    # an exact tie among candidates
    p_idx, p_cnt, _ = orc.select(z[:, :, :n0], W, R, sink)
    iv = orc.stream_intervals(z[0, 0], n0, T, W, R, p_idx[0, 0], int(p_cnt[0, 0]), sink)
    left_inside = [e for e in iv if e[2] < T]
    assert len(left_inside) >= 3                                                     # the cap does bind inside the chunk
    for i in range(n0, T):
        _, _, pool_i, cnt_i = orc.stream(q[:, :, :i + 1], k[:, :, :i + 1], v[:, :, :i + 1], z[:, :, :i + 1], W, R, sink)
        want = set(int(j) for j in pool_i[0, 0, :cnt_i[0, 0]])
        got = set(j for j, a, b in iv if a <= i < b)
        assert got == want, (i, sorted(got), sorted(want))
    # an entry is seen from the query that pushes it out of the window (position + W), or from the chunk's start
    assert all(a == max(j + W, n0) for j, a, b in iv)
