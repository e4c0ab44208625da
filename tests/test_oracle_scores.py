"""Pins for the oracle's scorer (Section 3.1.1 / Appendix A)."""
import numpy as np
import pytest

from oracle import lte_oracle as orc
from tests.bruteforce import scores_dense


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_delta_weights_pick_one_input():
    # w[h,t0,c0] = 1 -> z_j = x[j+t0-half, c0]: pins tap orientation (cross-correlation,
    # tap 0 = oldest neighbour), concat order (k then v) and the left zero padding.
    B, H, T, d, K = 2, 3, 20, 4, 5
    half = K // 2
    k, v = _rand((B, H, T, d), 0), _rand((B, H, T, d), 1)
    for t0 in range(K):
        for c0 in (0, d - 1, d, 2 * d - 1):
            w = np.zeros((H, K, 2 * d)); w[:, t0, c0] = 1.0
            z = orc.scores(k, v, w)
            src = k[..., c0] if c0 < d else v[..., c0 - d]
            for j in range(T):
                p = j + t0 - half
                if j + half > T - 1:
                    assert np.all(np.isneginf(z[:, :, j]))
                elif p < 0:
                    assert np.all(z[:, :, j] == 0.0)
                else:
                    assert np.array_equal(z[:, :, j], src[:, :, p])


def test_zero_weights_give_bias_and_tail_is_undefined():
    B, H, T, d, K = 1, 2, 16, 4, 7
    k, v = _rand((B, H, T, d), 2), _rand((B, H, T, d), 3)
    bias = np.array([0.3, -1.2])
    z = orc.scores(k, v, np.zeros((H, K, 2 * d)), bias)
    assert np.all(z[:, 0, :T - 3] == 0.3) and np.all(z[:, 1, :T - 3] == -1.2)
    assert np.all(np.isneginf(z[:, :, T - 3:]))


@pytest.mark.parametrize("K", [1, 3, 5, 7])
def test_against_dense_padding_formulation(K):
    B, H, T, d = 2, 2, 33, 8
    k, v, w = _rand((B, H, T, d), 4), _rand((B, H, T, d), 5), _rand((H, K, 2 * d), 6)
    bias = _rand((H,), 7)
    z = orc.scores(k, v, w, bias)
    for b in range(B):
        for h in range(H):
            ref = scores_dense(k[b, h], v[b, h], w[h], bias[h])
            fin = np.isfinite(ref)
            assert np.array_equal(np.isfinite(z[b, h]), fin)
            np.testing.assert_allclose(z[b, h][fin], ref[fin], rtol=0, atol=1e-12)


def test_linearity_in_weights():
    B, H, T, d, K = 1, 2, 24, 4, 5
    k, v = _rand((B, H, T, d), 8), _rand((B, H, T, d), 9)
    w1, w2 = _rand((H, K, 2 * d), 10), _rand((H, K, 2 * d), 11)
    za, zb, zc = orc.scores(k, v, w1), orc.scores(k, v, w2), orc.scores(k, v, 2 * w1 - 3 * w2)
    fin = np.isfinite(za)
    np.testing.assert_allclose(zc[fin], (2 * za - 3 * zb)[fin], atol=1e-12)


# ---- the paper's stack ------------------------------------------------------
def _stack_numpy(k, v, wl, bl, wout, bout, ks, dil):
    """One head, written position-centred: layer l's output lives on centred positions and reads
    its input at offsets (-dil, 0, +dil); inputs and hidden activations are zero left of time 0 of
    the shifted (causal) clock, which is the reading the oracle documents."""
    T, d = k.shape
    L = len(wl)
    x = np.concatenate([k, v], axis=1)
    cur = x                                   # causal clock: row t
    for l in range(L):
        cout = wl[l].shape[0]
        nxt = np.zeros((T, cout))
        for t in range(T):
            acc = np.zeros(cout) if bl[l] is None else bl[l].copy()
            for tau in range(ks):
                p = t - (ks - 1 - tau) * dil
                if p >= 0:
                    acc = acc + wl[l][:, tau, :] @ cur[p]
            nxt[t] = acc / (1.0 + np.exp(-acc))
        cur = nxt
    half = L * (ks - 1) * dil // 2
    z = np.full(T, -np.inf)
    for j in range(T - half):
        z[j] = wout @ cur[j + half] + (0.0 if bout is None else bout)
    return z


def test_stack_matches_numpy_and_receptive_field():
    B, H, T, d, ks, dil = 1, 2, 40, 8, 3, 2
    ch = [2 * d, d, d // 2, d // 4]
    k, v = _rand((B, H, T, d), 20), _rand((B, H, T, d), 21)
    wl = [_rand((H, ch[l + 1], ks, ch[l]), 22 + l) * 0.3 for l in range(3)]
    bl = [_rand((H, ch[l + 1]), 30 + l) * 0.1 for l in range(3)]
    wout, bout = _rand((H, ch[3]), 40), _rand((H,), 41)
    z = orc.scores_stack(k, v, wl, bl, wout, bout, ks, dil)
    for h in range(H):
        ref = _stack_numpy(k[0, h], v[0, h], [x[h] for x in wl], [x[h] for x in bl], wout[h], bout[h], ks, dil)
        fin = np.isfinite(ref)
        assert np.array_equal(np.isfinite(z[0, h]), fin)
        np.testing.assert_allclose(z[0, h][fin], ref[fin], atol=1e-12)
    # receptive field 13 (Section 3.1.1): z_j depends on positions j-6..j+6 and on nothing else
    j = 20
    for p in range(T):
        k2 = k.copy(); k2[0, :, p, :] += 1.0
        z2 = orc.scores_stack(k2, v, wl, bl, wout, bout, ks, dil)
        changed = not np.allclose(z2[0, :, j], z[0, :, j])
        assert changed == (abs(p - j) <= 6 and (p - j) % 2 == 0), (p, changed)
    assert np.all(np.isneginf(z[:, :, T - 6:])) and np.all(np.isfinite(z[:, :, :T - 6]))


def test_stack_parameter_share_at_0p4b():
    # Appendix A: channel width halves per layer; the module adds about 1.7 % parameters at 0.4B
    # (hidden 1024, 24 layers of which 12 are LTE layers, 16 KV heads, head dim 64).
    d, heads, lte_layers = 64, 16, 12
    ch = [2 * d, d, d // 2, d // 4]
    per_head = sum(ch[l + 1] * 3 * ch[l] + ch[l + 1] for l in range(3)) + ch[3] + 1
    total = per_head * heads * lte_layers
    assert 0.012 < total / 0.4e9 < 0.02


def test_rope_is_a_rotation_of_channel_pairs_and_inverts():
    """Pins for the rotary embedding the lazy scoring undoes on cached keys (Section 3.1.3): each pair (c, c + d/2) is
    multiplied by exp(i angle) as a complex number; position 0 is the identity; norms are kept; the inverse undoes it."""
    rng = np.random.default_rng(0)
    d, T = 16, 40
    x = rng.standard_normal((2, 3, T, d))
    cos, sin = orc.rope_tables(100, d)
    assert np.allclose(cos[0], 1.0) and np.allclose(sin[0], 0.0)
    assert np.allclose(cos[5, 0], np.cos(5.0)) and np.allclose(sin[7, d // 2 - 1], np.sin(7.0 * 10000.0 ** (-(d - 2) / d)))
    y = orc.rope(x, cos, sin, pos0=11)
    zc = (x[..., :d // 2] + 1j * x[..., d // 2:]) * np.exp(1j * np.arange(11, 11 + T)[:, None] * 10000.0 ** (-np.arange(0, d, 2) / d))
    np.testing.assert_allclose(y[..., :d // 2], zc.real, atol=1e-12)
    np.testing.assert_allclose(y[..., d // 2:], zc.imag, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    np.testing.assert_allclose(orc.rope(y, cos, sin, pos0=11, inverse=True), x, atol=1e-12)
    np.testing.assert_allclose(orc.rope(x[..., :1, :], cos, sin, pos0=0), x[..., :1, :], atol=0)


@pytest.mark.parametrize("tau0", [0, 1, 2])
def test_stack_single_tap_reads_one_hand_worked_position(tau0):
    """Tap order inside a layer (Appendix A: kernel 3, dilation 2, three layers; cross-correlation, tap 0 = the oldest
    input).  With only tap tau0 non-zero in every layer, layer l's output at time t reads its input at t - (2 - tau0) * 2
    and nothing else, so after three layers and the deferral of the logit by 6 the logit of token j reads exactly the
    input at j - 6 (tau0 = 0), j (tau0 = 1) or j + 6 (tau0 = 2): worked out by hand from those numbers, not from the
    oracle's index expression.  A tap order taken the other way round swaps the first and the last case.  The value is
    pinned too: through one channel with unit weights it is Swish applied three times to that input."""
    B, H, T, d = 1, 2, 40, 8
    ch = [2 * d, d, d // 2, d // 4]
    k, v = _rand((B, H, T, d), 50), _rand((B, H, T, d), 51)
    wl = [np.zeros((H, ch[l + 1], 3, ch[l])) for l in range(3)]
    c_in = 3                                              # a key channel
    wl[0][:, 1, tau0, c_in] = 1.0                         # input channel 3 -> hidden channel 1
    wl[1][:, 2, tau0, 1] = 1.0                            # hidden 1 -> hidden 2
    wl[2][:, 0, tau0, 2] = 1.0                            # hidden 2 -> hidden 0
    wout = np.zeros((H, ch[3])); wout[:, 0] = 1.0
    z = orc.scores_stack(k, v, wl, [None] * 3, wout, None, 3, 2)
    src = {0: -6, 1: 0, 2: 6}[tau0]
    sw = lambda a: a / (1.0 + np.exp(-a))
    for j in range(T - 6):
        p = j + src
        # left of time 0 the input is zero, and so is every hidden activation there: the logit is Swish^3(0) = 0
        want = sw(sw(sw(k[0, :, p, c_in]))) if p >= 0 else np.zeros(H)
        np.testing.assert_allclose(z[0, :, j], want, atol=1e-14)
    # support, by perturbation: exactly one input position moves the logit of token j
    j = 20
    for p in range(T):
        k2 = k.copy(); k2[0, :, p, c_in] += 1.0
        z2 = orc.scores_stack(k2, v, wl, [None] * 3, wout, None, 3, 2)
        assert (not np.allclose(z2[0, :, j], z[0, :, j])) == (p == j + src), (tau0, p)
