"""Pins for the oracle's backward (Section 3.1.2, Eq. 6 and Eq. 7) by central finite differences."""
import numpy as np
import pytest

from oracle import lte_oracle as orc


def _case(seed, B=2, H=2, T=26, d=4, W=5, R=4, K=5):
    rng = np.random.default_rng(seed)
    q, k, v, dO = (rng.standard_normal((B, H, T, d)) for _ in range(4))
    w = rng.standard_normal((H, K, 2 * d)) * 0.3
    z = orc.scores(k, v, w)
    idx, cnt, _ = orc.select(z, W, R)
    return q, k, v, dO, w, z, idx, cnt


def _loss(q, k, v, dO, idx, cnt, W, scale):
    o, _ = orc.attn_prefill(q, k, v, idx, cnt, W, scale)
    return float((o * dO).sum())


@pytest.mark.parametrize("seed", [0, 1])
def test_dq_dk_dv_by_finite_differences(seed):
    # The index sets are frozen (selection is not differentiated), so L = <O, dO> is smooth.
    q, k, v, dO, w, z, idx, cnt = _case(seed)
    W, scale, eps = 5, 0.6, 1e-6
    g = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, W, scale, cnn_input_grad=False)
    rng = np.random.default_rng(99)
    for name, arr in (("dq", q), ("dk", k), ("dv", v)):
        for _ in range(40):
            pos = tuple(int(rng.integers(0, s)) for s in arr.shape)
            a = {"dq": q, "dk": k, "dv": v}
            hi = {n: x.copy() for n, x in a.items()}; lo = {n: x.copy() for n, x in a.items()}
            hi[name][pos] += eps; lo[name][pos] -= eps
            fd = (_loss(hi["dq"], hi["dk"], hi["dv"], dO, idx, cnt, W, scale)
                  - _loss(lo["dq"], lo["dk"], lo["dv"], dO, idx, cnt, W, scale)) / (2 * eps)
            assert abs(fd - g[name][pos]) < 1e-6 * max(1.0, abs(fd)), (name, pos, fd, g[name][pos])


def test_surrogate_is_the_gradient_of_a_mask_on_v():
    # Eq. 6: dL/dr_j := dL/dm_j with v'_j = v_j * m_j, evaluated at m = 1.
    q, k, v, dO, w, z, idx, cnt = _case(2)
    B, H, T, d = q.shape
    W, scale, eps, K = 5, 0.5, 1e-6, 5
    g = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, W, scale, cnn_input_grad=False)
    rng = np.random.default_rng(5)
    for _ in range(30):
        b, h, j = int(rng.integers(B)), int(rng.integers(H)), int(rng.integers(T - K // 2))
        vh, vl = v.copy(), v.copy()
        vh[b, h, j] *= 1 + eps; vl[b, h, j] *= 1 - eps
        dr = (_loss(q, k, vh, dO, idx, cnt, W, scale) - _loss(q, k, vl, dO, idx, cnt, W, scale)) / (2 * eps)
        r = 1 / (1 + np.exp(-z[b, h, j]))
        assert abs(g["dz"][b, h, j] - dr * r * (1 - r)) < 1e-6 * max(1.0, abs(dr))
    # the undefined tail gets no gradient
    assert np.all(g["dz"][:, :, T - K // 2:] == 0)


def test_sigmoid_factor_and_sparsity_penalty():
    q, k, v, dO, w, z, idx, cnt = _case(3)
    lam = np.array([0.7, 0.2])
    g0 = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, 5, 0.5, cnn_input_grad=False)
    g1 = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, 5, 0.5, lam=lam, cnn_input_grad=False)
    fin = np.isfinite(z)
    r = 1 / (1 + np.exp(-np.where(fin, z, 0.0)))
    # Eq. 7: d/dr [lambda_h * ReLU(r - 0.5)] = lambda_h * 1[r > 0.5]; chain through sigma'(z) = r (1 - r)
    want = np.where(fin & (r > 0.5), lam[None, :, None] * r * (1 - r), 0.0)
    np.testing.assert_allclose(g1["dz"] - g0["dz"], want, atol=1e-12)
    # sigma'(z) by finite differences of the sigmoid itself
    eps = 1e-6
    fd = (1 / (1 + np.exp(-(z[fin] + eps))) - 1 / (1 + np.exp(-(z[fin] - eps)))) / (2 * eps)
    np.testing.assert_allclose(fd, (r * (1 - r))[fin], atol=1e-9)


def test_scorer_gradients_are_the_vjp_of_the_linear_scorer():
    # With g = dz frozen, dw, dbias and the scorer's share of dk, dv are the gradients of
    # sum_j g_j z_j(w, bias, k, v), a linear function: finite differences are exact up to rounding.
    q, k, v, dO, w, z, idx, cnt = _case(4)
    B, H, T, d = q.shape
    W, scale, eps = 5, 0.5, 1e-4
    g_off = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, W, scale, cnn_input_grad=False)
    g_on = orc.attn_bwd(q, k, v, dO, z, idx, cnt, w, W, scale, cnn_input_grad=True)
    gz = g_off["dz"]
    np.testing.assert_array_equal(g_on["dz"], gz)
    np.testing.assert_array_equal(g_on["dq"], g_off["dq"])

    def lin(w_, k_, v_, bias_):
        zz = orc.scores(k_, v_, w_, bias_)
        return float(np.where(np.isfinite(zz), zz * gz, 0.0).sum())

    rng = np.random.default_rng(7)
    zero_b = np.zeros(H)
    for _ in range(30):
        pos = tuple(int(rng.integers(0, s)) for s in w.shape)
        wh, wl = w.copy(), w.copy(); wh[pos] += eps; wl[pos] -= eps
        fd = (lin(wh, k, v, zero_b) - lin(wl, k, v, zero_b)) / (2 * eps)
        assert abs(fd - g_off["dw"][pos]) < 1e-7 * max(1.0, abs(fd))
    for h in range(H):
        bh, bl = zero_b.copy(), zero_b.copy(); bh[h] += eps; bl[h] -= eps
        fd = (lin(w, k, v, bh) - lin(w, k, v, bl)) / (2 * eps)
        assert abs(fd - g_off["dbias"][h]) < 1e-7 * max(1.0, abs(fd))
    for name, arr in (("dk", k), ("dv", v)):
        for _ in range(30):
            pos = tuple(int(rng.integers(0, s)) for s in arr.shape)
            ah, al = arr.copy(), arr.copy(); ah[pos] += eps; al[pos] -= eps
            fd = ((lin(w, ah, v, zero_b) - lin(w, al, v, zero_b)) if name == "dk"
                  else (lin(w, k, ah, zero_b) - lin(w, k, al, zero_b))) / (2 * eps)
            extra = g_on[name][pos] - g_off[name][pos]
            assert abs(fd - extra) < 1e-7 * max(1.0, abs(fd))


def test_row_sums_and_constant_upstream():
    # dO constant along d and equal for all queries: dV_j = c * sum_i P_ij, so sum_j dV_j = c * T per channel.
    q, k, v, dO, w, z, idx, cnt = _case(5)
    B, H, T, d = q.shape
    ones = np.ones_like(dO)
    g = orc.attn_bwd(q, k, v, ones, z, idx, cnt, w, 5, 0.5, cnn_input_grad=False)
    np.testing.assert_allclose(g["dv"].sum(axis=2), np.full((B, H, d), float(T)), atol=1e-10)
    # with v constant the output does not depend on q or k at all
    vc = np.broadcast_to(np.random.default_rng(1).standard_normal(d), v.shape).copy()
    g = orc.attn_bwd(q, k, vc, dO, z, idx, cnt, w, 5, 0.5, cnn_input_grad=False)
    assert np.abs(g["dq"]).max() < 1e-12 and np.abs(g["dk"]).max() < 1e-12


# ---- the three-layer scorer stack: its backward against central finite differences ------------------------------------
def _stack_case(seed, B=2, H=2, T=37, d=8, bias=True):
    rng = np.random.default_rng(seed)
    ch = [2 * d, d, d // 2, d // 4]
    k = rng.standard_normal((B, H, T, d)); v = rng.standard_normal((B, H, T, d))
    wl = [rng.standard_normal((H, ch[l + 1], 3, ch[l])) * 0.4 for l in range(3)]
    bl = [rng.standard_normal((H, ch[l + 1])) * 0.2 for l in range(3)] if bias else [None] * 3
    wout = rng.standard_normal((H, ch[3])); bout = rng.standard_normal((H,)) if bias else None
    g = rng.standard_normal((B, H, T))
    return rng, k, v, wl, bl, wout, bout, g


@pytest.mark.parametrize("seed,bias", [(0, True), (1, False)])
def test_stack_backward_matches_finite_differences(seed, bias):
    """L = sum_j g_j z_j over the defined logits; every gradient of the stack's backward is dL/d(parameter or input),
    checked entry by entry with central differences in fp64 (the definition, independent of the chain rule used)."""
    rng, k, v, wl, bl, wout, bout, g = _stack_case(seed, bias=bias)
    T = k.shape[2]

    def loss():
        z = orc.scores_stack(k, v, wl, bl, wout, bout)
        return float((g[:, :, : T - 6] * z[:, :, : T - 6]).sum())

    r = orc.scores_stack_bwd(k, v, wl, bl, wout, bout, g)        # g at the undefined tail is ignored
    groups = [("wl0", wl[0], r["dwl"][0]), ("wl1", wl[1], r["dwl"][1]), ("wl2", wl[2], r["dwl"][2]),
              ("wout", wout, r["dwout"]), ("k", k, r["dk"]), ("v", v, r["dv"])]
    if bias:
        groups += [("bl0", bl[0], r["dbl"][0]), ("bl1", bl[1], r["dbl"][1]), ("bl2", bl[2], r["dbl"][2]), ("bout", bout, r["dbout"])]
    eps = 1e-6
    for name, arr, grad in groups:
        picks = [tuple(rng.integers(0, n) for n in arr.shape) for _ in range(6)]
        if name in ("k", "v"):                                   # early and late times: the zero padding and the open right end
            picks += [(0, 0, 0, 1), (1, 1, 3, 2), (0, 1, T - 1, 0), (1, 0, T - 7, 3)]
        for ix in picks:
            old = arr[ix]
            arr[ix] = old + eps; a = loss()
            arr[ix] = old - eps; b = loss()
            arr[ix] = old
            fd = (a - b) / (2 * eps)
            assert abs(fd - grad[ix]) <= 1e-6 * max(1.0, abs(fd)), (name, ix, fd, grad[ix])


def test_stack_backward_structure():
    """Linearity in the upstream gradient, no gradient from the undefined tail, and the last inputs that cannot reach a
    defined logit (a token's receptive field reaches 6 positions to either side) get exactly zero."""
    rng, k, v, wl, bl, wout, bout, g = _stack_case(2)
    T = k.shape[2]
    r1 = orc.scores_stack_bwd(k, v, wl, bl, wout, bout, g)
    r2 = orc.scores_stack_bwd(k, v, wl, bl, wout, bout, 2.0 * g)
    assert np.allclose(r2["dwl"][0], 2 * r1["dwl"][0]) and np.allclose(r2["dk"], 2 * r1["dk"])
    g_tail = np.zeros_like(g); g_tail[:, :, T - 6:] = 1.0
    r0 = orc.scores_stack_bwd(k, v, wl, bl, wout, bout, g_tail)
    assert all(np.all(a == 0) for a in r0["dwl"]) and np.all(r0["dk"] == 0) and np.all(r0["dbout"] == 0)
    g_one = np.zeros_like(g); g_one[0, 0, 10] = 1.0                # one logit: inputs outside [10-6, 10+6] are untouched
    r3 = orc.scores_stack_bwd(k, v, wl, bl, wout, bout, g_one)
    live = np.abs(r3["dk"][0, 0]).sum(axis=1) > 0
    # dilation 2: the logit of token 10 is the output at time 16 and sees times 16, 14, ..., 4 only
    assert live[4:17:2].all() and not live[5:17:2].any() and not live[:4].any() and not live[17:].any()
    assert np.all(r3["dk"][1] == 0) and np.all(r3["dk"][0, 1] == 0)
