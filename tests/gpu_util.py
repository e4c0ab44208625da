"""Helpers of the GPU parity tests: tensor marshalling and the retained-list comparison rule."""
import numpy as np
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte

Z_TOL = 4e-5      # |z - theta| below this counts as "on the keep threshold" (1e-5 on r = sigmoid(z))


def dev(a, dtype):
    """numpy float32 array (already rounded to the storage dtype) -> CUDA tensor of that dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def tdtype(cfg):
    return lte.BF16 if cfg.dtype == "bf16" else lte.F32


def shape_of(cfg, T=None, **kw):
    return lte.shape(kw.get("B", cfg.B), cfg.H, cfg.T if T is None else T, cfg.d, cfg.W, cfg.R, tdtype(cfg),
                     sink=cfg.sink, tau=kw.get("tau", 0.5), softmax_scale=kw.get("scale", 0.0))


def check_idx(idx_gpu, cnt_gpu, z64, W, R, sink=0, tau=0.5):
    """Retained lists must equal the oracle's, except for positions whose logit lies within Z_TOL of a
    keep threshold: logit(tau), or (when the cap binds) the logits of the R-th / (R+1)-th ranked candidate.
    Structural invariants hold regardless.  Returns the number of heads whose lists differ (legitimately)."""
    B, H, T = z64.shape
    idx_o, cnt_o, _ = orc.select(z64, W, R, sink, tau)
    zthr = orc.logit(tau)
    ndiff = 0
    for b in range(B):
        for h in range(H):
            n = int(cnt_gpu[b, h])
            got = idx_gpu[b, h, :n]
            assert 0 <= n <= R
            assert np.all(idx_gpu[b, h, n:] == -1)
            assert np.all(np.diff(got) > 0), "ascending and unique"
            assert n == 0 or (got[0] >= 0 and got[-1] <= T - 1 - W), "older than the final window"
            want = idx_o[b, h, :cnt_o[b, h]]
            if n == len(want) and np.array_equal(got, want):
                continue
            ndiff += 1
            zz = z64[b, h]
            thetas = [zthr] if np.isfinite(zthr) else []
            cand = [j for j in range(max(T - W, 0)) if j >= sink and zz[j] > zthr - Z_TOL]
            ranked = sorted(cand, key=lambda j: (-zz[j], j))
            nsink = min(sink, max(T - W, 0))
            rr = R - nsink
            if 0 < rr <= len(ranked):
                thetas.append(zz[ranked[rr - 1]])
            if 0 <= rr < len(ranked):
                thetas.append(zz[ranked[rr]])
            for j in set(got.tolist()) ^ set(want.tolist()):
                assert any(abs(zz[j] - t) < Z_TOL for t in thetas), (b, h, j, zz[j], thetas)
    return ndiff


def rel_l2(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def assert_grad_close(name, got, want, tol, idx=None, cnt=None, block=128):
    """Gradient comparison at three granularities, each with the same relative-L2 bound: the whole tensor; for a
    [B,H,T,d] tensor every block of `block` consecutive rows of every (b,h); and, given a retained list, the rows
    idx[b,h,:cnt[b,h]] of every (b,h) on their own (Eq. 6 reads exactly those rows of dV, and a wrong head's worth of
    them moves the whole-tensor norm by far less than the bound).  For other tensors with a leading head axis
    ([H,...]) the per-head slices are compared.  A slice whose reference norm is below 1e-3 of the tensor's RMS slice
    norm is compared against that floor instead (a relative error on an all-but-zero slice says nothing)."""
    a = np.asarray(got, np.float64); b = np.asarray(want, np.float64)
    assert a.shape == b.shape, (name, a.shape, b.shape)
    assert np.all(np.isfinite(a)), name
    whole = rel_l2(a, b)
    assert whole <= tol, (name, "whole tensor", whole)
    if a.ndim == 4:
        B, H, T, d = a.shape
        nb = (T + block - 1) // block
        pad = nb * block - T
        ap = np.pad(a, ((0, 0), (0, 0), (0, pad), (0, 0))).reshape(B, H, nb, block * d)
        bp = np.pad(b, ((0, 0), (0, 0), (0, pad), (0, 0))).reshape(B, H, nb, block * d)
        num = np.linalg.norm(ap - bp, axis=-1); den = np.linalg.norm(bp, axis=-1)
        floor = 1e-3 * np.sqrt(np.mean(den ** 2)) + 1e-30
        rel = num / np.maximum(den, floor)
        worst = np.unravel_index(np.argmax(rel), rel.shape)
        assert rel[worst] <= tol, (name, "(b, h, row block)", worst, float(rel[worst]))
        if idx is not None:
            for bb in range(B):
                for h in range(H):
                    rows = idx[bb, h, :cnt[bb, h]]
                    if len(rows) == 0:
                        continue
                    r = rel_l2(a[bb, h, rows], b[bb, h, rows])
                    assert r <= tol, (name, "retained rows of (b, h)", bb, h, r)
    elif a.ndim >= 2:
        num = np.linalg.norm((a - b).reshape(a.shape[0], -1), axis=-1); den = np.linalg.norm(b.reshape(a.shape[0], -1), axis=-1)
        floor = 1e-3 * np.sqrt(np.mean(den ** 2)) + 1e-30
        rel = num / np.maximum(den, floor)
        assert np.max(rel) <= tol, (name, "head", int(np.argmax(rel)), float(np.max(rel)))
    return whole
