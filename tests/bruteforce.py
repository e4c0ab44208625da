"""Dense NumPy restatements of the definitions, used to pin the oracle.

Nothing here calls the oracle or the CUDA library: every function builds its
result directly from the set definition (Eq. 5 with a W-key window) with dense
arrays, so a mistake in the oracle's loops shows up as a disagreement.
"""
import numpy as np


def dense_mask(T, W, retained):
    """M[i, j] = True iff query i may attend key j: window i-W < j <= i, or j retained and j <= i-W."""
    i = np.arange(T)[:, None]
    j = np.arange(T)[None, :]
    win = (j <= i) & (j > i - W)
    ret = np.zeros(T, bool)
    ret[np.asarray(retained, dtype=np.int64)] = True
    far = ret[None, :] & (j <= i - W)
    return win | far


def dense_attention(q, k, v, mask, scale):
    """q,k,v [T,d] fp64, mask [T,T] -> o [T,d], lse [T], p [T,T]."""
    s = (q @ k.T) * scale
    s = np.where(mask, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    den = e.sum(axis=1, keepdims=True)
    p = e / den
    return p @ v, (m + np.log(den))[:, 0], p


def topr_bruteforce(z, W, R, sink, zthr):
    """One head: candidates j <= T-1-W with (j < sink or z > zthr); order = sink first, z desc, pos asc."""
    T = len(z)
    cand = [j for j in range(max(T - W, 0)) if j < sink or z[j] > zthr]
    key = sorted(cand, key=lambda j: (0 if j < sink else 1, j if j < sink else 0, -z[j] if j >= sink else 0.0, j))
    return sorted(key[:R]), len(cand)


def scores_dense(k, v, w, bias=None):
    """k,v [T,d], w [K,2d] -> z [T] by explicit left padding and a strided window view."""
    T, d = k.shape
    K = w.shape[0]
    half = K // 2
    x = np.concatenate([k, v], axis=1)
    xp = np.concatenate([np.zeros((half, 2 * d)), x], axis=0)      # position p -> row p + half
    z = np.full(T, -np.inf)
    for j in range(T - half):
        z[j] = float((xp[j:j + K] * w).sum()) + (0.0 if bias is None else bias)
    return z
