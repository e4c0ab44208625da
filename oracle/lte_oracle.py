"""ctypes front end of the fp64 CPU oracle (``lte_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's cpu_baseline / reference arm.  It shares nothing with the CUDA
library.  Every function widens its inputs to float64 (exact for fp32 and bf16
values) and returns float64 / int32 numpy arrays.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lte_oracle.c")
_LIB = os.path.join(_HERE, "liblte_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc (-O2 -fopenmp) if the .so is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads():
    return int(_load().oracle_num_threads())


def logit(tau):
    """Keep iff r > tau  <=>  z > logit(tau); tau <= 0 keeps every scored token."""
    if tau <= 0.0:
        return -np.inf
    if tau >= 1.0:
        return np.inf
    return float(np.log(tau) - np.log1p(-tau))


def scores(k, v, w, bias=None):
    """Single-layer scorer: k, v [B,H,T,d], w [H,K,2d], bias [H] -> z [B,H,T]."""
    k, v, w = _f64(k), _f64(v), _f64(w)
    B, H, T, d = k.shape
    K = w.shape[1]
    assert w.shape == (H, K, 2 * d)
    bias = None if bias is None else _f64(bias)
    z = np.empty((B, H, T), np.float64)
    _load().oracle_scores(B, H, T, d, K, _p(k), _p(v), _p(w), _p(bias), _p(z))
    return z


def scores_stack(k, v, wl, bl, wout, bout, ks=3, dil=2):
    """The paper's conv stack: wl[l] [H,c_{l+1},ks,c_l], bl[l] [H,c_{l+1}] or None,
    wout [H,c_L], bout [H] or None -> z [B,H,T]."""
    k, v = _f64(k), _f64(v)
    B, H, T, d = k.shape
    L = len(wl)
    wl = [_f64(x) for x in wl]
    bl = [None if x is None else _f64(x) for x in bl]
    ch = [2 * d] + [x.shape[1] for x in wl]
    for l in range(L):
        assert wl[l].shape == (H, ch[l + 1], ks, ch[l])
    wout = _f64(wout)
    bout = None if bout is None else _f64(bout)
    ch_a = (ctypes.c_int * (L + 1))(*ch)
    wl_a = (ctypes.c_void_p * L)(*[x.ctypes.data for x in wl])
    bl_a = (ctypes.c_void_p * L)(*[None if x is None else x.ctypes.data for x in bl])
    z = np.empty((B, H, T), np.float64)
    _load().oracle_scores_stack(B, H, T, d, L, ks, dil, ch_a, wl_a, bl_a,
                                _p(wout), _p(bout), _p(k), _p(v), _p(z))
    return z


def scores_stack_bwd(k, v, wl, bl, wout, bout, dz, ks=3, dil=2):
    """Gradients of the conv stack for a given dL/dz [B,H,T] (taken as zero where the logit is undefined):
    dict(dwl [list], dbl [list], dwout, dbout, dk, dv)."""
    k, v, dz = _f64(k), _f64(v), _f64(dz)
    B, H, T, d = k.shape
    L = len(wl)
    half = L * (ks - 1) * dil // 2
    dz = dz.copy()
    dz[:, :, max(T - half, 0):] = 0.0
    wl = [_f64(x) for x in wl]
    bl = [None if x is None else _f64(x) for x in bl]
    ch = [2 * d] + [x.shape[1] for x in wl]
    wout = _f64(wout)
    bout = None if bout is None else _f64(bout)
    dwl = [np.empty_like(x) for x in wl]
    dbl = [np.empty((H, ch[l + 1]), np.float64) for l in range(L)]
    dwout = np.empty_like(wout); dbout = np.empty((H,), np.float64)
    dk = np.empty_like(k); dv = np.empty_like(v)
    ch_a = (ctypes.c_int * (L + 1))(*ch)
    arr = lambda xs: (ctypes.c_void_p * L)(*[None if x is None else x.ctypes.data for x in xs])
    _load().oracle_scores_stack_bwd(B, H, T, d, L, ks, dil, ch_a, arr(wl), arr(bl), _p(wout), _p(bout),
                                    _p(k), _p(v), _p(dz), arr(dwl), arr(dbl), _p(dwout), _p(dbout), _p(dk), _p(dv))
    return dict(dwl=dwl, dbl=dbl, dwout=dwout, dbout=dbout, dk=dk, dv=dv)


def select(z, W, R, sink=0, tau=0.5):
    """One-shot capped selection -> idx [B,H,R] ascending (-1 unused), cnt, ncand."""
    z = _f64(z)
    B, H, T = z.shape
    idx = np.empty((B, H, max(R, 0)), np.int32)
    cnt = np.empty((B, H), np.int32)
    ncand = np.empty((B, H), np.int32)
    _load().oracle_select(B, H, T, W, R, sink, ctypes.c_double(logit(tau)),
                          _p(z), _p(idx), _p(cnt), _p(ncand))
    return idx, cnt, ncand


def attn_prefill(q, k, v, idx, cnt, W, scale=None, qpos=None):
    """Window + retained softmax attention -> o [B,H,nq,d], lse [B,H,nq]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, T, d = q.shape
    idx, cnt = _i32(idx), _i32(cnt)
    R = idx.shape[2]
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    if qpos is None:
        nq = T
    else:
        qpos = _i32(qpos)
        nq = qpos.shape[2]
    o = np.empty((B, H, nq, d), np.float64)
    lse = np.empty((B, H, nq), np.float64)
    _load().oracle_attn_prefill(B, H, T, d, W, R, ctypes.c_double(scale), _p(q), _p(k), _p(v),
                                _p(idx), _p(cnt), _p(qpos), nq, _p(o), _p(lse))
    return o, lse


def chunk_select(z, n0, n1, W, R, pool_idx, pool_cnt, sink=0, tau=0.5):
    """Retained list after a chunk of tokens [n0, n1) arrives on top of a cache that holds n0 tokens
    (Section 3.1.3, cached prefilling): the pool entries pool_idx[:pool_cnt] compete with the tokens that leave
    the window during the chunk, positions max(n0 - W, 0) .. n1 - 1 - W, of which only sink tokens and tokens
    with z > logit(tau) are candidates; the best R stay (sink first, then z descending, then position ascending).
    z [B,H,>=n1-W] are the logits of the whole sequence.  -> idx [B,H,R] ascending (-1 unused), cnt [B,H]."""
    z = _f64(z)
    B, H = z.shape[:2]
    thr = logit(tau)
    idx = np.full((B, H, max(R, 0)), -1, np.int32)
    cnt = np.zeros((B, H), np.int32)
    for b in range(B):
        for h in range(H):
            cand = [int(j) for j in pool_idx[b, h, :pool_cnt[b, h]]]
            for j in range(max(n0 - W, 0), n1 - W):
                if j < sink or z[b, h, j] > thr:
                    cand.append(j)
            assert len(set(cand)) == len(cand), "a pool entry is still inside the window"
            cand.sort(key=lambda j: (0 if j < sink else 1, 0.0 if j < sink else -z[b, h, j], j))
            keep = sorted(cand[:max(R, 0)])
            idx[b, h, :len(keep)] = keep
            cnt[b, h] = len(keep)
    return idx, cnt


def prefill_chunk(q, k, v, z, n0, W, R, pool_idx, pool_cnt, sink=0, tau=0.5, scale=None):
    """Attention of the chunk's queries [n0, n1) (n1 = sequence length of q, k, v) under the chunk-end reading:
    query i sees its window and the entries of the list after the chunk that are older than its window.
    -> o [B,H,n1-n0,d], lse [B,H,n1-n0], idx, cnt (the new pool)."""
    B, H, n1, d = np.asarray(q).shape
    idx, cnt = chunk_select(z, n0, n1, W, R, pool_idx, pool_cnt, sink, tau)
    qpos = np.broadcast_to(np.arange(n0, n1, dtype=np.int32), (B, H, n1 - n0)).copy()
    o, lse = attn_prefill(q, k, v, idx, cnt, W, scale, qpos=qpos)
    return o, lse, idx, cnt


def rope_tables(n_pos, d, base=10000.0):
    """cos, sin [n_pos, d/2] of the rotary position embedding: angle(p, c) = p base^(-2c/d)."""
    inv = base ** (-np.arange(0, d, 2, dtype=np.float64) / d)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def rope(x, cos, sin, pos0=0, inverse=False):
    """Rotary embedding of x [..., T, d] at positions pos0 .. pos0+T-1, half-split pairing: channels c and c + d/2 form
    the pair that is rotated by angle(p, c): (x1, x2) -> (x1 cos - x2 sin, x2 cos + x1 sin).  inverse=True rotates back
    (the same with the sine negated), which is what the scorer needs when the cache holds rotated keys
    (Section 3.1.3, lazy scoring paragraph)."""
    x = _f64(x)
    T, d = x.shape[-2], x.shape[-1]
    c, s = _f64(cos)[pos0:pos0 + T], _f64(sin)[pos0:pos0 + T]
    if inverse:
        s = -s
    x1, x2 = x[..., :d // 2], x[..., d // 2:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def sparsity_stats(z, lam=None, tau=0.5):
    """Eq. 7 and the retention count it is steered by: count[h] = mean over the batch of #{i : r_i > tau} per sequence,
    penalty = sum_h lam[h] sum_{b,i} ReLU(r_i - tau), r = sigmoid(z), over the scored positions (z > -inf)."""
    z = _f64(z)
    B, H, T = z.shape
    r = 1.0 / (1.0 + np.exp(-z))                       # sigmoid(-inf) = 0: unscored positions drop out of both sums
    count = (r > tau).sum(axis=2).mean(axis=0)
    pen = np.maximum(r - tau, 0.0).sum(axis=(0, 2))
    lam = np.ones(H) if lam is None else _f64(lam)
    return count, float((lam * pen).sum())


def lambda_update(lam, cbar, count, step, u=32, cap=512.0, alpha=1.2, band=0.95, lam_floor=1e-9, lam_max=1.0):
    """One step of Algorithm 1's feedback loop for the penalty weights (arrays over heads, returned as new arrays).
    Every step: cbar <- (1 - a) cbar + a count with a = 2 / (1 + u / 2) (the new sample takes the weight a: the
    listing prints the two weights the other way round, which would freeze cbar).  Every u-th step (step mod u == 0):
    lam <- lam alpha^s with s = [cbar > cap] - [cbar < band cap]; lam <- min(lam, lam_max); lam below lam_floor -> 0;
    a head whose cbar exceeds the cap with lam = 0 is re-enabled at lam_floor."""
    lam, cbar, count = _f64(lam).copy(), _f64(cbar).copy(), _f64(count)
    a = 2.0 / (1.0 + u / 2.0)
    cbar = (1.0 - a) * cbar + a * count
    if step % u == 0:
        s = (cbar > cap).astype(np.float64) - (cbar < band * cap).astype(np.float64)
        lam = lam * np.power(alpha, s)
        lam = np.minimum(lam, lam_max)
        lam[lam < lam_floor] = 0.0
        lam[(cbar > cap) & (lam == 0.0)] = lam_floor
    return lam, cbar


def stream(q, k, v, z, W, R, sink=0, tau=0.5, scale=None, n_from=0):
    """Token-by-token simulation from an empty cache; outputs for steps >= n_from
    and the final pool (ascending positions)."""
    q, k, v, z = _f64(q), _f64(k), _f64(v), _f64(z)
    B, H, T, d = q.shape
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    o = np.empty((B, H, T - n_from, d), np.float64)
    lse = np.empty((B, H, T - n_from), np.float64)
    pidx = np.empty((B, H, max(R, 0)), np.int32)
    pcnt = np.empty((B, H), np.int32)
    _load().oracle_stream(B, H, T, d, W, R, sink, ctypes.c_double(logit(tau)),
                          ctypes.c_double(scale), n_from, _p(q), _p(k), _p(v), _p(z),
                          _p(o), _p(lse), _p(pidx), _p(pcnt))
    return o, lse, pidx, pcnt


def attn_bwd(q, k, v, dO, z, idx, cnt, w, W, scale=None, tau=0.5, lam=None,
             cnn_input_grad=True):
    """Backward with the straight-through surrogate -> dict(dq, dk, dv, dw, dbias, dz)."""
    q, k, v, dO, z, w = _f64(q), _f64(k), _f64(v), _f64(dO), _f64(z), _f64(w)
    B, H, T, d = q.shape
    idx, cnt = _i32(idx), _i32(cnt)
    R = idx.shape[2]
    K = w.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    lam = None if lam is None else _f64(lam)
    dq = np.empty_like(q); dk = np.empty_like(q); dv = np.empty_like(q)
    dw = np.empty_like(w); db = np.empty((H,), np.float64); dz = np.empty((B, H, T), np.float64)
    _load().oracle_attn_bwd(B, H, T, d, W, R, K, ctypes.c_double(scale),
                            ctypes.c_double(logit(tau)), int(bool(cnn_input_grad)),
                            _p(q), _p(k), _p(v), _p(dO), _p(z), _p(idx), _p(cnt), _p(w), _p(lam),
                            _p(dq), _p(dk), _p(dv), _p(dw), _p(db), _p(dz))
    return dict(dq=dq, dk=dk, dv=dv, dw=dw, dbias=db, dz=dz)


# ---- training-free selection rules of the ablation (Section 4, last paragraph) ---------------------------------
RULE_LEARNED, RULE_UNIFORM, RULE_ACCUM_ATTN = 0, 1, 2


def select_uniform(B, H, T, W, R, sink=0):
    """"Unif.+SWA": out-of-window tokens retained at a uniform stride.  Eligible positions are 0 .. E-1 with
    E = max(T - W, 0).  Sink positions j < sink come first and count against R; the n = R - #sink remaining slots
    go to the positions sink, sink + stride, sink + 2 stride, ... < E with the smallest stride that fits:
    stride = max(1, ceil((E - sink) / n)).  The same list for every head.  -> idx [B,H,R] ascending (-1 unused), cnt."""
    E = max(T - W, 0)
    keep = list(range(min(sink, E, max(R, 0))))
    n = max(R, 0) - len(keep)
    rest = E - min(sink, E)
    if n > 0 and rest > 0:
        stride = max(1, -(-rest // n))
        keep += list(range(sink, E, stride))
    idx = np.full((B, H, max(R, 0)), -1, np.int32)
    cnt = np.full((B, H), len(keep), np.int32)
    idx[:, :, :len(keep)] = np.asarray(keep, np.int32)
    return idx, cnt


def attn_colsum(q, k, idx, cnt, W, scale=None):
    """Accumulated attention of every key: a[b,h,j] = sum over the queries i that attend j (window i-W < j <= i, or j in
    the list and j <= i-W) of P_ij, P = the softmax weights of lte_attn_prefill over those sets.  The ranking quantity of
    the accumulated-attention eviction heuristics the ablation compares with.  -> a [B,H,T]."""
    q, k = _f64(q), _f64(k)
    B, H, T, d = q.shape
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    a = np.zeros((B, H, T), np.float64)
    for b in range(B):
        for h in range(H):
            kept = [int(j) for j in idx[b, h, :cnt[b, h]]]
            for i in range(T):
                js = [j for j in kept if j <= i - W] + list(range(max(i - W + 1, 0), i + 1))
                s = np.array([scale * float(q[b, h, i] @ k[b, h, j]) for j in js])
                p = np.exp(s - s.max())
                p /= p.sum()
                for j, pj in zip(js, p):
                    a[b, h, j] += pj
    return a


def select_rule(rule, score, T, W, R, sink=0, tau=0.5, B=None, H=None):
    """lte_select with a rule: RULE_LEARNED = select(score = z, threshold tau); RULE_UNIFORM = select_uniform (score
    unused); RULE_ACCUM_ATTN: every out-of-window token is a candidate, the R with the largest accumulated attention
    stay (sink first, ties to the older token): select() without a threshold."""
    if rule == RULE_UNIFORM:
        if score is not None:
            B, H = np.asarray(score).shape[:2]
        return select_uniform(B, H, T, W, R, sink)
    if rule == RULE_ACCUM_ATTN:
        idx, cnt, _ = select(score, W, R, sink, tau=0.0)
        return idx, cnt
    idx, cnt, _ = select(score, W, R, sink, tau)
    return idx, cnt


def stream_intervals(z, n0, n1, W, R, pool_idx, pool_cnt, sink=0, tau=0.5):
    """The streaming rule of Section 3.1.3 (decoding paragraph: a token leaving the window is appended while the pool has
    room, else it replaces the lowest-scoring entry iff it scores strictly higher) applied token by token while a chunk
    [n0, n1) arrives on top of a pool, written as visibility intervals: entry j is in the pool for the queries
    enter <= i < leave.  One (b,h): z [>= n1 - W] logits of the whole sequence, pool_idx[:pool_cnt] the pool before the
    chunk (entries of the pool before the chunk get enter = n0).  Sink tokens are never evicted; among equal lowest
    scores the youngest goes.  -> list of (position, enter, leave) in order of entering; leave = n1 for the survivors."""
    thr = logit(tau)
    pool = [int(j) for j in pool_idx[:pool_cnt]]
    rec = {j: [j, n0, n1] for j in pool}
    order = list(pool)
    for n in range(n0, n1):
        p = n - W
        if p < 0 or R <= 0 or p in rec or not (p < sink or z[p] > thr):
            continue
        if len(pool) < R:
            pool.append(p)
        elif p >= sink:
            cand = [j for j in pool if j >= sink]
            if not cand:
                continue
            worst = min(cand, key=lambda j: (z[j], -j))
            if not z[p] > z[worst]:
                continue
            rec[worst][2] = n
            pool[pool.index(worst)] = p
        else:
            continue
        rec[p] = [p, n, n1]
        order.append(p)
    return [tuple(rec[j]) for j in order]
