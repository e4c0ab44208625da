"""GPU parity: lte_attn_prefill_chunk (chunked prefill on top of a cache) against the oracle's chunk-end reading,
through the C ABI: outputs of the chunk's queries, the pool the cache holds afterwards, and decode steps that follow."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import dev, shape_of
from tests.test_gpu_decode import _read_pool

pytestmark = pytest.mark.gpu

TOL = {"bf16": 2e-2, "f32": 1e-4}


def _cfg(dtype="bf16", B=2, H=3, d=64, W=32, R=24, K=7, sink=0):
    return synth.Config("chunk", dtype, B, H, d, 0, W, R, K, 0.05 if dtype == "bf16" else 0.1, sink=sink)


def _run(cfg, plan, seed=0, scale=0.0, group=1, streaming=False):
    """plan: list of ("prefill", n) (first only), ("decode", n), ("chunk", n).  Returns per-phase GPU outputs and the
    final cache; every phase continues the same sequence."""
    Ttot = sum(n for _, n in plan)
    x = synth.make(cfg, seed, T=Ttot)
    rng = np.random.default_rng(seed + 100)
    if group > 1:          # query heads: group per key/value head, adjacent
        x["q"] = synth.round_bf16(rng.standard_normal((cfg.B, cfg.H * group, Ttot, cfg.d)).astype(np.float32) / cfg.d ** 0.25)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = (dev(x[t], cfg.dtype) for t in "qkv")
    n = 0
    cache = None
    outs = []
    for kind, m in plan:
        s = lte.shape(cfg.B, cfg.H, max(m, 0), cfg.d, cfg.W, cfg.R, lte.BF16 if cfg.dtype == "bf16" else lte.F32, sink=cfg.sink,
                      softmax_scale=scale, group=group)
        if kind == "prefill":
            assert n == 0
            if m > 0:
                kp, vp = k[:, :, :m].contiguous(), v[:, :, :m].contiguous()
                z = lte.lte_scores(s, c, kp, vp)
                idx, cnt = lte.lte_select(s, z)
                cache = lte.lte_cache_init(s, c, kp, vp, z, idx, cnt)
            else:
                cache = lte.lte_cache_init(s, c)
            outs.append(None)
        elif kind == "decode":
            oo, ll = [], []
            for t in range(n, n + m):
                o1, l1 = lte.lte_attn_decode(s, c, cache, q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous())
                oo.append(o1.float().cpu().numpy()); ll.append(l1.cpu().numpy())
            outs.append((np.stack(oo, axis=2), np.stack(ll, axis=2)))
        else:
            o, l = lte.lte_attn_prefill_chunk(s, c, cache, n, q[:, :, n:n + m].contiguous(), k[:, :, n:n + m].contiguous(),
                                              v[:, :, n:n + m].contiguous(), streaming=streaming)
            outs.append((o.float().cpu().numpy(), l.cpu().numpy()))
        n += m
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    return x, outs, cache


def _oracle(cfg, x, plan, scale=0.0, group=1, streaming=False):
    """The same plan on the oracle: decode steps by the token-by-token simulation (its pool at any time is the one-shot
    list of the prefix), chunks by prefill_chunk on top of that pool."""
    sc = None if scale == 0.0 else scale
    z = orc.scores(x["k"], x["v"], x["w"])
    kq = np.repeat(x["k"], group, axis=1); vq = np.repeat(x["v"], group, axis=1); zq = np.repeat(z, group, axis=1)
    n = 0
    outs = []
    for kind, m in plan:
        if kind == "prefill":
            outs.append(None)
        elif kind == "decode" or streaming:                        # the streaming reading of a chunk IS the token-by-token simulation
            o, l, _, _ = orc.stream(x["q"][:, :, :n + m], kq[:, :, :n + m], vq[:, :, :n + m], zq[:, :, :n + m], cfg.W, cfg.R, cfg.sink, scale=sc, n_from=n)
            outs.append((o, l))
        else:
            if n > 0:
                p_idx, p_cnt, _ = orc.select(zq[:, :, :n], cfg.W, cfg.R, cfg.sink)
            else:
                p_idx = np.full((cfg.B, cfg.H * group, cfg.R), -1, np.int32); p_cnt = np.zeros((cfg.B, cfg.H * group), np.int32)
            o, l, _, _ = orc.prefill_chunk(x["q"][:, :, :n + m], kq[:, :, :n + m], vq[:, :, :n + m], zq, n, cfg.W, cfg.R, p_idx, p_cnt,
                                           cfg.sink, scale=sc)
            outs.append((o, l))
        n += m
    f_idx, f_cnt, _ = orc.select(z[:, :, :n], cfg.W, cfg.R, cfg.sink)
    return outs, f_idx, f_cnt, n


def _compare(cfg, plan, seed=0, scale=0.0, group=1, streaming=False):
    x, got, cache = _run(cfg, plan, seed, scale, group, streaming)
    want, f_idx, f_cnt, n = _oracle(cfg, x, plan, scale, group, streaming)
    for (kind, m), g, w in zip(plan, got, want):
        if g is None:
            continue
        assert np.max(np.abs(g[0] - w[0])) <= TOL[cfg.dtype], (kind, m, np.max(np.abs(g[0] - w[0])))
        assert np.max(np.abs(g[1] - w[1])) <= TOL[cfg.dtype], (kind, m)
    pools, ns = _read_pool(cache, cfg, cfg.B)
    assert all(t == n for t in ns)
    for bh, pool in enumerate(pools):
        b, h = divmod(bh, cfg.H)
        assert np.array_equal(pool, f_idx[b, h, :f_cnt[b, h]]), (bh, pool, f_idx[b, h, :f_cnt[b, h]])


@pytest.mark.parametrize("plan", [
    [("prefill", 200), ("chunk", 150), ("decode", 12)],
    [("prefill", 100), ("decode", 30), ("chunk", 80), ("decode", 10)],
    [("prefill", 0), ("chunk", 100), ("chunk", 60), ("decode", 5)],
    [("prefill", 10), ("chunk", 70)],                      # fewer tokens than the window in the cache
    [("prefill", 32), ("chunk", 40)],                      # exactly the window
    [("prefill", 33), ("chunk", 5), ("chunk", 1), ("chunk", 3), ("decode", 4)],   # chunks shorter than the window
    [("prefill", 0), ("chunk", 3), ("chunk", 20), ("chunk", 300)],
])
def test_chunk_plans_bf16(plan):
    _compare(_cfg(), plan)


@pytest.mark.parametrize("kw,plan,scale,group", [
    (dict(dtype="f32", d=32, W=16, R=8, K=5, B=1, H=2), [("prefill", 60), ("chunk", 50), ("decode", 6)], 0.0, 1),
    (dict(d=128, W=40, R=30, B=1, H=2), [("prefill", 150), ("chunk", 140), ("decode", 6)], 0.0, 1),
    (dict(sink=3), [("prefill", 34), ("chunk", 120), ("decode", 6)], 0.0, 1),
    (dict(sink=2, W=8, R=5), [("prefill", 0), ("chunk", 9), ("chunk", 40)], 1.0, 1),
    (dict(W=64, R=64, B=1, H=2), [("prefill", 300), ("chunk", 200), ("decode", 6)], 0.0, 4),
    (dict(W=128, R=128, B=2, H=4), [("prefill", 700), ("chunk", 650)], 0.0, 1),      # several tiles, ragged tail
    (dict(W=32, R=0), [("prefill", 50), ("chunk", 90), ("decode", 5)], 0.0, 1),           # no pool at all: sliding window only
    (dict(dtype="f32", d=64, W=20, R=10, K=3, B=1, H=2), [("prefill", 0), ("chunk", 45), ("decode", 3), ("chunk", 30)], 0.0, 3),
])
def test_chunk_dtypes_sinks_groups(kw, plan, scale, group):
    _compare(_cfg(**kw), plan, seed=1, scale=scale, group=group)


def test_serving_shape_chunk_on_a_big_cache():
    """The "serving-like" chunk of the benchmark: a 512-token chunk on a W = 768, R = 512 cache with sink tokens,
    after a prompt, followed by decode steps."""
    _compare(_cfg(B=1, H=2, W=768, R=512, sink=4), [("prefill", 2000), ("chunk", 512), ("decode", 4)], seed=2)


@pytest.mark.parametrize("kw,plan", [
    (dict(B=1, H=2, W=768, R=512, sink=4), [("prefill", 2000), ("chunk", 512), ("decode", 4)]),   # the benchmark's serving-like chunk
    (dict(B=1, H=2, W=128, R=128), [("prefill", 1500), ("chunk", 1200)]),                          # the C2 window and budget: several retained tiles
    (dict(B=1, H=2, d=128, W=96, R=70), [("prefill", 700), ("chunk", 900), ("decode", 3)]),        # d = 128: the other tiled kernel
    (dict(B=2, H=2, d=32, W=48, R=40), [("prefill", 300), ("chunk", 500), ("decode", 3)]),         # d = 32: the d = 64 kernel on zero-filled columns
])
def test_streaming_reading_at_the_benchmark_shapes(kw, plan):
    """The streaming reading on the tiled tensor-core kernel (bf16, d = 64): retained tiles of the entry list with the leave
    times as one more mask; equal to token-by-token decoding."""
    _compare(_cfg(**kw), plan, seed=2, streaming=True)


def test_wrong_token_count_is_reported_and_leaves_the_cache_alone():
    cfg = _cfg(B=1, H=2)
    x = synth.make(cfg, 0, T=120)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = (dev(x[t], cfg.dtype) for t in "qkv")
    s = shape_of(cfg, T=80)
    z = lte.lte_scores(s, c, k[:, :, :80].contiguous(), v[:, :, :80].contiguous())
    idx, cnt = lte.lte_select(s, z)
    cache = lte.lte_cache_init(s, c, k[:, :, :80].contiguous(), v[:, :, :80].contiguous(), z, idx, cnt)
    before = cache.clone()
    s2 = shape_of(cfg, T=40)
    lte.lte_attn_prefill_chunk(s2, c, cache, 79, q[:, :, 80:].contiguous(), k[:, :, 80:].contiguous(), v[:, :, 80:].contiguous())
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() != 0
    assert torch.equal(before, cache)
    assert lte.lib().lte_device_status() == 0               # the status is cleared by reading it


def test_a_reported_mismatch_does_not_stop_the_next_call_from_committing():
    """A call that named the wrong token count is reported and leaves the cache alone; a correct call made after it,
    with the report still unread, must advance the cache as if nothing had happened (the report word is not a gate)."""
    cfg = _cfg(B=1, H=2)
    x = synth.make(cfg, 0, T=120)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = (dev(x[t], cfg.dtype) for t in "qkv")
    s = shape_of(cfg, T=80)
    z = lte.lte_scores(s, c, k[:, :, :80].contiguous(), v[:, :, :80].contiguous())
    idx, cnt = lte.lte_select(s, z)
    cache = lte.lte_cache_init(s, c, k[:, :, :80].contiguous(), v[:, :, :80].contiguous(), z, idx, cnt)
    good = cache.clone()
    s2 = shape_of(cfg, T=40)
    qc, kc, vc = (t[:, :, 80:].contiguous() for t in (q, k, v))
    lte.lte_attn_prefill_chunk(s2, c, cache, 79, qc, kc, vc)                  # wrong count: reported, cache untouched
    o1, l1 = lte.lte_attn_prefill_chunk(s2, c, cache, 80, qc, kc, vc)         # right count, report still unread
    o2, l2 = lte.lte_attn_prefill_chunk(s2, c, good, 80, qc, kc, vc)          # the same call on an untouched copy
    torch.cuda.synchronize()
    assert torch.equal(cache, good) and torch.equal(o1, o2) and torch.equal(l1, l2)
    _, ns = _read_pool(cache, cfg, cfg.B)
    assert all(n == 120 for n in ns)
    assert lte.lib().lte_device_status() != 0                                 # the first call's report is still there
    assert lte.lib().lte_device_status() == 0


@pytest.mark.parametrize("kw,plan,group", [
    (dict(), [("prefill", 200), ("chunk", 150), ("decode", 12)], 1),
    (dict(), [("prefill", 0), ("chunk", 100), ("chunk", 60), ("decode", 5)], 1),
    (dict(), [("prefill", 33), ("chunk", 5), ("chunk", 1), ("chunk", 300), ("decode", 4)], 1),
    (dict(sink=3, W=16, R=9), [("prefill", 40), ("decode", 7), ("chunk", 220)], 1),
    (dict(dtype="f32", d=32, W=16, R=8, K=5, B=1, H=2), [("prefill", 60), ("chunk", 90), ("decode", 6)], 1),
    (dict(d=128, W=40, R=30, B=1, H=2), [("prefill", 150), ("chunk", 140)], 1),
    (dict(W=64, R=40, B=1, H=2), [("prefill", 300), ("chunk", 260), ("decode", 3)], 3),
    (dict(W=32, R=0), [("prefill", 50), ("chunk", 90)], 1),
])
def test_streaming_reading_equals_token_by_token_decoding_with_a_binding_cap(kw, plan, group):
    """LTE_CHUNK_STREAMING: every chunk query sees the pool the replace-the-lowest rule holds at that query, so a chunk
    equals as many decode steps, also where the cap binds (about half of all tokens pass the threshold here and the
    budgets are small: entries are pushed out inside the chunk)."""
    _compare(_cfg(**kw), plan, seed=3, group=group, streaming=True)


def test_the_two_readings_differ_where_the_cap_binds_and_leave_the_same_cache():
    cfg = _cfg(B=1, H=2)
    plan = [("prefill", 200), ("chunk", 150)]
    x, a, cache_a = _run(cfg, plan, seed=3)
    _, b, cache_b = _run(cfg, plan, seed=3, streaming=True)
    assert np.max(np.abs(a[1][0] - b[1][0])) > 5e-2                  # an early query sees entries that leave later in the chunk
    pa, na = _read_pool(cache_a, cfg, cfg.B); pb, nb = _read_pool(cache_b, cfg, cfg.B)
    assert na == nb and all(np.array_equal(u, v) for u, v in zip(pa, pb))
    # the last query of the chunk sees the final pool under both readings
    assert np.max(np.abs(a[1][0][:, :, -1] - b[1][0][:, :, -1])) <= 2e-2
