"""GPU parity: the three-layer scorer stack of lte_scores against the fp64 oracle, and the selection that follows."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import assert_grad_close, check_idx, dev, shape_of

pytestmark = pytest.mark.gpu


def _stack_params(H, d, seed, with_bias):
    rng = np.random.default_rng([seed, 77])
    ch = [2 * d, d, d // 2, d // 4]
    wl = [(rng.standard_normal((H, ch[l + 1], 3, ch[l])) * (1.5 / np.sqrt(3 * ch[l]))).astype(np.float32) for l in range(3)]
    wout = (rng.standard_normal((H, ch[3])) * (2.0 / np.sqrt(ch[3]))).astype(np.float32)
    bl = [(rng.standard_normal((H, ch[l + 1])) * 0.1).astype(np.float32) for l in range(3)] if with_bias else [None] * 3
    bout = (rng.standard_normal((H,)) * 0.1).astype(np.float32) if with_bias else None
    return wl, wout, bl, bout


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,T,W,R,bias", [(64, 300, 16, 20, True), (32, 131, 9, 6, False), (64, 64, 7, 4, True),
                                          (32, 5, 7, 2, True), (64, 1000, 40, 50, False)])
def test_stack_logits_and_selection(dtype, d, T, W, R, bias):
    cfg = synth.Config("stack", dtype, 2, 3, d, T, W, R, 7, 0.1)
    x = synth.make(cfg, 3)
    wl, wout, bl, bout = _stack_params(cfg.H, d, 3, bias)
    z64 = orc.scores_stack(x["k"], x["v"], wl, bl, wout, bout)
    s = shape_of(cfg, B=cfg.B)
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl] if bias else None, t(bout))
    k, v = dev(x["k"], dtype), dev(x["v"], dtype)
    z = lte.lte_scores(s, c, k, v)
    torch.cuda.synchronize()
    zn = z.cpu().numpy().astype(np.float64)
    fin = np.isfinite(z64)
    assert np.array_equal(np.isfinite(zn), fin)                      # the unscored tail (last 6 positions) is -inf on both sides
    assert fin[..., : max(T - 6, 0)].all() and not fin[..., max(T - 6, 0):].any()
    if fin.any():
        assert np.max(np.abs(zn[fin] - z64[fin])) <= 2e-5 * max(1.0, np.max(np.abs(z64[fin])))
    idx, cnt = lte.lte_select(s, z)
    torch.cuda.synchronize()
    check_idx(idx.cpu().numpy(), cnt.cpu().numpy(), z64, W, R, 0, 0.5)


@pytest.mark.parametrize("B,H,T,bias,d", [(1, 1, 13, True, 64), (2, 2, 126, False, 64), (1, 2, 127, True, 64), (2, 1, 246, True, 64),
                                          (1, 3, 247, False, 64), (3, 20, 500, True, 64), (4, 16, 4096, True, 64),
                                          (2, 3, 300, True, 32), (1, 2, 127, False, 32), (4, 16, 2048, True, 32)])
def test_stack_tensor_core_path(B, H, T, bias, d):
    """bf16, d = 64 or 32 with a workspace: the tensor-core kernel (three-way split operands; d = 32 as the d = 64 problem
    with zero channels).  Tile edges (120 logits per tile), several heads per thread block and several thread blocks per
    head; the same call without a workspace runs the fp32 kernel, and both have to agree with the oracle."""
    cfg = synth.Config("stack", "bf16", B, H, d, T, 8, 12, 7, 0.1)
    x = synth.make(cfg, 5)
    wl, wout, bl, bout = _stack_params(H, d, 5, bias)
    z64 = orc.scores_stack(x["k"], x["v"], wl, bl, wout, bout)
    s = shape_of(cfg, B=B)
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl] if bias else None, t(bout))
    k, v = dev(x["k"], "bf16"), dev(x["v"], "bf16")
    need = lte.lte_workspace_bytes(lte.OP_SCORES, s, c)
    assert need == H * 194176
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    r = torch.empty((B, H, T), dtype=torch.float32, device="cuda")
    fin = np.isfinite(z64)
    tol = 2e-5 * max(1.0, np.max(np.abs(z64[fin])))
    for rep in range(2):                                             # twice: the kernel's barriers and the workspace are reusable
        z = lte.lte_scores(s, c, k, v, r=r, ws=ws)
        torch.cuda.synchronize()
        assert lte.lib().lte_device_status() == 0
        zn = z.cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isfinite(zn), fin) and np.all(np.isneginf(zn[~fin]))
        assert np.max(np.abs(zn[fin] - z64[fin])) <= tol
        rn = r.cpu().numpy()
        assert np.max(np.abs(rn[fin] - 1 / (1 + np.exp(-z64[fin])))) < 1e-5 and np.all(rn[~fin] == 0)
    z32 = lte.lte_scores(s, c, k, v, ws=False).cpu().numpy().astype(np.float64)     # no workspace: the fp32 kernel
    assert np.max(np.abs(z32[fin] - z64[fin])) <= tol
    idx, cnt = lte.lte_select(s, z)
    torch.cuda.synchronize()
    check_idx(idx.cpu().numpy(), cnt.cpu().numpy(), z64, cfg.W, cfg.R, 0, 0.5)


@pytest.mark.parametrize("dtype,d,W,R,T0,steps,period", [("bf16", 64, 32, 24, 100, 90, 19), ("bf16", 64, 40, 16, 0, 120, 27),
                                                         ("f32", 32, 24, 12, 30, 70, 5), ("bf16", 64, 128, 64, 300, 150, 115)])
def test_stack_in_decode(dtype, d, W, R, T0, steps, period):
    """Prefill with the stack, then decode: the step scores nothing, lte_cache_score runs every `period` <= W - 13 steps
    (lazy batches), and outputs and the final pool equal the oracle's streaming simulation on the stack's logits."""
    cfg = synth.Config("stackdec", dtype, 2, 2, d, T0 + steps, W, R, 7, 0.1)
    Ttot = T0 + steps
    x = synth.make(cfg, 4, T=Ttot)
    wl, wout, bl, bout = _stack_params(cfg.H, d, 4, True)
    t = lambda a: torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl], t(bout))
    q, k, v = (dev(x[n], dtype) for n in "qkv")
    s0 = shape_of(cfg, T=T0, B=cfg.B)
    if T0 > 0:
        kp, vp = k[:, :, :T0].contiguous(), v[:, :, :T0].contiguous()
        z = lte.lte_scores(s0, c, kp, vp)
        idx, cnt = lte.lte_select(s0, z)
        cache = lte.lte_cache_init(s0, c, kp, vp, z, idx, cnt)
    else:
        cache = lte.lte_cache_init(s0, c)
    outs, lses = [], []
    for i, n in enumerate(range(T0, Ttot)):
        if i % period == 0:
            lte.lte_cache_score(s0, c, cache)
        o1, l1 = lte.lte_attn_decode(s0, c, cache, q[:, :, n].contiguous(), k[:, :, n].contiguous(), v[:, :, n].contiguous())
        outs.append(o1.float().cpu().numpy()); lses.append(l1.cpu().numpy())
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    z64 = orc.scores_stack(x["k"], x["v"], wl, bl, wout, bout)
    o64, l64, pidx, pcnt = orc.stream(x["q"], x["k"], x["v"], z64, W, R, 0, n_from=T0)
    tol = 2e-2 if dtype == "bf16" else 1e-4
    assert np.max(np.abs(np.stack(outs, axis=2) - o64)) <= tol
    assert np.max(np.abs(np.stack(lses, axis=2) - l64)) <= tol
    from tests.test_gpu_decode import _read_pool
    pools, ns = _read_pool(cache, cfg, cfg.B)
    assert all(n == Ttot for n in ns)
    for bh, pool in enumerate(pools):
        b, h = divmod(bh, cfg.H)
        assert np.array_equal(pool, pidx[b, h, :pcnt[b, h]])


@pytest.mark.parametrize("dtype,d,W,R,T0,dec,Tc", [("bf16", 64, 32, 24, 100, 20, 90), ("f32", 32, 24, 12, 0, 0, 70), ("bf16", 64, 64, 40, 30, 50, 200)])
def test_stack_in_chunked_prefill(dtype, d, W, R, T0, dec, Tc):
    """Prefill with the stack, decode with lazy scoring, then a chunk on top of the cache: ring tokens the lazy scoring has
    not reached are scored with the chunk as right context; outputs equal the oracle's chunk-end reading on the stack's
    logits, and decode steps continue from the cache the chunk leaves."""
    cfg = synth.Config("stackchunk", dtype, 2, 2, d, 0, W, R, 7, 0.1)
    n0, Ttot = T0 + dec, T0 + dec + Tc + 8
    x = synth.make(cfg, 6, T=Ttot)
    wl, wout, bl, bout = _stack_params(cfg.H, d, 6, True)
    t = lambda a: torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl], t(bout))
    q, k, v = (dev(x[n], dtype) for n in "qkv")
    s0 = shape_of(cfg, T=T0, B=cfg.B)
    if T0 > 0:
        kp, vp = k[:, :, :T0].contiguous(), v[:, :, :T0].contiguous()
        z = lte.lte_scores(s0, c, kp, vp)
        idx, cnt = lte.lte_select(s0, z)
        cache = lte.lte_cache_init(s0, c, kp, vp, z, idx, cnt)
    else:
        cache = lte.lte_cache_init(s0, c)
    period = W - 13
    for i, n in enumerate(range(T0, n0)):
        if i % period == 0:
            lte.lte_cache_score(s0, c, cache)
        lte.lte_attn_decode(s0, c, cache, q[:, :, n].contiguous(), k[:, :, n].contiguous(), v[:, :, n].contiguous())
    sc = shape_of(cfg, T=Tc, B=cfg.B)
    o, l = lte.lte_attn_prefill_chunk(sc, c, cache, n0, q[:, :, n0:n0 + Tc].contiguous(), k[:, :, n0:n0 + Tc].contiguous(),
                                      v[:, :, n0:n0 + Tc].contiguous())
    outs, lses = [], []
    for i, n in enumerate(range(n0 + Tc, Ttot)):
        if i % period == 0:
            lte.lte_cache_score(s0, c, cache)
        o1, l1 = lte.lte_attn_decode(s0, c, cache, q[:, :, n].contiguous(), k[:, :, n].contiguous(), v[:, :, n].contiguous())
        outs.append(o1.float().cpu().numpy()); lses.append(l1.cpu().numpy())
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    z64 = orc.scores_stack(x["k"], x["v"], wl, bl, wout, bout)
    if n0 > 0:
        p_idx, p_cnt, _ = orc.select(z64[:, :, :n0], W, R)
    else:
        p_idx, p_cnt = np.full((cfg.B, cfg.H, R), -1, np.int32), np.zeros((cfg.B, cfg.H), np.int32)
    n1 = n0 + Tc
    o64, l64, _, _ = orc.prefill_chunk(x["q"][:, :, :n1], x["k"][:, :, :n1], x["v"][:, :, :n1], z64, n0, W, R, p_idx, p_cnt)
    tol = 2e-2 if dtype == "bf16" else 1e-4
    assert np.max(np.abs(o.float().cpu().numpy() - o64)) <= tol
    assert np.max(np.abs(l.cpu().numpy() - l64)) <= tol
    od, ld, pidx, pcnt = orc.stream(x["q"], x["k"], x["v"], z64, W, R, 0, n_from=n1)
    assert np.max(np.abs(np.stack(outs, axis=2) - od)) <= tol
    assert np.max(np.abs(np.stack(lses, axis=2) - ld)) <= tol
    from tests.test_gpu_decode import _read_pool
    pools, ns = _read_pool(cache, cfg, cfg.B)
    assert all(n == Ttot for n in ns)
    for bh, pool in enumerate(pools):
        b, h = divmod(bh, cfg.H)
        assert np.array_equal(pool, pidx[b, h, :pcnt[b, h]])


@pytest.mark.parametrize("dtype,d,W,R,T0,steps,period", [("bf16", 64, 32, 24, 100, 60, 19), ("f32", 32, 24, 12, 0, 70, 11), ("bf16", 64, 64, 30, 200, 90, 40)])
def test_stack_decode_with_rotated_keys(dtype, d, W, R, T0, steps, period):
    """The cache holds keys with a rotary position embedding, the scorer wants them without: the prompt is scored on the
    un-rotated keys, and lte_cache_score_unrope rotates the ring's keys back before the lazy batches of the decode."""
    cfg = synth.Config("stackrope", dtype, 2, 2, d, T0 + steps, W, R, 7, 0.1)
    Ttot = T0 + steps
    x = synth.make(cfg, 8, T=Ttot)
    wl, wout, bl, bout = _stack_params(cfg.H, d, 8, True)
    t = lambda a: torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl], t(bout))
    cos, sin = (a.astype(np.float32) for a in orc.rope_tables(Ttot, d))
    rnd = synth.round_bf16 if dtype == "bf16" else (lambda a: a.astype(np.float32))
    kr = rnd(orc.rope(x["k"], cos, sin).astype(np.float32))                 # what the cache holds
    q, k0, krd, v = dev(x["q"], dtype), dev(x["k"], dtype), dev(kr, dtype), dev(x["v"], dtype)
    s0 = shape_of(cfg, T=T0, B=cfg.B)
    if T0 > 0:
        z = lte.lte_scores(s0, c, k0[:, :, :T0].contiguous(), v[:, :, :T0].contiguous())      # the prompt: un-rotated keys
        idx, cnt = lte.lte_select(s0, z)
        cache = lte.lte_cache_init(s0, c, krd[:, :, :T0].contiguous(), v[:, :, :T0].contiguous(), z, idx, cnt)
    else:
        cache = lte.lte_cache_init(s0, c)
    outs, lses = [], []
    for i, n in enumerate(range(T0, Ttot)):
        if i % period == 0:
            lte.lte_cache_score_unrope(s0, c, cache, t(cos), t(sin))
        o1, l1 = lte.lte_attn_decode(s0, c, cache, q[:, :, n].contiguous(), krd[:, :, n].contiguous(), v[:, :, n].contiguous())
        outs.append(o1.float().cpu().numpy()); lses.append(l1.cpu().numpy())
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    ku = rnd(orc.rope(kr, cos, sin, inverse=True).astype(np.float32))        # the keys the lazy batches see (storage precision)
    za = orc.scores_stack(x["k"], x["v"], wl, bl, wout, bout)
    zb = orc.scores_stack(ku, x["v"], wl, bl, wout, bout)
    z64 = np.where(np.arange(Ttot)[None, None, :] <= T0 - 1 - 6, za, zb)
    o64, l64, pidx, pcnt = orc.stream(x["q"], kr, x["v"], z64, W, R, 0, n_from=T0)
    tol = 2e-2 if dtype == "bf16" else 1e-4
    assert np.max(np.abs(np.stack(outs, axis=2) - o64)) <= tol
    assert np.max(np.abs(np.stack(lses, axis=2) - l64)) <= tol
    from tests.test_gpu_decode import _read_pool
    pools, ns = _read_pool(cache, cfg, cfg.B)
    for bh, pool in enumerate(pools):
        b, h = divmod(bh, cfg.H)
        assert np.array_equal(pool, pidx[b, h, :pcnt[b, h]])
    # tables that do not reach the newest position are reported, not silently applied
    lte.lte_cache_score_unrope(s0, c, cache, t(cos[:Ttot - 5]), t(sin[:Ttot - 5]))
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() != 0


# ---- backward through the stack (lte_attn_bwd with the three-layer scorer) ---------------------------------------------
def _rel(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / (np.linalg.norm(b) + 1e-30))


@pytest.mark.parametrize("dtype,T,W,R,bias,in_grad,B,H,d", [("bf16", 200, 16, 12, True, True, 2, 2, 64), ("bf16", 333, 24, 40, False, True, 2, 2, 64),
                                                            ("f32", 150, 16, 10, True, True, 2, 2, 64), ("bf16", 260, 32, 16, True, False, 2, 2, 64),
                                                            ("bf16", 2048, 64, 64, True, True, 5, 8, 64), ("bf16", 700, 64, 32, True, True, 40, 8, 64),
                                                            ("f32", 150, 16, 10, True, True, 2, 2, 32), ("bf16", 333, 24, 40, True, True, 2, 3, 32),
                                                            ("f32", 700, 32, 16, False, False, 3, 2, 32)])
def test_stack_backward(dtype, T, W, R, bias, in_grad, B, H, d):
    """dq, dk, dv and the gradients of every parameter of the stack against the oracle: the attention backward and the
    straight-through surrogate give dz, the stack's backward (pinned by finite differences on the CPU) the rest.  d = 32 takes
    the fp32 kernels for the attention part and for the stack."""
    cfg = synth.Config("stackbwd", dtype, B, H, d, T, W, R, 7, 0.1)   # the last two: several tiles per thread block
    x = synth.make(cfg, 8, with_dO=True)
    wl, wout, bl, bout = _stack_params(cfg.H, d, 8, bias)
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    c = lte.conv_stack([t(w) for w in wl], t(wout), [t(b) for b in bl] if bias else None, t(bout))
    s = shape_of(cfg, B=cfg.B)
    q, k, v, dO = (dev(x[n], dtype) for n in ("q", "k", "v", "dO"))
    z = lte.lte_scores(s, c, k, v, ws=False)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    flags = lte.BWD_CNN_INPUT_GRAD if in_grad else 0
    dq, dk, dv, dw, db = lte.lte_attn_bwd(s, c, q, k, v, o, lse, dO, z, idx, cnt, flags=flags)
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    # oracle: same logits, same list; the single-layer weight argument only sets the width of the undefined tail (13 taps)
    z64 = z.cpu().numpy().astype(np.float64)
    w13 = np.zeros((cfg.H, 13, 2 * d))
    ra = orc.attn_bwd(x["q"], x["k"], x["v"], x["dO"], z64, idx.cpu().numpy(), cnt.cpu().numpy(), w13, W, cnn_input_grad=False)
    rs = orc.scores_stack_bwd(x["k"], x["v"], wl, bl, wout, bout, ra["dz"])
    dk64 = ra["dk"] + (rs["dk"] if in_grad else 0.0)
    dv64 = ra["dv"] + (rs["dv"] if in_grad else 0.0)
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    assert_grad_close("dq", dq.float().cpu().numpy(), ra["dq"], 5e-2)
    assert_grad_close("dk", dk.float().cpu().numpy(), dk64, 5e-2, idx_n, cnt_n)
    assert_grad_close("dv", dv.float().cpu().numpy(), dv64, 5e-2, idx_n, cnt_n)
    dwl, dwout, dbl, dbout = lte.unpack_stack_grads(cfg.H, d, dw, db)
    for l in range(3):                                               # per head as well as per tensor
        assert_grad_close("dwl%d" % l, dwl[l].cpu().numpy(), rs["dwl"][l], 5e-2)
        assert_grad_close("dbl%d" % l, dbl[l].cpu().numpy(), rs["dbl"][l], 5e-2)
    assert_grad_close("dwout", dwout.cpu().numpy(), rs["dwout"], 5e-2)
    assert _rel(dbout.cpu().numpy(), rs["dbout"]) < 5e-2
    if dtype == "f32":                                               # fp32 storage: the scorer's part is exact to rounding
        for l in range(3):
            assert _rel(dwl[l].cpu().numpy(), rs["dwl"][l]) < 1e-4
