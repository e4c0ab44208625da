"""GPU parity with grouped-query attention (several query heads share a key/value head, its retained list and its
decode cache): lte_attn_prefill and lte_attn_decode against the oracle run per query head on repeated keys/values."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import assert_grad_close, dev, tdtype

pytestmark = pytest.mark.gpu

TOL = {"bf16": 2e-2, "f32": 1e-4}


def _inputs(cfg, G, seed, T=None):
    """k, v, w for cfg.H key/value heads; q for cfg.H * G query heads (query heads of one key/value head adjacent)."""
    x = synth.make(cfg, seed, T=T)
    xq = synth.make(cfg.with_(H=cfg.H * G), seed + 100, T=T)
    return x, xq["q"]


@pytest.mark.parametrize("dtype,d,T,W,R,G", [("bf16", 64, 700, 64, 48, 4), ("bf16", 64, 300, 32, 16, 2), ("bf16", 128, 520, 96, 64, 4),
                                             ("f32", 32, 200, 16, 12, 3), ("bf16", 32, 260, 24, 10, 2)])
def test_prefill_gqa(dtype, d, T, W, R, G):
    cfg = synth.Config("gqa", dtype, 2, 3, d, T, W, R, 7, 0.1, sink=1)
    x, q = _inputs(cfg, G, 11)
    s = lte.shape(cfg.B, cfg.H, T, d, W, R, tdtype(cfg), sink=cfg.sink, group=G)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    k, v = dev(x["k"], dtype), dev(x["v"], dtype)
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, dev(q, dtype), k, v, idx, cnt)
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    assert o.shape == (cfg.B, cfg.H * G, T, d) and lse.shape == (cfg.B, cfg.H * G, T)
    rep = lambda a: np.repeat(a, G, axis=1)
    o64, l64 = orc.attn_prefill(q, rep(x["k"]), rep(x["v"]), rep(idx.cpu().numpy()), rep(cnt.cpu().numpy()), W)
    assert np.max(np.abs(o.float().cpu().numpy() - o64)) <= TOL[dtype]
    assert np.max(np.abs(lse.cpu().numpy() - l64)) <= TOL[dtype]
    # group = 1 through the same entry point gives the plain result for the first query head of every group
    s1 = lte.shape(cfg.B, cfg.H, T, d, W, R, tdtype(cfg), sink=cfg.sink)
    o1, _ = lte.lte_attn_prefill(s1, dev(np.ascontiguousarray(q[:, ::G]), dtype), k, v, idx, cnt)
    assert torch.equal(o1, o[:, ::G].contiguous())


@pytest.mark.parametrize("dtype,d,W,R,G,T0,steps", [("bf16", 64, 32, 24, 4, 100, 40), ("bf16", 64, 16, 8, 2, 0, 60), ("bf16", 128, 24, 16, 4, 64, 30),
                                                    ("f32", 32, 16, 12, 3, 40, 30), ("bf16", 64, 200, 150, 2, 260, 20),
                                                    # few heads, long blocks: a cluster of blocks shares a head (2 x 320, 4 x 260 rows), 5 query heads = two passes
                                                    ("bf16", 64, 384, 256, 5, 700, 12), ("f32", 32, 600, 440, 2, 1300, 8), ("bf16", 128, 300, 220, 6, 10, 14)])
def test_decode_gqa(dtype, d, W, R, G, T0, steps):
    cfg = synth.Config("gqa", dtype, 2, 2, d, T0 + steps, W, R, 7, 0.1)
    Ttot = T0 + steps
    x, q = _inputs(cfg, G, 5, T=Ttot)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    k, v, qd = dev(x["k"], dtype), dev(x["v"], dtype), dev(q, dtype)
    s0 = lte.shape(cfg.B, cfg.H, T0, d, W, R, tdtype(cfg), group=G)
    if T0 > 0:
        kp, vp = k[:, :, :T0].contiguous(), v[:, :, :T0].contiguous()
        z = lte.lte_scores(s0, c, kp, vp)
        idx, cnt = lte.lte_select(s0, z)
        cache = lte.lte_cache_init(s0, c, kp, vp, z, idx, cnt)
    else:
        cache = lte.lte_cache_init(s0, c)
    outs, lses = [], []
    for n in range(T0, Ttot):
        o1, l1 = lte.lte_attn_decode(s0, c, cache, qd[:, :, n].contiguous(), k[:, :, n].contiguous(), v[:, :, n].contiguous())
        outs.append(o1.float().cpu().numpy()); lses.append(l1.cpu().numpy())
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    o_n, l_n = np.stack(outs, axis=2), np.stack(lses, axis=2)
    assert o_n.shape == (cfg.B, cfg.H * G, steps, d)
    rep = lambda a: np.repeat(a, G, axis=1)
    z64 = orc.scores(x["k"], x["v"], x["w"])
    o64, l64, _, _ = orc.stream(q, rep(x["k"]), rep(x["v"]), rep(z64), W, R, 0, n_from=T0)
    assert np.max(np.abs(o_n - o64)) <= TOL[dtype], np.max(np.abs(o_n - o64))
    assert np.max(np.abs(l_n - l64)) <= TOL[dtype]


@pytest.mark.parametrize("dtype,d,T,W,R,G,in_grad", [("bf16", 64, 300, 32, 24, 4, True), ("bf16", 128, 260, 48, 32, 2, True),
                                                     ("f32", 32, 150, 16, 10, 3, True), ("bf16", 64, 520, 64, 64, 2, False)])
def test_backward_gqa(dtype, d, T, W, R, G, in_grad):
    """dq per query head; dk, dv, dw, dbias summed over the query heads of a group.  Everything downstream of dV is linear
    in it (no Eq. 7 term here), so the reference is the oracle run per query head on repeated keys/values, summed."""
    cfg = synth.Config("gqa", dtype, 2, 2, d, T, W, R, 7, 0.1)
    x, q = _inputs(cfg, G, 21)
    dO = synth.make(cfg.with_(H=cfg.H * G), 321, with_dO=True)["dO"]
    s = lte.shape(cfg.B, cfg.H, T, d, W, R, tdtype(cfg), group=G)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    k, v, qd, gd = dev(x["k"], dtype), dev(x["v"], dtype), dev(q, dtype), dev(dO, dtype)
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, qd, k, v, idx, cnt)
    flags = lte.BWD_CNN_INPUT_GRAD if in_grad else 0
    dq, dk, dv, dw, db = lte.lte_attn_bwd(s, c, qd, k, v, o, lse, gd, z, idx, cnt, flags=flags)
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    rep = lambda a: np.repeat(a, G, axis=1)
    z64 = z.cpu().numpy().astype(np.float64)
    r = orc.attn_bwd(q, rep(x["k"]), rep(x["v"]), dO, rep(z64), rep(idx.cpu().numpy()), rep(cnt.cpu().numpy()),
                     np.repeat(x["w"], G, axis=0), W, cnn_input_grad=in_grad)
    grp = lambda a: a.reshape(a.shape[0], cfg.H, G, *a.shape[2:]).sum(axis=2)          # [B, H*G, ...] -> sum over the group
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    # each at three granularities: whole tensor, every 128-row block of every head, dk / dv on the retained rows alone
    assert_grad_close("dq", dq.float().cpu().numpy(), r["dq"], 5e-2)
    assert_grad_close("dk", dk.float().cpu().numpy(), grp(r["dk"]), 5e-2, idx_n, cnt_n)
    assert_grad_close("dv", dv.float().cpu().numpy(), grp(r["dv"]), 5e-2, idx_n, cnt_n)
    assert_grad_close("dw", dw.cpu().numpy(), r["dw"].reshape(cfg.H, G, *r["dw"].shape[1:]).sum(axis=1), 5e-2)
    assert_grad_close("dbias", db.cpu().numpy(), r["dbias"].reshape(cfg.H, G).sum(axis=1), 5e-2)
