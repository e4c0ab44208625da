"""GPU parity: lte_attn_bwd against the fp64 oracle gradients, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import assert_grad_close, check_idx, dev, shape_of

pytestmark = pytest.mark.gpu

REL = {"bf16": 5e-2, "f32": 1e-4}


def _bwd(cfg, seed=0, batch=None, flags=lte.BWD_CNN_INPUT_GRAD, lam=None, bias=None, scale=0.0):
    x = synth.make(cfg, seed, batch=batch, with_dO=True)
    B = x["k"].shape[0]
    s = shape_of(cfg, B=B, scale=scale)
    bt = None if bias is None else torch.from_numpy(bias.astype(np.float32)).cuda()
    c = lte.conv(torch.from_numpy(x["w"]).cuda(), bt)
    q, k, v, dO = (dev(x[t], cfg.dtype) for t in ("q", "k", "v", "dO"))
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    lt = None if lam is None else torch.from_numpy(lam.astype(np.float32)).cuda()
    dq, dk, dv, dw, db = lte.lte_attn_bwd(s, c, q, k, v, o, lse, dO, z, idx, cnt, lam=lt, flags=flags)
    torch.cuda.synchronize()
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    z64 = orc.scores(x["k"], x["v"], x["w"], bias)
    check_idx(idx_n, cnt_n, z64, cfg.W, cfg.R, cfg.sink)
    g = orc.attn_bwd(x["q"], x["k"], x["v"], x["dO"], z64, idx_n, cnt_n, x["w"], cfg.W,
                     None if scale == 0.0 else scale, lam=lam, cnn_input_grad=bool(flags & 1))
    got = dict(dq=dq, dk=dk, dv=dv, dw=dw, dbias=db)
    res = {n: (t.float().cpu().numpy(), g[n]) for n, t in got.items()}
    res["_list"] = (idx_n, cnt_n)
    return res


def _assert(cfg, res):
    idx_n, cnt_n = res["_list"]
    for name, (a, b) in res.items():
        if name == "_list":
            continue
        # whole tensor, every 128-row block of every (b,h), and for dk, dv the retained rows of every (b,h) alone
        assert_grad_close(name, a, b, REL[cfg.dtype], *((idx_n, cnt_n) if name in ("dk", "dv") else ()))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,K,T,W,R,sink", [(32, 5, 128, 16, 8, 0), (64, 7, 300, 40, 25, 2), (128, 3, 130, 9, 200, 0),
                                            (64, 7, 260, 300, 10, 0), (32, 1, 50, 4, 0, 0), (64, 13, 777, 64, 64, 0),
                                            (32, 7, 900, 64, 150, 1), (32, 9, 700, 100, 40, 0)])   # bf16 d = 32: the d = 64 tensor-core kernels on zero-filled columns
@pytest.mark.parametrize("flags", [0, 1])
def test_small_shapes(dtype, d, K, T, W, R, sink, flags):
    cfg = synth.Config("bwd", dtype, 2, 3, d, T, W, R, K, 0.1, sink=sink, qk_unit=(dtype == "f32"))
    _assert(cfg, _bwd(cfg, seed=7, flags=flags, lam=np.array([0.5, 0.0, 0.1]), bias=np.array([0.1, -0.2, 0.0])))


def test_config5_two_sequences():
    cfg = synth.CONFIGS["C5"]
    _assert(cfg, _bwd(cfg, seed=0, batch=[0, 6]))
    _assert(cfg, _bwd(cfg, seed=0, batch=[3], flags=0))


def test_config5_full_batch_weight_gradient():
    cfg = synth.CONFIGS["C5"]
    _assert(cfg, _bwd(cfg, seed=0))


def test_deterministic():
    cfg = synth.CONFIGS["C5"].with_(B=1)
    a = _bwd(cfg, seed=1)
    b = _bwd(cfg, seed=1)
    for n in a:
        assert np.array_equal(a[n][0], b[n][0])


@pytest.mark.parametrize("d,T,W,R", [(128, 9000, 64, 200), (64, 4500, 100, 130)])
def test_long_sequence_two_retained_tiles(d, T, W, R):
    # thousands of tokens: a retained tile walks many query blocks (the double-buffered products at d = 128 and the
    # stage ring wrap many times), and the list spans two tiles, the second one partly filled
    cfg = synth.Config("bwdlong", "bf16", 1, 2, d, T, W, R, 7, 0.05)
    _assert(cfg, _bwd(cfg, seed=3))


def test_long_prefill_shape_four_retained_tiles():
    # the long-context shape of the benchmark (d = 128, W = R = 512) at a length the oracle finishes in seconds: four
    # full retained tiles of 128 rows, each walking every later query block; window tiles wider than a key tile
    cfg = synth.Config("bwdc3", "bf16", 1, 2, 128, 3300, 512, 512, 7, 0.05)
    res = _bwd(cfg, seed=4)
    assert np.all(res["_list"][1] == 512)
    _assert(cfg, res)


@pytest.mark.parametrize("B,H,T,W,R,sink", [
    (1, 1, 100, 64, 20, 0),         # a single ragged tile
    (2, 3, 129, 64, 200, 0),        # second tile of one row; list longer than the sequence allows
    (3, 5, 1000, 33, 300, 2),       # several list chunks per tile, sink tokens, a window that is no multiple of anything
    (7, 23, 640, 64, 64, 0),        # more (head, tile) pairs than SMs: a thread block's run crosses heads and starts inside one
    (2, 2, 520, 7, 40, 0),          # the narrowest window the scorer allows
    (2, 2, 700, 9, 0, 0),           # no list at all
    (1, 2, 4100, 64, 700, 0),       # eleven list chunks: the chunk ring wraps inside an item
])
def test_short_window_shapes(B, H, T, W, R, sink):
    """bf16, d = 64, windows of at most one key tile (the training shape's regime): ragged tiles, lists longer than a tile,
    more (head, tile) pairs than SMs, sink tokens, no list at all."""
    cfg = synth.Config("fused", "bf16", B, H, 64, T, W, R, 7, 0.1, sink=sink)
    _assert(cfg, _bwd(cfg, seed=9, lam=np.linspace(0.0, 0.5, H), scale=0.0))
    assert lte.lte_device_status() == 0
