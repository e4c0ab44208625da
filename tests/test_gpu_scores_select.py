"""GPU parity: lte_scores / lte_select against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import check_idx, dev, shape_of

pytestmark = pytest.mark.gpu


def _run(cfg, seed=0, bias=None, tau=0.5, batch=None):
    x = synth.make(cfg, seed, batch=batch)
    B = x["k"].shape[0]
    s = shape_of(cfg, B=B, tau=tau)
    w = torch.from_numpy(x["w"]).cuda()
    bt = None if bias is None else torch.from_numpy(bias.astype(np.float32)).cuda()
    c = lte.conv(w, bt)
    k, v = dev(x["k"], cfg.dtype), dev(x["v"], cfg.dtype)
    r = torch.empty((B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")
    z = lte.lte_scores(s, c, k, v, r=r)
    ncand = torch.empty((B, cfg.H), dtype=torch.int32, device="cuda")
    idx, cnt = lte.lte_select(s, z, ncand=ncand)
    torch.cuda.synchronize()
    z64 = orc.scores(x["k"], x["v"], x["w"], bias)
    return x, z.cpu().numpy(), r.cpu().numpy(), idx.cpu().numpy(), cnt.cpu().numpy(), ncand.cpu().numpy(), z64


def _check(cfg, out, tau=0.5):
    x, z, r, idx, cnt, ncand, z64 = out
    fin = np.isfinite(z64)
    assert np.array_equal(np.isneginf(z), ~fin)
    assert np.max(np.abs(z[fin] - z64[fin])) < 2e-5
    assert np.max(np.abs(r[fin] - 1 / (1 + np.exp(-z64[fin])))) < 1e-5 and np.all(r[~fin] == 0)
    check_idx(idx, cnt, z64, cfg.W, cfg.R, cfg.sink, tau)
    return out


def test_config1_scores_and_list():
    cfg = synth.CONFIGS["C1"]
    x, z, r, idx, cnt, ncand, z64 = _check(cfg, _run(cfg, seed=0))
    idx_o, cnt_o, nc_o = orc.select(z64, cfg.W, cfg.R)
    assert np.array_equal(idx, idx_o) and np.array_equal(cnt, cnt_o) and np.array_equal(ncand, nc_o)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,K,T,W,R,sink", [
    (32, 1, 1, 1, 1, 0), (32, 3, 7, 3, 2, 0), (64, 5, 123, 16, 8, 2), (128, 7, 130, 9, 200, 0),
    (64, 7, 517, 40, 0, 0), (32, 13, 1000, 64, 33, 4), (64, 9, 300, 400, 16, 0), (128, 11, 259, 11, 5, 7),
    (32, 7, 4000, 128, 128, 0), (32, 5, 777, 40, 30, 2),     # bf16: the d = 64 tensor-core kernel on zero-filled tile columns
])
def test_odd_shapes(dtype, d, K, T, W, R, sink):
    cfg = synth.Config("odd", dtype, 2, 3, d, T, W, R, K, 0.1, sink=sink)
    bias = np.array([0.25, -0.5, 0.0])
    _check(cfg, _run(cfg, seed=3, bias=bias))


def test_threshold_disabled_keeps_every_scored_token():
    cfg = synth.Config("tau0", "bf16", 1, 2, 64, 200, 16, 300, 5, 0.1)
    x, z, r, idx, cnt, ncand, z64 = _check(cfg, _run(cfg, tau=0.0), tau=0.0)
    assert np.all(cnt == cfg.T - cfg.W)


@pytest.mark.parametrize("name,batch", [("C2", None), ("C3", None), ("C5", [0, 5]), ("C4", [3])])
def test_benchmark_shapes(name, batch):
    cfg = synth.CONFIGS[name]
    x, z, r, idx, cnt, ncand, z64 = _check(cfg, _run(cfg, seed=0, batch=batch))
    assert np.all(cnt == cfg.R)          # with these weights about half the tokens pass: the cap binds


def test_select_exact_on_ties_and_ranks():
    # lte_select alone on hand-made logits with many exact ties: must equal the oracle bit for bit.
    rng = np.random.default_rng(0)
    for T, W, R, sink in [(50, 7, 5, 0), (4096, 128, 128, 0), (3000, 1, 2999, 3), (9000, 500, 1, 0), (40000, 512, 512, 4),
                          (20001, 100, 77, 2), (65000, 64, 4000, 0),   # these three and the next: a cluster of blocks per head
                          (16512, 128, 0, 0), (20000, 100, 25000, 1), (16384 + 64, 64, 3, 0)]:   # no budget; budget above the candidates; smallest N
        z = (np.round(rng.standard_normal((2, 3, T)) * 4) / 4).astype(np.float32)
        z[0, 0] = 1.0                      # all equal and positive: oldest R win
        z[0, 1] = -1.0                     # nothing passes
        z[1, 0] = np.arange(T)             # increasing: youngest eligible win
        s = lte.shape(2, 3, T, 32, W, R, lte.F32, sink=sink)
        nc = torch.empty((2, 3), dtype=torch.int32, device="cuda")
        idx, cnt = lte.lte_select(s, torch.from_numpy(z).cuda(), ncand=nc)
        idx_o, cnt_o, nc_o = orc.select(z, W, R, sink)
        assert np.array_equal(idx.cpu().numpy(), idx_o)
        assert np.array_equal(cnt.cpu().numpy(), cnt_o)
        assert np.array_equal(nc.cpu().numpy(), nc_o)


def test_deterministic():
    cfg = synth.CONFIGS["C2"].with_(B=1)
    a = _run(cfg, seed=1)
    b = _run(cfg, seed=1)
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[3], b[3])
