"""GPU parity: the three-layer scorer stack of lte_scores against the fp64 oracle, and the selection that follows."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import check_idx, dev, shape_of

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


def test_stack_rejected_elsewhere():
    """decode, cache_init and the backward take the single layer only."""
    cfg = synth.Config("stack", "bf16", 1, 2, 64, 64, 16, 8, 7, 0.1)
    wl, wout, bl, bout = _stack_params(cfg.H, 64, 1, False)
    c = lte.conv_stack([torch.from_numpy(w).cuda() for w in wl], torch.from_numpy(wout).cuda())
    s = shape_of(cfg, B=1)
    x = synth.make(cfg, 0)
    k, v = dev(x["k"], "bf16"), dev(x["v"], "bf16")
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    with pytest.raises(Exception):
        lte.lte_cache_init(s, c, k, v, z, idx, cnt)
