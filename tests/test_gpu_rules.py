"""GPU parity: the training-free selection rules behind lte_select_rule and the accumulated attention of lte_attn_colsum,
against the oracle (Section 4, ablation: uniform stride + window; ranking by accumulated attention)."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import dev, shape_of, tdtype

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,W,R,sink", [(30, 6, 7, 2), (30, 6, 30, 2), (30, 6, 3, 2), (5, 8, 4, 0), (4096, 128, 128, 0), (1000, 64, 0, 3),
                                        (777, 100, 50, 60), (2048, 768, 256, 4)])
def test_uniform_stride_lists_are_the_oracles(T, W, R, sink):
    s = lte.shape(2, 3, T, 64, W, R, lte.BF16, sink=sink)
    ncand = torch.empty((2, 3), dtype=torch.int32, device="cuda")
    idx, cnt = lte.lte_select_rule(s, lte.RULE_UNIFORM, ncand=ncand)
    torch.cuda.synchronize()
    idx_o, cnt_o = orc.select_uniform(2, 3, T, W, R, sink)
    assert np.array_equal(idx.cpu().numpy(), idx_o) and np.array_equal(cnt.cpu().numpy(), cnt_o)
    assert np.all(ncand.cpu().numpy() == max(T - W, 0))


@pytest.mark.parametrize("dtype,d,T,W,R,G", [("bf16", 64, 300, 32, 24, 1), ("f32", 32, 150, 16, 10, 1), ("bf16", 128, 260, 48, 300, 1),
                                             ("bf16", 64, 200, 24, 16, 3)])
def test_accumulated_attention_and_its_ranking(dtype, d, T, W, R, G):
    cfg = synth.Config("rules", dtype, 2, 2, d, T, W, R, 7, 0.1)
    x = synth.make(cfg, 3)
    qx = synth.make(cfg.with_(H=cfg.H * G), 103)["q"] if G > 1 else x["q"]
    s = lte.shape(cfg.B, cfg.H, T, d, W, R, tdtype(cfg), group=G)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = dev(qx, dtype), dev(x["k"], dtype), dev(x["v"], dtype)
    idx, cnt = lte.lte_select(s, lte.lte_scores(s, c, k, v))
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    a = lte.lte_attn_colsum(s, q, k, lse, idx, cnt)
    torch.cuda.synchronize()
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    rep = lambda t: np.repeat(t, G, axis=1)
    a64 = orc.attn_colsum(qx, rep(x["k"]), rep(idx_n), rep(cnt_n), W)
    a64 = a64.reshape(cfg.B, cfg.H, G, T).sum(axis=2)                       # accumulated over the query heads of a group
    a_n = a.cpu().numpy()
    # the kernel uses the GPU's own logsumexp (bf16 operands, fp32 accumulation): relative agreement per key
    assert np.max(np.abs(a_n - a64) / (a64 + 1e-3)) <= (2e-2 if dtype == "bf16" else 1e-4)
    np.testing.assert_allclose(a_n.sum(axis=-1), T * G, rtol=2e-3 if dtype == "bf16" else 1e-5)
    # the rule: top-R of the GPU's own a (exact on those values), every out-of-window token a candidate
    idx2, cnt2 = lte.lte_select_rule(s, lte.RULE_ACCUM_ATTN, a)
    idx_o, cnt_o = orc.select_rule(orc.RULE_ACCUM_ATTN, a_n.astype(np.float64), T, W, R)
    assert np.array_equal(idx2.cpu().numpy(), idx_o) and np.array_equal(cnt2.cpu().numpy(), cnt_o)
    assert np.all(cnt_o == min(R, max(T - W, 0)))
    # and the learned rule through the same entry point is lte_select
    z = lte.lte_scores(s, c, k, v)
    i3, c3 = lte.lte_select_rule(s, lte.RULE_LEARNED, z)
    assert torch.equal(i3, idx) and torch.equal(c3, cnt)
