"""GPU parity: lte_attn_prefill against the fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import check_idx, dev, shape_of

pytestmark = pytest.mark.gpu

TOL = {"bf16": 2e-2, "f32": 1e-4}


def _pipeline(cfg, seed=0, scale=0.0, batch=None, qpos=None, tau=0.5):
    """scores -> select -> prefill on the GPU; the oracle attends over the GPU's list once that list has
    passed the retained-list rule, so a legitimate threshold difference cannot leak into the O comparison."""
    x = synth.make(cfg, seed, batch=batch)
    B = x["k"].shape[0]
    s = shape_of(cfg, B=B, scale=scale, tau=tau)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = (dev(x[t], cfg.dtype) for t in "qkv")
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    torch.cuda.synchronize()
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    z64 = orc.scores(x["k"], x["v"], x["w"])
    check_idx(idx_n, cnt_n, z64, cfg.W, cfg.R, cfg.sink, tau)
    o64, l64 = orc.attn_prefill(x["q"], x["k"], x["v"], idx_n, cnt_n, cfg.W, None if scale == 0.0 else scale, qpos)
    o_n, l_n = o.float().cpu().numpy(), lse.cpu().numpy()
    if qpos is not None:
        o_n = np.take_along_axis(o_n, qpos[..., None].astype(np.int64), axis=2)
        l_n = np.take_along_axis(l_n, qpos.astype(np.int64), axis=2)
    return o_n, l_n, o64, l64


def _assert_close(cfg, res):
    o_n, l_n, o64, l64 = res
    assert np.all(np.isfinite(o_n)) and np.all(np.isfinite(l_n))
    assert np.max(np.abs(o_n - o64)) <= TOL[cfg.dtype], np.max(np.abs(o_n - o64))
    assert np.max(np.abs(l_n - l64)) <= TOL[cfg.dtype], np.max(np.abs(l_n - l64))


def test_config1_every_output():
    cfg = synth.CONFIGS["C1"]
    _assert_close(cfg, _pipeline(cfg, seed=0))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,K,T,W,R,sink", [
    (32, 1, 1, 1, 1, 0), (32, 3, 7, 3, 2, 0), (64, 5, 123, 16, 8, 2), (128, 7, 130, 9, 200, 0),
    (64, 7, 517, 40, 0, 0), (32, 13, 1000, 64, 33, 4), (64, 9, 300, 400, 16, 0), (128, 11, 259, 11, 5, 7),
    (64, 7, 700, 128, 128, 0), (128, 7, 1500, 512, 512, 0), (64, 7, 640, 64, 64, 0), (64, 7, 385, 129, 77, 1),
])
def test_odd_shapes(dtype, d, K, T, W, R, sink):
    cfg = synth.Config("odd", dtype, 2, 3, d, T, W, R, K, 0.1, sink=sink)
    _assert_close(cfg, _pipeline(cfg, seed=5))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sharp_softmax_and_threshold_off(dtype):
    cfg = synth.Config("sharp", dtype, 1, 4, 64, 600, 32, 48, 7, 0.1, qk_unit=True)
    _assert_close(cfg, _pipeline(cfg, seed=6, scale=1.0))
    _assert_close(cfg, _pipeline(cfg.with_(R=600), seed=6, tau=0.0))       # dense causal for scored far keys


def test_config2_full():
    cfg = synth.CONFIGS["C2"]
    _assert_close(cfg, _pipeline(cfg, seed=0))
    _assert_close(cfg, _pipeline(cfg.with_(B=1), seed=1, scale=1.0))


def test_config3_sampled_queries():
    cfg = synth.CONFIGS["C3"]
    qpos = synth.query_sample(cfg, 2048, seed=0)
    _assert_close(cfg, _pipeline(cfg, seed=0, qpos=qpos))


def test_serving_shape_with_sink():
    """The paper-like serving shape of the benchmark: W = 768, R = 512, 4 sink tokens (window of six key tiles, a list
    that is not full on every head because the sink entries take slots)."""
    cfg = synth.Config("serve", "bf16", 1, 2, 64, 4096, 768, 512, 7, 0.05, sink=4)
    _assert_close(cfg, _pipeline(cfg, seed=3))
    _assert_close(cfg.with_(d=128), _pipeline(cfg.with_(d=128, T=2500), seed=3))


def test_config5_forward():
    cfg = synth.CONFIGS["C5"]
    _assert_close(cfg, _pipeline(cfg, seed=0, batch=[0, 7]))


def test_persistent_schedule_ragged_many_items():
    """More work items than resident CTAs (each CTA walks several items), a last query tile that is ragged, lists
    longer than the prefetched 128 entries and sink tokens: covers the item-to-item hand-over of the persistent
    d = 64 kernel (Q buffer, accumulator, stage ring, prefetched list) on a shape unlike the benchmark's."""
    cfg = synth.Config("ragged", "bf16", 3, 8, 64, 2075, 96, 200, 7, 0.1, sink=3)
    assert 3 * 8 * ((2075 + 127) // 128) > 2 * 148
    _assert_close(cfg, _pipeline(cfg, seed=11))


def test_random_shapes_many_items():
    """Seeded random shapes with more work items than resident CTAs (d = 64: the persistent schedule; d = 128: one CTA
    per tile), windows and budgets of every relation to the tile sizes, with and without sink tokens."""
    rng = np.random.default_rng(77)
    for n in range(6):
        d = 64 if n % 3 else 128
        T = int(rng.integers(1500, 4200)) if d == 64 else int(rng.integers(300, 1400))
        cfg = synth.Config("rnd", "bf16", int(rng.integers(2, 5)), int(rng.integers(6, 13)), d, T,
                           int(rng.integers(16, 400)), int(rng.integers(0, 520)), 7, 0.1, sink=int(rng.integers(0, 5)))
        _assert_close(cfg, _pipeline(cfg, seed=100 + n))
    assert lte.lte_device_status() == 0


def test_zero_query_pins_set_sizes_on_gpu():
    cfg = synth.Config("q0", "bf16", 1, 2, 64, 900, 100, 60, 7, 0.1)
    x = synth.make(cfg, 2)
    s = shape_of(cfg)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    k, v = dev(x["k"], "bf16"), dev(x["v"], "bf16")
    idx, cnt = lte.lte_select(s, lte.lte_scores(s, c, k, v))
    o, lse = lte.lte_attn_prefill(s, torch.zeros_like(k), k, v, idx, cnt)
    idx_n, cnt_n = idx.cpu().numpy(), cnt.cpu().numpy()
    for h in range(2):
        kept = idx_n[0, h, :cnt_n[0, h]]
        sizes = np.array([min(i + 1, cfg.W) + np.sum(kept <= i - cfg.W) for i in range(cfg.T)])
        np.testing.assert_allclose(np.exp(lse[0, h].cpu().numpy()), sizes, rtol=1e-5)


def test_no_bounded_wait_expired():
    # runs after the cases above in this file: the tensor-core kernel's waits are bounded, and none gave up
    assert lte.lte_device_status() == 0


@pytest.mark.parametrize("dtype,d,T,W,R", [("bf16", 64, 1500, 96, 80, ), ("bf16", 128, 900, 64, 50), ("f32", 32, 400, 24, 30)])
def test_caller_made_list_uniform_stride(dtype, d, T, W, R):
    """The attention takes any ascending list: the training-free "uniform stride + sliding window" rule of the paper's
    ablation (Section 4, ablation paragraph) needs no scorer, the caller writes the list; heads may hold different counts."""
    cfg = synth.Config("unif", dtype, 2, 3, d, T, W, R, 7, 0.1)
    x = synth.make(cfg, 9)
    q, k, v = (dev(x[t], dtype) for t in "qkv")
    idx = np.full((cfg.B, cfg.H, R), -1, np.int32); cnt = np.zeros((cfg.B, cfg.H), np.int32)
    for b in range(cfg.B):
        for h in range(cfg.H):
            n = R - (b * cfg.H + h) * 3                                       # a different budget per head
            stride = max((T - W + n - 1) // n, 1)
            pos = np.arange(h % stride, T - W, stride, dtype=np.int32)[:n]    # out-of-window tokens at a uniform stride
            idx[b, h, :len(pos)] = pos; cnt[b, h] = len(pos)
    s = shape_of(cfg)
    o, lse = lte.lte_attn_prefill(s, q, k, v, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda())
    torch.cuda.synchronize()
    o64, l64 = orc.attn_prefill(x["q"], x["k"], x["v"], idx, cnt, W)
    _assert_close(cfg, (o.float().cpu().numpy(), lse.cpu().numpy(), o64, l64))


@pytest.mark.parametrize("d,T,W,R", [(64, 1100, 96, 200), (128, 900, 64, 130), (64, 300, 40, 0), (32, 700, 48, 90)])
def test_compacted_and_gathered_retained_rows_agree(d, T, W, R):
    """With a workspace the retained rows are compacted and fetched as tiles, without one they are gathered row by row:
    two kernels variants, the same numbers (bit for bit: the products and their order are the same)."""
    cfg = synth.Config("cmp", "bf16", 2, 3, d, T, W, R, 7, 0.1)
    x = synth.make(cfg, 12)
    s = shape_of(cfg)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v = (dev(x[t], "bf16") for t in "qkv")
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    need = lte.lte_workspace_bytes(lte.OP_PREFILL, s, None)
    assert need == (0 if R == 0 else 2 * ((cfg.B * cfg.H * R * d * 2 + 127) // 128 * 128))
    o1, l1 = lte.lte_attn_prefill(s, q, k, v, idx, cnt, ws=False)
    o2, l2 = lte.lte_attn_prefill(s, q, k, v, idx, cnt)                      # allocates the workspace
    ws = torch.empty(need + 128, dtype=torch.uint8, device="cuda")
    o3, l3 = lte.lte_attn_prefill(s, q, k, v, idx, cnt, ws=ws[64:64 + max(need, 1)] if need else False)   # misaligned: falls back to gathering
    torch.cuda.synchronize()
    assert lte.lib().lte_device_status() == 0
    assert torch.equal(o1, o2) and torch.equal(l1, l2) and torch.equal(o1, o3)


def test_second_device_after_the_first():
    """A process that drives two GPUs: the tiny fp32 configuration and a tensor-core shape on device 0, then on device 1
    (raised shared-memory limits, SM count and status words are per device).  Skipped unless two devices are visible."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible devices")
    for dev_id in (0, 1):
        with torch.cuda.device(dev_id):
            for cfg in (synth.CONFIGS["C1"], synth.Config("dev", "bf16", 1, 2, 64, 700, 64, 48, 7, 0.1)):
                _assert_close(cfg, _pipeline(cfg, seed=0))
            assert lte.lte_device_status() == 0
