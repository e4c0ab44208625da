"""The calls of the hot path inside a CUDA graph: they allocate nothing, synchronise nothing and keep no per-call host state,
so a captured step (scores, select, prefill attention, backward) replays on new inputs written into the same buffers and
gives what the same calls give when made directly."""
import numpy as np
import pytest
import torch

from paper_2510_20787_b200 import lte, synth
from gpu_util import dev, shape_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d,T,W,R", [("bf16", 64, 700, 64, 48), ("bf16", 128, 520, 40, 60), ("f32", 32, 200, 16, 12)])
def test_a_captured_step_replays_on_new_inputs(dtype, d, T, W, R):
    cfg = synth.Config("graph", dtype, 2, 3, d, T, W, R, 7, 0.1)
    xs = [synth.make(cfg, seed, with_dO=True) for seed in (0, 1)]
    s = shape_of(cfg)
    c = lte.conv(torch.from_numpy(xs[0]["w"]).cuda())
    q, k, v, dO = (dev(xs[0][n], dtype) for n in ("q", "k", "v", "dO"))
    z = torch.empty((cfg.B, cfg.H, T), dtype=torch.float32, device="cuda")
    idx = torch.empty((cfg.B, cfg.H, R), dtype=torch.int32, device="cuda")
    cnt = torch.empty((cfg.B, cfg.H), dtype=torch.int32, device="cuda")
    o = torch.empty_like(q); lse = torch.empty((cfg.B, cfg.H, T), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    dw = torch.empty((cfg.H, 7, 2 * d), dtype=torch.float32, device="cuda"); db = torch.empty((cfg.H,), dtype=torch.float32, device="cuda")
    need = lte.lte_workspace_bytes(lte.OP_PREFILL, s, None)
    ws_p = torch.empty(max(need, 1), dtype=torch.uint8, device="cuda") if need else False

    def step():
        lte.lte_scores(s, c, k, v, z=z)
        lte.lte_select(s, z, idx=idx, cnt=cnt)
        lte.lte_attn_prefill(s, q, k, v, idx, cnt, o=o, lse=lse, ws=ws_p)
        lte.lte_attn_bwd_static(s, c, q, k, v, o, lse, dO, z, idx, cnt, outs=(dq, dk, dv, dw, db))   # caller-owned outputs, built-in scratch

    outs = (z, idx, cnt, o, lse, dq, dk, dv, dw, db)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        step()                                                           # warm-up outside the capture (attributes, first-use set-up)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            step()
    torch.cuda.synchronize()
    for x in reversed(xs):                                               # second inputs first, then the first again
        for t, n in ((q, "q"), (k, "k"), (v, "v"), (dO, "dO")):
            t.copy_(dev(x[n], dtype))
        for t in outs:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        got = [t.clone() for t in outs]
        for t in outs:
            t.zero_()
        step()
        torch.cuda.synchronize()
        assert lte.lib().lte_device_status() == 0
        for a, b in zip(got, outs):
            assert torch.equal(a, b)                                     # the same kernels on the same bits: identical results
