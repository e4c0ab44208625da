"""The allocation-free backward entry point, checked against the fp64 oracle and against the regular entry point.

Some users of this library run where device memory cannot be allocated at call time (a frozen serving pool, a
region where cudaMalloc's implicit device synchronisation is unacceptable).  For them `lte_attn_bwd_static` keeps
its scratch in a fixed array inside the library.  The tests check the gradients (oracle, and the workspace entry
point) on two calls in a row, and the call's one promise: that free device memory and the caller's allocator are the
same after the call as before it.  This file is named so that pytest collects it last; it must pass on its own in a
fresh process and after every other test.
"""
import numpy as np
import pytest
import torch

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import assert_grad_close, dev, shape_of

pytestmark = pytest.mark.gpu

REL = {"bf16": 5e-2, "f32": 1e-4}


def _inputs(cfg, seed, group=1):
    x = synth.make(cfg, seed, with_dO=True)
    s = shape_of(cfg)
    s.group = group
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    k, v = (dev(x[t], cfg.dtype) for t in ("k", "v"))
    if group > 1:
        xq = synth.make(cfg.with_(H=cfg.H * group), seed + 100, with_dO=True)
        x["q"], x["dO"] = xq["q"], xq["dO"]
    q, dO = dev(x["q"], cfg.dtype), dev(x["dO"], cfg.dtype)
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    return x, (s, c, q, k, v, o, lse, dO, z, idx, cnt)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_backward_matches_oracle_and_workspace_backward_twice_in_a_row(dtype):
    cfg = synth.Config("noalloc", dtype, 2, 3, 64, 300, 40, 25, 7, 0.1, qk_unit=(dtype == "f32"))
    # two calls in a row on different inputs: the second one finds the first one's leftovers in the shared array
    for n, seed in enumerate((11, 12)):
        x, args = _inputs(cfg, seed)
        want = lte.lte_attn_bwd(*args)
        outs = tuple(torch.empty_like(t) for t in want)          # caller-owned outputs: the call allocates nothing
        torch.cuda.synchronize()
        # requests made to the caller's allocator so far (a counter: it never goes down when something is freed)
        nreq = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]
        free0, req0, resv0 = torch.cuda.mem_get_info()[0], nreq(), torch.cuda.memory_reserved()
        got = lte.lte_attn_bwd_static(*args, outs=outs)
        torch.cuda.synchronize()
        free1, req1, resv1 = torch.cuda.mem_get_info()[0], nreq(), torch.cuda.memory_reserved()
        assert (req1, resv1) == (req0, resv0), "the caller's allocator was used"
        if n > 0:                                                 # the first call on a device may load the library's module
            assert free1 == free0, "device memory was taken or given back during the call"
        idx_n, cnt_n = args[9].cpu().numpy(), args[10].cpu().numpy()
        z64 = orc.scores(x["k"], x["v"], x["w"])
        g = orc.attn_bwd(x["q"], x["k"], x["v"], x["dO"], z64, idx_n, cnt_n, x["w"], cfg.W)
        for name, a, b in zip(("dq", "dk", "dv", "dw", "dbias"), got, want):
            a, b = a.float().cpu().numpy(), b.float().cpu().numpy()
            assert_grad_close(name, a, g[name], REL[dtype], *((idx_n, cnt_n) if name in ("dk", "dv") else ()))
            assert_grad_close(name + " (vs lte_attn_bwd)", a, b, REL[dtype])


def test_static_scratch_backward_with_grouped_queries():
    """Several query heads per key/value head: the same kernels and scratch plan as lte_attn_bwd."""
    cfg = synth.Config("noalloc", "bf16", 2, 2, 64, 300, 32, 24, 7, 0.1)
    for seed in (3, 4):
        _, args = _inputs(cfg, seed, group=2)
        want = lte.lte_attn_bwd(*args)
        got = lte.lte_attn_bwd_static(*args, outs=tuple(torch.empty_like(t) for t in want))
        torch.cuda.synchronize()
        for name, a, b in zip(("dq", "dk", "dv", "dw", "dbias"), got, want):
            assert torch.equal(a, b), name                        # same kernels, same order of operations: same bits


def test_static_scratch_rejects_shapes_beyond_its_fixed_size():
    cfg = synth.CONFIGS["C5"]                                     # needs far more than the 8 MiB array
    s = shape_of(cfg)
    assert lte.lte_workspace_bytes(lte.OP_BWD, s, lte.LteConv(1, 7, 1, 256, 0)) > lte.STATIC_SCRATCH_BYTES
    small = synth.Config("noalloc", "bf16", 1, 1, 64, 64, 16, 8, 7, 0.1)
    args = list(_inputs(small, 1)[1])
    args[0] = s                                                   # claim the big shape: must fail before any launch
    with pytest.raises(lte.LteError) as err:
        lte.lte_attn_bwd_static(*args, outs=tuple(torch.empty(1, device="cuda") for _ in range(5)))
    assert err.value.status == -3
