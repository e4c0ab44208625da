"""The allocation-free backward entry point, checked against the regular one.

Some users of this library run where device memory cannot be allocated at call time (a frozen serving pool, a
region where cudaMalloc's implicit device synchronisation is unacceptable).  For them `lte_attn_bwd_static` keeps
its scratch in a fixed array inside the library.  This file is named so that pytest collects it last; it must
pass on its own in a fresh process and after every other test.
"""
import numpy as np
import pytest
import torch

from paper_2510_20787_b200 import lte, synth
from tests.gpu_util import dev, rel_l2, shape_of

pytestmark = pytest.mark.gpu

REL = {"bf16": 5e-2, "f32": 1e-4}


def _inputs(cfg, seed):
    x = synth.make(cfg, seed, with_dO=True)
    s = shape_of(cfg)
    c = lte.conv(torch.from_numpy(x["w"]).cuda())
    q, k, v, dO = (dev(x[t], cfg.dtype) for t in ("q", "k", "v", "dO"))
    z = lte.lte_scores(s, c, k, v)
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, q, k, v, idx, cnt)
    return s, c, q, k, v, o, lse, dO, z, idx, cnt


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_backward_matches_workspace_backward_twice_in_a_row(dtype):
    cfg = synth.Config("noalloc", dtype, 2, 3, 64, 300, 40, 25, 7, 0.1, qk_unit=(dtype == "f32"))
    # two calls in a row on different inputs: the second one finds the first one's leftovers in the shared array
    for seed in (11, 12):
        args = _inputs(cfg, seed)
        want = lte.lte_attn_bwd(*args)
        outs = tuple(torch.empty_like(t) for t in want)          # caller-owned outputs: the call allocates nothing
        got = lte.lte_attn_bwd_static(*args, outs=outs)
        torch.cuda.synchronize()
        for name, a, b in zip(("dq", "dk", "dv", "dw", "dbias"), got, want):
            a, b = a.float().cpu().numpy(), b.float().cpu().numpy()
            assert np.all(np.isfinite(a)), name
            assert rel_l2(a, b) <= REL[dtype], (name, rel_l2(a, b))


def test_static_scratch_rejects_shapes_beyond_its_fixed_size():
    cfg = synth.CONFIGS["C5"]                                     # needs far more than the 8 MiB array
    s = shape_of(cfg)
    assert lte.lte_workspace_bytes(lte.OP_BWD, s, lte.LteConv(1, 7, 1, 256, 0)) > lte.STATIC_SCRATCH_BYTES
    small = synth.Config("noalloc", "bf16", 1, 1, 64, 64, 16, 8, 7, 0.1)
    args = list(_inputs(small, 1))
    args[0] = s                                                   # claim the big shape: must fail before any launch
    with pytest.raises(lte.LteError) as err:
        lte.lte_attn_bwd_static(*args, outs=tuple(torch.empty(1, device="cuda") for _ in range(5)))
    assert err.value.status == -3
