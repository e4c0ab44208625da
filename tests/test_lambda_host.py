"""Host side of the training pieces: lte_lambda_update (Algorithm 1's feedback loop, plain host arithmetic in the C-ABI
library) against the oracle, alone and with the counts averaged over two gloo ranks."""
import ctypes
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lte_oracle as orc
from paper_2510_20787_b200 import lte

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_follows_the_oracle_over_a_long_run():
    rng = np.random.default_rng(0)
    n = 24
    lam = torch.full((n,), 1e-9, dtype=torch.float32); cbar = torch.zeros(n, dtype=torch.float32)
    lam_o, cbar_o = np.full(n, 1e-9), np.zeros(n)
    base = rng.uniform(300, 800, n)                                         # some heads above the cap of 512, some below
    cfg = lte.LteLambdaCfg(8, 512.0, 2.0, 0.95, 1e-9, 1.0)
    for step in range(1, 400):
        count = base + rng.normal(0, 5, n) - (0.4 * step if step > 200 else 0.0)   # later every head drifts below the band
        lte.lte_lambda_update(lam, cbar, torch.from_numpy(count), step, cfg)
        lam_o, cbar_o = orc.lambda_update(lam_o, cbar_o, count, step, u=8, cap=512.0, alpha=2.0)
        np.testing.assert_allclose(cbar.numpy(), cbar_o, rtol=2e-5)
        np.testing.assert_allclose(lam.numpy(), lam_o, rtol=1e-4, atol=0)
    assert (lam.numpy() == 0).any() and step == 399


def test_moving_average_weights_the_new_sample_by_a_hand_computed():
    """Algorithm 1's average with the new sample weighted by a = 2 / (1 + u/2) (the reading taken): u = 6 gives a = 1/2,
    so from 0 the counts 8, 4, 10 give 4, 4, 7 by hand; the listing's weights the other way round would give the same
    numbers here only by accident of a = 1/2, so u = 2 (a = 1: the average IS the last count) is checked as well."""
    lam = torch.full((1,), 0.5, dtype=torch.float32); cbar = torch.zeros(1, dtype=torch.float32)
    cfg = lte.LteLambdaCfg(6, 512.0, 2.0, 0.95, 1e-9, 1.0)
    seen = []
    for step, cnt in enumerate([8.0, 4.0, 10.0], start=1):
        lte.lte_lambda_update(lam, cbar, torch.tensor([cnt], dtype=torch.float64), step, cfg)
        seen.append(float(cbar[0]))
    assert seen == [4.0, 4.0, 7.0]
    cbar.zero_()
    cfg2 = lte.LteLambdaCfg(2, 512.0, 2.0, 0.95, 1e-9, 1.0)
    for step, cnt in enumerate([8.0, 4.0, 10.0], start=1):
        lte.lte_lambda_update(lam, cbar, torch.tensor([cnt], dtype=torch.float64), step, cfg2)
        assert float(cbar[0]) == cnt


def test_defaults_and_argument_checks():
    L = lte.lib()
    lam = (ctypes.c_float * 2)(0.5, 0.0); cbar = (ctypes.c_float * 2)(600.0, 600.0); cnt = (ctypes.c_float * 2)(600.0, 600.0)
    assert L.lte_lambda_update(2, lam, cbar, cnt, 32, None) == 0           # defaults: period 32, cap 512, alpha 1.2
    assert abs(lam[0] - 0.6) < 1e-6 and abs(lam[1] - 1e-9) < 1e-15
    assert L.lte_lambda_update(2, lam, cbar, cnt, 33, None) == 0 and abs(lam[0] - 0.6) < 1e-6
    assert L.lte_lambda_update(2, None, cbar, cnt, 1, None) == -1
    assert L.lte_lambda_update(-1, lam, cbar, cnt, 1, None) == -1
    assert L.lte_lambda_update(2, lam, cbar, cnt, -5, None) == -1
    bad = lte.LteLambdaCfg(0, 512.0, 1.2, 0.95, 1e-9, 1.0)
    assert L.lte_lambda_update(2, lam, cbar, cnt, 1, ctypes.byref(bad)) == -1
    bad = lte.LteLambdaCfg(32, 512.0, 1.0, 0.95, 1e-9, 1.0)
    assert L.lte_lambda_update(2, lam, cbar, cnt, 1, ctypes.byref(bad)) == -1
    assert L.lte_lambda_update(0, None, None, None, 1, None) == 0


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lam = torch.tensor([0.25, 1e-9, 0.0]); cbar = torch.tensor([500.0, 500.0, 500.0])
    cfg = lte.LteLambdaCfg(2, 512.0, 2.0, 0.95, 1e-9, 1.0)
    # the ranks see different batches: alone, rank 0 would lower the first weight and rank 1 raise it
    mine = torch.tensor([300.0, 700.0, 900.0]) if rank == 0 else torch.tensor([900.0, 100.0, 900.0])
    for step in (1, 2):
        lte.lte_lambda_update(lam, cbar, mine, step, cfg)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (lam.tolist(), cbar.tolist())


def test_counts_are_averaged_over_ranks_so_all_ranks_decide_alike():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29541, out), nprocs=world, join=True)
        assert out[0] == out[1]
        lam, cbar = out[0]
    mean = np.array([600.0, 400.0, 900.0])
    lam_o, cbar_o = np.array([0.25, 1e-9, 0.0]), np.array([500.0, 500.0, 500.0])
    for step in (1, 2):
        lam_o, cbar_o = orc.lambda_update(lam_o, cbar_o, mean, step, u=2, cap=512.0, alpha=2.0)
    np.testing.assert_allclose(cbar, cbar_o, rtol=1e-6)
    np.testing.assert_allclose(lam, lam_o, rtol=1e-6)
