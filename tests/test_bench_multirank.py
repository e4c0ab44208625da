"""The N > 1 path of bench.py is replicas only (no data-path collective): what ranks share is the timing rule
(max over ranks) and the whole-job rate.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(1.0 + rank, dist, "cpu")            # rank 1 is the slow one
    rate = bench.whole_job_rate(1000, world, ms)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (ms, rate)


def test_slowest_rank_sets_the_time_and_rate_is_the_aggregate():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29533, out), nprocs=world, join=True)
        assert out[0] == out[1]
        ms, rate = out[0]
        assert ms == 2.0
        assert abs(rate - 2 * 1000 / 2e-3) < 1e-6


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` outside a launcher starts two local ranks itself (the same start-up function the GPU
    run goes through); here with the gloo backend and only the rank plumbing, so that it runs without a GPU."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo", "--selftest-ranks"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                               # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 2.0 and abs(lines[0]["value"] - 2 * 1000 / 2e-3) < 1e-6


def test_inside_a_launcher_nothing_is_spawned(monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "0"); monkeypatch.setenv("WORLD_SIZE", "2")
    assert bench.spawn_ranks(2, []) is None
    monkeypatch.delenv("RANK"); monkeypatch.delenv("WORLD_SIZE")
    assert bench.spawn_ranks(1, []) is None


def test_traffic_figure_is_dropped_when_the_kernel_sources_changed(tmp_path, monkeypatch):
    import json
    sys.path.insert(0, ROOT)
    import bench
    f = tmp_path / "t.json"
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    assert bench.ncu_traffic("prefill_attn_C2")[0] is None          # no record at all
    src = bench.TRAFFIC_SOURCES["prefill_attn_C2"]
    f.write_text(json.dumps({"prefill_attn_C2": {"dram_bytes_per_launch": 1.5e8, "commit": "abc", "summary": "x.md", "sources": src,
                                                 "sources_sha256": bench.sources_digest(src)}}))
    val, prov = bench.ncu_traffic("prefill_attn_C2")
    assert val == 1.5e8 and prov["sources_unchanged"] and prov["capture_commit"] == "abc"
    f.write_text(json.dumps({"prefill_attn_C2": {"dram_bytes_per_launch": 1.5e8, "commit": "abc", "summary": "x.md", "sources": src,
                                                 "sources_sha256": "0" * 64}}))
    assert bench.ncu_traffic("prefill_attn_C2") == (None, {"capture_commit": "abc", "summary": "x.md", "sources_unchanged": False})


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_rate(16384, 1, 0.5) == 16384 / 0.5e-3
