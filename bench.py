#!/usr/bin/env python
"""Benchmark of the LTE sparse-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl lte|reference] [--no-extras]

A step is one pass of the prefill hot path (lte_scores -> lte_select -> lte_attn_prefill) over one
synthetic batch of the bf16 prefill configuration (B=4, H=16, d=64, T=4096, W=128, R=128, 7 taps).
`value` is whole-job prefill tokens/s with the inputs resident in HBM; `e2e` is the same metric through
the same calls with host buffers (pinned host -> device copies of q, k, v and the device -> host read of
O, logsumexp and the retained lists inside the timed region).  With N > 1 every rank runs the same
per-GPU batch on its own GPU (the (batch, head) units are independent: no data-path collective, weak
scaling) and the slowest rank sets the time.  Extra sections time the other rows of the path on their
own configurations: long prefill, batched decode (us per step, HBM GB/s) and forward+backward.

`--impl reference` times the fp64 CPU oracle, as it stands, on the host cores for the same metric.
"""
import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "LTE attn prefill tokens/s & % bf16 TC peak; decode step us & % HBM BW"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOAD = "C2 bf16 prefill: B=4 H=16 d=64 T=4096 W=128 R=128 K=7 per GPU, scores+select+attention"
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")


def bench_config(world):
    """The `config` object of the bench line (both arms print the same one: the reference arm times this workload too)."""
    return {"workload": WORKLOAD, "l2": "flushed between timed steps (256 MB written, then 256 MB read so that no dirty line is left to write back inside a step)",
            "parallelism": "replicas x%d (independent (batch, head) units)" % world}


def sources_digest(files):
    """sha256 over the named kernel sources (paths relative to the package's csrc/), in the given order."""
    import hashlib
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2510_20787_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(key):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of a kernel, from the record of its last ncu capture
    (profiles/ncu_traffic.json: bytes, the commit the capture was taken at, and a digest of the kernel's sources at that
    commit).  The figure is reported only while the sources still have that digest; after a change to the kernel it is
    None until the kernel is captured again.  Returns (bytes or None, provenance dict)."""
    try:
        rec = json.load(open(TRAFFIC_FILE))[key]
    except (OSError, KeyError, ValueError):
        return None, {"capture": None}
    try:
        current = sources_digest(rec["sources"])
    except OSError:
        current = None
    prov = {"capture_commit": rec.get("commit"), "summary": rec.get("summary"), "sources_unchanged": current == rec.get("sources_sha256")}
    return (float(rec["dram_bytes_per_launch"]) if prov["sources_unchanged"] else None), prov


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
def device_inputs(cfg, seed, torch, T=None, with_dO=False):
    """Seeded synthetic tensors of the configuration's distributions, drawn on the device."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    T = cfg.T if T is None else T
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    shp = (cfg.B, cfg.H, T, cfg.d)
    qk = 1.0 if cfg.qk_unit else cfg.d ** -0.25
    out = {}
    for name, sc in (("q", qk), ("k", qk), ("v", 1.0)) + ((("dO", 1.0),) if with_dO else ()):
        out[name] = (torch.randn(shp, generator=g, device="cuda", dtype=torch.float32) * sc).to(dt)
    out["w"] = torch.randn((cfg.H, cfg.K, 2 * cfg.d), generator=g, device="cuda", dtype=torch.float32) * cfg.sigma_w
    return out


_PREFILL_WS = {}


def prefill_ws(torch, lte, s):
    """The prefill attention's workspace (compacted retained rows) for a shape, allocated once."""
    key = (s.B, s.H, s.R, s.d, s.dtype)
    if key not in _PREFILL_WS:
        need = lte.lte_workspace_bytes(lte.OP_PREFILL, s, None)
        _PREFILL_WS[key] = torch.empty(need, dtype=torch.uint8, device="cuda") if need > 0 else False
    return _PREFILL_WS[key]


def make_flush(torch):
    """L2 flush between timed steps: 256 MB are written, then another 256 MB are read.  The write alone would leave the L2
    full of dirty lines of the flush buffer, and their write-back would land inside the next timed region (it cost the first
    kernel of a step about 7 us at C2); after the read the L2 holds clean lines of a buffer no kernel uses."""
    wr = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    rd = torch.zeros(32 << 20, dtype=torch.int64, device="cuda")

    def flush():
        wr.fill_(1)
        rd.sum()
    return flush


def timed(torch, fn, steps, warmup, flush, sub_events=0):
    """Run fn() warmup + steps times; returns per-step ms list and, if fn returns event lists, their deltas."""
    for _ in range(warmup):
        flush(); fn()
    torch.cuda.synchronize()
    ms, subs = [], []
    for _ in range(steps):
        flush()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        marks = fn()
        e1.record()
        ms.append((e0, e1)); subs.append(marks)
    torch.cuda.synchronize()
    out = [a.elapsed_time(b) for a, b in ms]
    sub = None
    if subs and subs[0]:
        sub = [[m[i].elapsed_time(m[i + 1]) for i in range(len(m) - 1)] for m in subs]
    return out, sub


def mid3(xs):
    """Mean of the middle values (the paper's protocol: middle three of five runs)."""
    xs = sorted(xs)
    if len(xs) >= 5:
        k = (len(xs) - 3) // 2
        xs = xs[k:k + 3]
    return float(np.mean(xs))


def attn_flops(idx, cnt, T, W, d, torch):
    """Algorithmic attention FLOPs 4*d*|A_i| summed from the actual retained lists."""
    B, H, R = idx.shape
    i = torch.arange(T, device=idx.device)
    win = torch.clamp(i + 1, max=W).sum().item() * B * H
    thr = (i - W)                                               # entry visible iff idx <= i - W
    ids = idx.reshape(B * H, R).to(torch.int64)
    valid = torch.arange(R, device=idx.device)[None, :] < cnt.reshape(B * H, 1)
    # number of queries that see entry j: T - (j + W) for j + W <= T - 1
    vis = torch.where(valid, torch.clamp(T - (ids + W), min=0), torch.zeros_like(ids)).sum().item()
    del thr
    return 4.0 * d * (win + vis)


def max_over_ranks(ms, dist, device):
    """The slowest rank sets the time: all-reduce(MAX) of a per-rank duration (no-op without a process group)."""
    import torch
    if dist is None:
        return float(ms)
    t = torch.tensor([float(ms)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank, world, ms):
    """Weak scaling: every rank processes `units_per_rank` in `ms` (max over ranks) -> aggregate units per second."""
    return units_per_rank * world / (ms * 1e-3)


def run_lte(args):
    import torch
    from paper_2510_20787_b200 import lte, synth

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(args.backend, device_id=torch.device("cuda", local))
    lte.lib()
    pk = peaks()
    if args.section and args.skip_main:
        # only the named section (used for profiler captures of its kernels)
        flush = make_flush(torch)
        print(json.dumps({"section": args.section,
                          "extras": extras(torch, lte, synth, pk, flush, args, only=(args.section,))}))
        return

    cfg = synth.CONFIGS["C2"]
    x = device_inputs(cfg, 1000 + rank, torch)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    c = lte.conv(x["w"])
    q, k, v = x["q"], x["k"], x["v"]
    z = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")
    idx = torch.empty((cfg.B, cfg.H, cfg.R), dtype=torch.int32, device="cuda")
    cnt = torch.empty((cfg.B, cfg.H), dtype=torch.int32, device="cuda")
    o = torch.empty_like(q)
    lse = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")
    flush = make_flush(torch)

    def ev():
        e = torch.cuda.Event(enable_timing=True); e.record(); return e

    def step():                               # the three calls as a user makes them: nothing between the launches
        lte.lte_scores(s, c, k, v, z=z)
        lte.lte_select(s, z, idx=idx, cnt=cnt)
        lte.lte_attn_prefill(s, q, k, v, idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s))
        return None

    def step_marked():                        # the same step with an event after every launch (per-kernel durations)
        m = [ev()]
        lte.lte_scores(s, c, k, v, z=z); m.append(ev())
        lte.lte_select(s, z, idx=idx, cnt=cnt); m.append(ev())
        lte.lte_attn_prefill(s, q, k, v, idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s)); m.append(ev())
        return m

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    barrier()
    for _ in range(args.warmup):
        flush(); step()
    barrier()
    if rank == 0:
        sampler.start()
    t_wall = time.time()
    ms, _ = timed(torch, step, args.steps, 0, flush)
    barrier()
    t_wall = time.time() - t_wall
    # second pass over the same steps with an event after every launch: the per-kernel durations the roofline uses
    # (events between launches keep a kernel from starting under its predecessor's tail, so this pass is a little slower)
    ms_marked, sub = timed(torch, step_marked, args.steps, 0, flush)
    barrier()
    # keep the GPU busy long enough for a few clock samples
    if rank == 0:
        t0 = time.time()
        while time.time() - t0 < 1.0:
            step()
        torch.cuda.synchronize()
        clocks = sampler.stop()
    step_ms = max_over_ranks(float(np.mean(ms)), dist, "cuda")
    tokens = cfg.B * cfg.T * world
    value = whole_job_rate(cfg.B * cfg.T, world, step_ms)
    sub = np.array(sub)                       # [steps, 3] ms: scores, select, attention
    k_ms = sub.mean(axis=0)

    # ---- end to end through the same calls, host buffers --------------------------------------
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty(o.shape, dtype=o.dtype).pin_memory()
    hl = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
    hi = torch.empty(idx.shape, dtype=idx.dtype).pin_memory()
    hc = torch.empty(cnt.shape, dtype=cnt.dtype).pin_memory()
    dq_, dk_, dv_ = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)

    # Three streams: all host->device copies in order on one (k, v of an element first, then its q), the kernels of the
    # elements on the current stream as their inputs arrive, all device->host copies on a third: the copy of element b+1, the
    # kernels of element b and the read-back of element b-1 overlap (the two copy directions use different engines), and
    # each engine sees one queue of large copies.
    s1 = lte.shape(1, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    st_in, st_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_kv = [torch.cuda.Event() for _ in range(cfg.B)]
    ev_q = [torch.cuda.Event() for _ in range(cfg.B)]
    ev_done = [torch.cuda.Event() for _ in range(cfg.B)]

    def e2e_step():
        cur = torch.cuda.current_stream()
        st_in.wait_stream(cur); st_out.wait_stream(cur)
        with torch.cuda.stream(st_in):
            for b in range(cfg.B):
                sl = slice(b, b + 1)
                dk_[sl].copy_(hk[sl], non_blocking=True); dv_[sl].copy_(hv[sl], non_blocking=True)
                ev_kv[b].record(st_in)
                dq_[sl].copy_(hq[sl], non_blocking=True)
                ev_q[b].record(st_in)
        for b in range(cfg.B):
            sl = slice(b, b + 1)
            cur.wait_event(ev_kv[b])
            lte.lte_scores(s1, c, dk_[sl], dv_[sl], z=z[sl])
            lte.lte_select(s1, z[sl], idx=idx[sl], cnt=cnt[sl])
            cur.wait_event(ev_q[b])
            lte.lte_attn_prefill(s1, dq_[sl], dk_[sl], dv_[sl], idx[sl], cnt[sl], o=o[sl], lse=lse[sl], ws=prefill_ws(torch, lte, s1))
            ev_done[b].record(cur)
            with torch.cuda.stream(st_out):
                st_out.wait_event(ev_done[b])
                ho[sl].copy_(o[sl], non_blocking=True); hl[sl].copy_(lse[sl], non_blocking=True)
                hi[sl].copy_(idx[sl], non_blocking=True); hc[sl].copy_(cnt[sl], non_blocking=True)
        cur.wait_stream(st_out)
        return None

    barrier()
    e_ms, _ = timed(torch, e2e_step, args.steps, max(args.warmup, 3), flush)
    barrier()
    e2e_ms = max_over_ranks(float(np.mean(e_ms)), dist, "cuda")
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = sum(t.numel() * t.element_size() for t in (ho, hl, hi, hc))

    # ---- roofline of the dominant kernel -----------------------------------------------------------
    esz = 2
    attn_bytes = 4 * cfg.B * cfg.H * cfg.T * cfg.d * esz + cfg.B * cfg.H * cfg.T * 4 + cfg.B * cfg.H * (cfg.R + 1) * 4
    score_bytes = 2 * cfg.B * cfg.H * cfg.T * cfg.d * esz + cfg.B * cfg.H * cfg.T * 4
    flops = attn_flops(idx, cnt, cfg.T, cfg.W, cfg.d, torch)
    attn_s = k_ms[2] * 1e-3
    roof = {"bound": "hbm", "kernel": "lte_attn_prefill", "achieved": attn_bytes / attn_s / 1e9,
            "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": attn_bytes / attn_s / 1e9 / pk["hbm_gbs"],
            "traffic": ncu_traffic("prefill_attn_C2")[0], "traffic_capture": ncu_traffic("prefill_attn_C2")[1],
            "peak_source": pk["source"],
            "algorithmic_bytes": attn_bytes, "algorithmic_flops": flops,
            "tensor_tflops": flops / attn_s / 1e12, "tensor_frac": flops / attn_s / 1e12 / pk["bf16_tflops"],
            "kernel_ms": {"lte_scores": float(k_ms[0]), "lte_select": float(k_ms[1]), "lte_attn_prefill": float(k_ms[2])},
            "scores_gbs": score_bytes / (k_ms[0] * 1e-3) / 1e9}

    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": bench_config(world),
            "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": 4 * args.steps, "roofline": roof, "wall_s": t_wall,
            "ms_per_step_marked": float(np.mean(ms_marked)),
            "timing_note": "value: K steps of three back-to-back calls (four launches: scores, select, compaction of the retained rows, attention); roofline.kernel_ms: a second pass of K steps with an event after every call (lte_attn_prefill = compaction + attention kernel)"}
    if rank == 0:
        line["clocks"] = clocks

    # ---- the other rows of the path on their own configurations --------------------------------
    if args.section and rank == 0 and world == 1:
        del hq, hk, hv, ho, dq_, dk_, dv_
        print(json.dumps({"section": args.section, "extras": extras(torch, lte, synth, pk, flush, args,
                                                                    only=(args.section,))}))
        return
    if not args.no_extras and rank == 0 and world == 1:
        del hq, hk, hv, ho, dq_, dk_, dv_
        line["extras"] = extras(torch, lte, synth, pk, flush, args)
        line["cpu_baseline"] = cpu_baseline(synth)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def extras(torch, lte, synth, pk, flush, args, only=None):
    """The other rows of the path on their own configurations; `only` restricts the sections run."""
    return _extras_sections(torch, lte, synth, pk, flush, args, only if only is not None else ("C3", "C5", "C4"))


def _extras_sections(torch, lte, synth, pk, flush, args, which):
    out = {}
    n5 = 5
    if "C3" in which:
        _extra_c3(out, torch, lte, synth, pk, flush, n5)
    if "C5" in which:
        _extra_c5(out, torch, lte, synth, pk, flush, n5)
    if "C4" in which:
        _extra_c4(out, torch, lte, synth, pk, flush, n5)
    if "P" in which:
        _extra_p(out, torch, lte, synth, pk, flush, n5)
    if "S" in which:
        _extra_s(out, torch, lte, synth, pk, flush, n5)
    if "K" in which:
        _extra_k(out, torch, lte, synth, pk, flush, n5)
    return out


def _extra_k(out, torch, lte, synth, pk, flush, n5):
    """Chunked prefill on top of a cache (lte_attn_prefill_chunk): a prompt of T tokens is prefilled in one shot and cached,
    then a chunk of Tc more tokens arrives.  Two shapes: C2's (chunk = another 4096 tokens) and a serving-like one with the
    paper's window and budget (W = 768, R = 512; chunk of 512 tokens), where the local sequence is mostly cache rows."""
    import dataclasses
    res = {}
    for tag, cfg, Tc in (("C2_shape", synth.CONFIGS["C2"], 4096),
                         ("serving_like", dataclasses.replace(synth.CONFIGS["C2"], B=8, W=768, R=512), 512)):
        x = device_inputs(cfg, 11, torch, T=cfg.T + Tc)
        s0 = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
        sc = lte.shape(cfg.B, cfg.H, Tc, cfg.d, cfg.W, cfg.R, lte.BF16)
        c = lte.conv(x["w"])
        kp, vp = x["k"][:, :, :cfg.T].contiguous(), x["v"][:, :, :cfg.T].contiguous()
        z = lte.lte_scores(s0, c, kp, vp)
        idx, cnt = lte.lte_select(s0, z)
        cache0 = lte.lte_cache_init(s0, c, kp, vp, z, idx, cnt)
        cache = cache0.clone()
        qc, kc, vc = (x[t][:, :, cfg.T:].contiguous() for t in "qkv")
        o = torch.empty_like(qc); lse = torch.empty((cfg.B, cfg.H, Tc), dtype=torch.float32, device="cuda")
        ws = torch.empty(lte.lte_workspace_bytes(lte.OP_CHUNK, sc, c), dtype=torch.uint8, device="cuda")
        ms = []
        for it in range(3 + n5):
            cache.copy_(cache0)
            flush()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            lte.lte_attn_prefill_chunk(sc, c, cache, cfg.T, qc, kc, vc, o=o, lse=lse, ws=ws)
            e1.record(); torch.cuda.synchronize()
            if it >= 3:
                ms.append(e0.elapsed_time(e1))
        # the one-shot path over a prompt of the chunk's length, for scale
        s1 = lte.shape(cfg.B, cfg.H, Tc, cfg.d, cfg.W, cfg.R, lte.BF16)
        z1 = torch.empty((cfg.B, cfg.H, Tc), dtype=torch.float32, device="cuda")
        i1 = torch.empty((cfg.B, cfg.H, cfg.R), dtype=torch.int32, device="cuda"); c1 = torch.empty((cfg.B, cfg.H), dtype=torch.int32, device="cuda")

        def one_shot():
            lte.lte_scores(s1, c, kc, vc, z=z1); lte.lte_select(s1, z1, idx=i1, cnt=c1)
            lte.lte_attn_prefill(s1, qc, kc, vc, i1, c1, o=o, lse=lse, ws=prefill_ws(torch, lte, s1))

        ms1, _ = timed(torch, one_shot, n5, 3, flush)
        # the streaming reading of the same chunk (exact under a binding cap; row-by-row attention on the fp32 ALUs)
        ws_s = torch.empty(lte.lte_workspace_bytes(lte.OP_CHUNK_STREAM, sc, c), dtype=torch.uint8, device="cuda")
        ms_s = []
        for it in range(2 + n5):
            cache.copy_(cache0)
            flush()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            lte.lte_attn_prefill_chunk(sc, c, cache, cfg.T, qc, kc, vc, o=o, lse=lse, ws=ws_s, streaming=True)
            e1.record(); torch.cuda.synchronize()
            if it >= 2:
                ms_s.append(e0.elapsed_time(e1))
        del ws_s
        t = mid3(ms) * 1e-3
        res[tag] = {"workload": "B=%d H=%d d=%d, cache after %d tokens (W=%d, R=%d), chunk of %d tokens" % (cfg.B, cfg.H, cfg.d, cfg.T, cfg.W, cfg.R, Tc),
                    "chunk_ms": t * 1e3, "tokens_per_s": cfg.B * Tc / t, "local_rows": cfg.R + cfg.W + Tc,
                    "one_shot_prefill_of_a_prompt_of_the_chunks_length_ms": mid3(ms1),
                    "streaming_reading_chunk_ms": mid3(ms_s),
                    "workspace_bytes": int(ws.numel())}
        del x, cache, cache0, ws, o, lse, qc, kc, vc
    out["K_chunked_prefill"] = res


def _extra_s(out, torch, lte, synth, pk, flush, n5):
    """The paper's three-layer scorer (kernel 3, dilation 2, channels 2d -> d -> d/2 -> d/4 -> 1) at the C2 shape.
    With a workspace: the tensor-core kernel (three-way split bf16 operands, so 3x to 6x the algorithmic products are
    executed); without: the fp32 kernel on the ordinary ALUs, bounded by 148 SMs x 128 lanes x 2 FLOP x the SM clock."""
    cfg = synth.CONFIGS["C2"]
    x = device_inputs(cfg, 7, torch)
    d, H = cfg.d, cfg.H
    g = torch.Generator(device="cuda"); g.manual_seed(70)
    ch = [2 * d, d, d // 2, d // 4]
    wl = [torch.randn((H, ch[l + 1], 3, ch[l]), generator=g, device="cuda") * (1.5 / (3 * ch[l]) ** 0.5) for l in range(3)]
    wout = torch.randn((H, ch[3]), generator=g, device="cuda") * (2.0 / ch[3] ** 0.5)
    c = lte.conv_stack(wl, wout)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    z = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")
    ws = torch.empty(lte.lte_workspace_bytes(lte.OP_SCORES, s, c), dtype=torch.uint8, device="cuda")

    def f_tc():
        lte.lte_scores(s, c, x["k"], x["v"], z=z, ws=ws)

    def f_alu():
        lte.lte_scores(s, c, x["k"], x["v"], z=z, ws=False)

    t_tc = mid3(timed(torch, f_tc, n5, 3, flush)[0]) * 1e-3
    kept = float((z[:, :, : cfg.T - 6] > 0).float().mean())
    z_tc = z.clone()
    t_alu = mid3(timed(torch, f_alu, n5, 3, flush)[0]) * 1e-3
    dz = (z_tc - z)[:, :, : cfg.T - 6].abs().max()
    macs = 3 * (ch[0] * ch[1] + ch[1] * ch[2] + ch[2] * ch[3]) + ch[3]
    macs_exec = 3 * (3 * ch[0] * ch[1] + 6 * ch[1] * ch[2] + 6 * ch[2] * ch[3])      # weight pieces x activation pieces
    fl = 2.0 * macs * cfg.B * cfg.H * cfg.T
    props = torch.cuda.get_device_properties(0)
    alu_peak = props.multi_processor_count * 128 * 2 * 1.965e9
    out["S_scorer_stack"] = {
        "workload": "C2 shape, 3 conv layers k=3 dil=2, channels 128 -> 64 -> 32 -> 16 -> 1",
        "scores_ms": t_tc * 1e3, "tokens_per_s": cfg.B * cfg.T / t_tc, "algorithmic_tflops": fl / t_tc / 1e12,
        "executed_tflops": fl / t_tc / 1e12 * macs_exec / macs,
        "roofline": {"bound": "tensor", "achieved": fl / t_tc / 1e12, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": fl / t_tc / 1e12 / pk["bf16_tflops"], "peak_source": pk["source"],
                     "note": "algorithmic products; every one is executed 3 to 6 times over (split operands)"},
        "fp32_alu_kernel": {"scores_ms": t_alu * 1e3,
                            "roofline": {"bound": "alu", "achieved": fl / t_alu / 1e12, "peak": alu_peak / 1e12, "unit": "TFLOP/s",
                                         "frac": fl / t_alu / alu_peak, "peak_source": "SMs x 128 fp32 lanes x 2 x 1.965 GHz"}},
        "max_abs_z_difference_between_kernels": float(dz), "fraction_kept": kept}
    del x, z
    # backward through the stack at the training shape (C5): the attention backward is the same as with the single layer,
    # the scorer's part runs on the tensor cores (plain bf16 operands)
    cfg5 = synth.CONFIGS["C5"]
    x5 = device_inputs(cfg5, 8, torch, with_dO=True)
    s5 = lte.shape(cfg5.B, cfg5.H, cfg5.T, cfg5.d, cfg5.W, cfg5.R, lte.BF16)
    z5 = lte.lte_scores(s5, c, x5["k"], x5["v"])
    idx5, cnt5 = lte.lte_select(s5, z5)
    o5, lse5 = lte.lte_attn_prefill(s5, x5["q"], x5["k"], x5["v"], idx5, cnt5, ws=prefill_ws(torch, lte, s5))
    ws5 = torch.empty(lte.lte_workspace_bytes(lte.OP_BWD, s5, c), dtype=torch.uint8, device="cuda")
    c1 = lte.conv(x5["w"])
    ws1 = torch.empty(lte.lte_workspace_bytes(lte.OP_BWD, s5, c1), dtype=torch.uint8, device="cuda")

    def b_stack():
        lte.lte_attn_bwd(s5, c, x5["q"], x5["k"], x5["v"], o5, lse5, x5["dO"], z5, idx5, cnt5, ws=ws5)

    def b_single():
        lte.lte_attn_bwd(s5, c1, x5["q"], x5["k"], x5["v"], o5, lse5, x5["dO"], z5, idx5, cnt5, ws=ws1)

    t_bs = mid3(timed(torch, b_stack, n5, 3, flush)[0]) * 1e-3
    t_b1 = mid3(timed(torch, b_single, n5, 3, flush)[0]) * 1e-3
    fl5 = 2.0 * macs * cfg5.B * cfg5.H * cfg5.T
    out["S_scorer_stack"]["backward_C5"] = {
        "workload": "C5 shape, lte_attn_bwd with the stack (weight, bias and input gradients)",
        "bwd_ms": t_bs * 1e3, "bwd_ms_single_layer_scorer": t_b1 * 1e3,
        "stack_part_ms": (t_bs - t_b1) * 1e3 if t_bs > t_b1 else None,
        "roofline": {"bound": "tensor", "achieved": 3 * fl5 / max(t_bs - t_b1, 1e-9) / 1e12, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": 3 * fl5 / max(t_bs - t_b1, 1e-9) / 1e12 / pk["bf16_tflops"], "peak_source": pk["source"],
                     "note": "3 x the forward's products (forward again, transposed products, weight gradients) over the time the stack adds"}}
    del x5, o5, lse5, z5
    # the stack in decode at the C4 cache shape (prompt of 1024 tokens): the step scores nothing, lte_cache_score runs once per
    # W - 13 steps over the whole ring (lazy batches)
    cfg4 = synth.CONFIGS["C4"].with_(T=1024)
    x4 = device_inputs(cfg4, 9, torch)
    s4 = lte.shape(cfg4.B, cfg4.H, cfg4.T, cfg4.d, cfg4.W, cfg4.R, lte.BF16)
    z4 = lte.lte_scores(s4, c, x4["k"], x4["v"])
    idx4, cnt4 = lte.lte_select(s4, z4)
    cache = lte.lte_cache_init(s4, c, x4["k"], x4["v"], z4, idx4, cnt4)
    wsd = torch.empty(lte.lte_workspace_bytes(lte.OP_DECODE, s4, c), dtype=torch.uint8, device="cuda")
    g4 = torch.Generator(device="cuda"); g4.manual_seed(91)
    q1, k1, v1 = ((torch.randn((cfg4.B, cfg4.H, cfg4.d), generator=g4, device="cuda") * f).to(torch.bfloat16) for f in (0.35, 0.35, 1.0))
    o1 = torch.empty_like(q1); l1 = torch.empty((cfg4.B, cfg4.H), dtype=torch.float32, device="cuda")

    def f_score():
        lte.lte_cache_score(s4, c, cache, ws=wsd)

    def f_step():
        lte.lte_attn_decode(s4, c, cache, q1, k1, v1, o1=o1, lse1=l1)

    t_sc = mid3(timed(torch, f_score, n5, 3, flush)[0]) * 1e-3
    t_st = mid3(timed(torch, f_step, n5, 3, flush)[0]) * 1e-3
    out["S_scorer_stack"]["decode_C4_cache"] = {
        "workload": "B=128 H=16 d=64 W=128 R=128, stack scorer: lte_cache_score every W - 13 = 115 steps",
        "cache_score_ms": t_sc * 1e3, "amortised_us_per_step": t_sc * 1e6 / (cfg4.W - 13),
        "decode_step_us_single_launch": t_st * 1e6,
        "note": "single launches with the L2 flushed in between (the C4 section times the step in a CUDA graph)"}
    del x4, cache, wsd


def _extra_p(out, torch, lte, synth, pk, flush, n5):
    """Context, not a gate: a serving shape like the paper's (batch 32, 4K prompt, window 768, budget 512, 4 sink
    tokens) with a per-head bias chosen so that about half the budget is used (cap not binding, list half full)."""
    from statistics import NormalDist
    cfg = synth.CONFIGS["C2"].with_(name="P", B=32, W=768, R=512, sink=4)
    x = device_inputs(cfg, 6, torch)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16, sink=cfg.sink)
    z0 = lte.lte_scores(s, lte.conv(x["w"]), x["k"], x["v"])
    zc = z0[:, :, : cfg.T - cfg.K // 2]                           # the tail positions have no score yet
    sigma = zc.transpose(0, 1).reshape(cfg.H, -1).std(dim=1)
    beta = (-sigma * NormalDist().inv_cdf(1.0 - cfg.R / (2.0 * (cfg.T - cfg.W)))).to(torch.float32).contiguous()
    c = lte.conv(x["w"], beta)
    z = torch.empty_like(z0)
    idx = torch.empty((cfg.B, cfg.H, cfg.R), dtype=torch.int32, device="cuda")
    cnt = torch.empty((cfg.B, cfg.H), dtype=torch.int32, device="cuda")
    o = torch.empty_like(x["q"]); lse = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")

    def step():
        lte.lte_scores(s, c, x["k"], x["v"], z=z)
        lte.lte_select(s, z, idx=idx, cnt=cnt)
        lte.lte_attn_prefill(s, x["q"], x["k"], x["v"], idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s))

    def f_attn():
        lte.lte_attn_prefill(s, x["q"], x["k"], x["v"], idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s))

    ms, _ = timed(torch, step, n5, 3, flush)
    ms_a, _ = timed(torch, f_attn, n5, 3, flush)
    fl = attn_flops(idx, cnt, cfg.T, cfg.W, cfg.d, torch)
    t, ta = mid3(ms) * 1e-3, mid3(ms_a) * 1e-3
    # decode from that prompt: 32 steps in a CUDA graph after 8 warm-up steps
    cache = lte.lte_cache_init(s, c, x["k"], x["v"], z, idx, cnt)
    n_dec = 40
    g = torch.Generator(device="cuda"); g.manual_seed(61)
    sc = cfg.d ** -0.25
    qs, ks, vs = ((torch.randn((n_dec, cfg.B, cfg.H, cfg.d), generator=g, device="cuda") * f).to(torch.bfloat16)
                  for f in (sc, sc, 1.0))
    o1 = torch.empty((cfg.B, cfg.H, cfg.d), dtype=torch.bfloat16, device="cuda")
    l1 = torch.empty((cfg.B, cfg.H), dtype=torch.float32, device="cuda")
    for i in range(8):
        lte.lte_attn_decode(s, c, cache, qs[i], ks[i], vs[i], o1=o1, lse1=l1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(8, n_dec):
            lte.lte_attn_decode(s, c, cache, qs[i], ks[i], vs[i], o1=o1, lse1=l1)
    reps = []
    for _ in range(5):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); graph.replay(); e1.record()
        torch.cuda.synchronize()
        reps.append(e0.elapsed_time(e1) * 1e3 / (n_dec - 8))
    dec_us = mid3(reps)
    dec_bytes = (2 * (cfg.W + cfg.R) * cfg.d * 2 + cfg.R * 4 + 1024 + 16) * cfg.B * cfg.H
    out["P_paper_like"] = {"workload": "B=32 H=16 d=64 T=4096 W=768 R=512 sink=4 K=7, bias set for ~R/2 retained per head",
                           "step_ms": t * 1e3, "tokens_per_s": cfg.B * cfg.T / t, "attn_ms": ta * 1e3,
                           "attn_algorithmic_tflops": fl / ta / 1e12, "attn_tensor_frac": fl / ta / 1e12 / pk["bf16_tflops"],
                           "mean_retained": float(cnt.float().mean()), "max_retained": int(cnt.max()),
                           "decode_us_per_step": dec_us, "decode_hbm_gbs": dec_bytes / dec_us / 1e3,
                           "decode_hbm_frac": dec_bytes / dec_us / 1e3 / pk["hbm_gbs"]}
    del o, lse, z, z0, cache
    # the same serving shape with grouped queries as in the paper's models: 32 query heads on 8 key/value heads
    G, Hk = 4, 8
    sg = lte.shape(cfg.B, Hk, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16, sink=cfg.sink, group=G)
    kg, vg = x["k"][:, :Hk].contiguous(), x["v"][:, :Hk].contiguous()
    cg = lte.conv(x["w"][:Hk].contiguous(), beta[:Hk].contiguous())
    gq = torch.Generator(device="cuda"); gq.manual_seed(62)
    qg = (torch.randn((cfg.B, Hk * G, cfg.T, cfg.d), generator=gq, device="cuda") * sc).to(torch.bfloat16)
    del x
    zg = lte.lte_scores(sg, cg, kg, vg)
    idxg, cntg = lte.lte_select(sg, zg)
    og = torch.empty_like(qg); lseg = torch.empty((cfg.B, Hk * G, cfg.T), dtype=torch.float32, device="cuda")

    def step_g():
        lte.lte_scores(sg, cg, kg, vg, z=zg)
        lte.lte_select(sg, zg, idx=idxg, cnt=cntg)
        lte.lte_attn_prefill(sg, qg, kg, vg, idxg, cntg, o=og, lse=lseg, ws=prefill_ws(torch, lte, sg))

    def attn_g():
        lte.lte_attn_prefill(sg, qg, kg, vg, idxg, cntg, o=og, lse=lseg, ws=prefill_ws(torch, lte, sg))

    tg, tag = mid3(timed(torch, step_g, n5, 3, flush)[0]) * 1e-3, mid3(timed(torch, attn_g, n5, 3, flush)[0]) * 1e-3
    flg = attn_flops(idxg, cntg, cfg.T, cfg.W, cfg.d, torch) * G
    cache = lte.lte_cache_init(sg, cg, kg, vg, zg, idxg, cntg)
    qs = (torch.randn((n_dec, cfg.B, Hk * G, cfg.d), generator=gq, device="cuda") * sc).to(torch.bfloat16)
    o1 = torch.empty((cfg.B, Hk * G, cfg.d), dtype=torch.bfloat16, device="cuda")
    l1 = torch.empty((cfg.B, Hk * G), dtype=torch.float32, device="cuda")
    ks8, vs8 = ks[:, :, :Hk].contiguous(), vs[:, :, :Hk].contiguous()
    for i in range(8):
        lte.lte_attn_decode(sg, cg, cache, qs[i], ks8[i], vs8[i], o1=o1, lse1=l1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(8, n_dec):
            lte.lte_attn_decode(sg, cg, cache, qs[i], ks8[i], vs8[i], o1=o1, lse1=l1)
    reps = []
    for _ in range(5):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); graph.replay(); e1.record()
        torch.cuda.synchronize()
        reps.append(e0.elapsed_time(e1) * 1e3 / (n_dec - 8))
    out["P_paper_like"]["grouped_queries"] = {
        "workload": "the same with 32 query heads on 8 key/value heads (group = 4)",
        "step_ms": tg * 1e3, "tokens_per_s": cfg.B * cfg.T / tg, "attn_ms": tag * 1e3,
        "attn_algorithmic_tflops": flg / tag / 1e12, "attn_tensor_frac": flg / tag / 1e12 / pk["bf16_tflops"],
        "decode_us_per_step": mid3(reps),
        "note": "decode: one kernel updates the cache block of a key/value head and attends for the four query heads of its group"}
    del og, lseg, zg, cache, qg


def _extra_c3(out, torch, lte, synth, pk, flush, n5):

    # long prefill (tensor-core bound)
    cfg = synth.CONFIGS["C3"]
    x = device_inputs(cfg, 3, torch)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    c = lte.conv(x["w"])
    z = lte.lte_scores(s, c, x["k"], x["v"])
    idx, cnt = lte.lte_select(s, z)
    o = torch.empty_like(x["q"]); lse = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device="cuda")
    def f_attn():
        lte.lte_attn_prefill(s, x["q"], x["k"], x["v"], idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s))

    def f_scores():
        lte.lte_scores(s, c, x["k"], x["v"], z=z)

    def f_select():
        lte.lte_select(s, z, idx=idx, cnt=cnt)

    ms, _ = timed(torch, f_attn, n5, 3, flush)
    ms_sc, _ = timed(torch, f_scores, n5, 3, flush)
    ms_se, _ = timed(torch, f_select, n5, 3, flush)
    fl = attn_flops(idx, cnt, cfg.T, cfg.W, cfg.d, torch)
    t = mid3(ms) * 1e-3
    out["C3_long_prefill"] = {"attn_ms": t * 1e3, "tokens_per_s": cfg.B * cfg.T / t, "algorithmic_tflops": fl / t / 1e12,
                              "tensor_frac": fl / t / 1e12 / pk["bf16_tflops"], "scores_ms": mid3(ms_sc),
                              "select_ms": mid3(ms_se)}
    # backward at the same shape: the only configuration whose backward is tensor-core bound (2.5 x the forward's FLOPs)
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    dO = torch.randn(x["q"].shape, device="cuda", generator=g).to(x["q"].dtype)
    ws = torch.empty(lte.lte_workspace_bytes(lte.OP_BWD, s, c), dtype=torch.uint8, device="cuda")

    def f_bwd():
        lte.lte_attn_bwd(s, c, x["q"], x["k"], x["v"], o, lse, dO, z, idx, cnt, ws=ws)

    ms_b, _ = timed(torch, f_bwd, n5, 3, flush)
    tb = mid3(ms_b) * 1e-3
    out["C3_long_prefill"].update({"bwd_ms": tb * 1e3, "bwd_algorithmic_tflops": 2.5 * fl / tb / 1e12,
                                   "bwd_tensor_frac": 2.5 * fl / tb / 1e12 / pk["bf16_tflops"]})
    del x, o, lse, z, dO, ws


def _extra_c5(out, torch, lte, synth, pk, flush, n5):
    # forward + backward
    cfg = synth.CONFIGS["C5"]
    x = device_inputs(cfg, 5, torch, with_dO=True)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    c = lte.conv(x["w"])
    z = lte.lte_scores(s, c, x["k"], x["v"])
    idx, cnt = lte.lte_select(s, z)
    o, lse = lte.lte_attn_prefill(s, x["q"], x["k"], x["v"], idx, cnt, ws=prefill_ws(torch, lte, s))
    ws = torch.empty(lte.lte_workspace_bytes(lte.OP_BWD, s, c), dtype=torch.uint8, device="cuda")

    def fwd():
        lte.lte_scores(s, c, x["k"], x["v"], z=z); lte.lte_select(s, z, idx=idx, cnt=cnt)
        lte.lte_attn_prefill(s, x["q"], x["k"], x["v"], idx, cnt, o=o, lse=lse, ws=prefill_ws(torch, lte, s))

    def bwd():
        lte.lte_attn_bwd(s, c, x["q"], x["k"], x["v"], o, lse, x["dO"], z, idx, cnt, ws=ws)

    ms_f, _ = timed(torch, fwd, n5, 3, flush)
    ms_b, _ = timed(torch, bwd, n5, 3, flush)
    fl = attn_flops(idx, cnt, cfg.T, cfg.W, cfg.d, torch)
    tf, tb = mid3(ms_f) * 1e-3, mid3(ms_b) * 1e-3
    nb = cfg.B * cfg.H * cfg.T * cfg.d * 2
    out["C5_fwd_bwd"] = {"fwd_ms": tf * 1e3, "bwd_ms": tb * 1e3, "tokens_per_s": cfg.B * cfg.T / (tf + tb),
                         "bwd_algorithmic_tflops": 2.5 * fl / tb / 1e12, "bwd_hbm_gbs": 8 * nb / tb / 1e9,
                         "bwd_hbm_frac": 8 * nb / tb / 1e9 / pk["hbm_gbs"]}
    del x, o, lse, z, ws


def _extra_c4(out, torch, lte, synth, pk, flush, n5):
    # batched decode
    cfg = synth.CONFIGS["C4"]
    x = device_inputs(cfg, 4, torch)
    s = lte.shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.W, cfg.R, lte.BF16)
    c = lte.conv(x["w"])
    z = lte.lte_scores(s, c, x["k"], x["v"])
    idx, cnt = lte.lte_select(s, z)
    cache = lte.lte_cache_init(s, c, x["k"], x["v"], z, idx, cnt)
    del x, z
    g = torch.Generator(device="cuda"); g.manual_seed(44)
    sc = cfg.d ** -0.25
    qs, ks, vs = ((torch.randn((cfg.steps, cfg.B, cfg.H, cfg.d), generator=g, device="cuda") * f).to(torch.bfloat16)
                  for f in (sc, sc, 1.0))
    o1 = torch.empty((cfg.B, cfg.H, cfg.d), dtype=torch.bfloat16, device="cuda")
    l1 = torch.empty((cfg.B, cfg.H), dtype=torch.float32, device="cuda")
    for i in range(8):                                            # warm-up steps advance the cache too
        lte.lte_attn_decode(s, c, cache, qs[i], ks[i], vs[i], o1=o1, lse1=l1)
    torch.cuda.synchronize()
    # (a) launch by launch from Python (includes the host's per-call cost when the GPU outruns it)
    evs = []
    for i in range(8, cfg.steps):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); lte.lte_attn_decode(s, c, cache, qs[i], ks[i], vs[i], o1=o1, lse1=l1); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    us_eager = float(np.mean([a.elapsed_time(b) for a, b in evs])) * 1e3
    # (b) the same 248 steps captured once in a CUDA graph and replayed: the launch-bound loop without the host
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(8, cfg.steps):
            lte.lte_attn_decode(s, c, cache, qs[i], ks[i], vs[i], o1=o1, lse1=l1)
    reps = []
    for _ in range(5):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); graph.replay(); e1.record()
        torch.cuda.synchronize()
        reps.append(e0.elapsed_time(e1) * 1e3 / (cfg.steps - 8))
    us = mid3(reps)
    per = 2 * (cfg.W + cfg.R) * cfg.d * 2 + cfg.R * 4 + 1024 + 16      # ring+pool K,V, pool logits, q/k/v/o + row writes, meta
    by = per * cfg.B * cfg.H
    out["C4_decode"] = {"us_per_step": us, "us_per_step_python_launches": us_eager, "steps_timed": len(evs),
                        "timing": "CUDA graph of the 248 steps, middle 3 of 5 replays", "algorithmic_bytes_per_step": by,
                        "hbm_gbs": by / (us * 1e-6) / 1e9, "hbm_frac": by / (us * 1e-6) / 1e9 / pk["hbm_gbs"],
                        "traffic": ncu_traffic("decode_C4")[0], "traffic_capture": ncu_traffic("decode_C4")[1],
                        "note": "the 138 MB cache is about the size of L2: see the ncu DRAM bytes in profiles/"}


def oracle_step(orc, x, cfg):
    z = orc.scores(x["k"], x["v"], x["w"])
    idx, cnt, _ = orc.select(z, cfg.W, cfg.R)
    orc.attn_prefill(x["q"], x["k"], x["v"], idx, cnt, cfg.W)


def cpu_baseline(synth, reps=8):
    """The fp64 oracle, as it stands, on the host cores: the whole C2 batch, `reps` times."""
    from oracle import lte_oracle as orc
    cfg = synth.CONFIGS["C2"]
    x = synth.make(cfg, 0)
    x = {n: np.asarray(a, np.float64) for n, a in x.items()}
    oracle_step(orc, x, cfg)
    t0 = time.time()
    for _ in range(reps):
        oracle_step(orc, x, cfg)
    dt = (time.time() - t0) / reps
    return {"value": cfg.B * cfg.T / dt, "unit": "tokens/s", "cores": orc.num_threads(), "kind": "oracle",
            "sample": "the full C2 batch (B=4, 16384 tokens), scores+select+attention, mean of %d passes" % reps,
            "ms_per_step": dt * 1e3}


def run_reference(args):
    """Reference arm: the oracle on the host cores, same metric and configuration; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import lte_oracle as orc
    from paper_2510_20787_b200 import synth
    cfg = synth.CONFIGS["C2"]
    x = synth.make(cfg, 0)
    x = {n: np.asarray(a, np.float64) for n, a in x.items()}
    for _ in range(args.warmup):
        oracle_step(orc, x, cfg)
    steps = args.steps
    t0 = time.time()
    for _ in range(steps):
        oracle_step(orc, x, cfg)
    dt = (time.time() - t0) / steps
    val = cfg.B * cfg.T / dt
    sample = "each step = the full C2 batch once (B=4, 16384 tokens) on rank 0's host cores; %d steps timed" % steps
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": bench_config(max(args.gpus, 1)),
        "host_note": "the oracle runs on rank 0's host cores only (OpenMP over (batch, head)); no GPU, no L2 flush",
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": orc.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


TRAFFIC_SOURCES = {
    "prefill_attn_C2": ["prefill_tc.cu", "prefill_tc_long.cu", "tc_common.cuh", "tma_util.cuh", "common.cuh"],
    "decode_C4": ["decode_tc.cu", "tc_common.cuh", "tma_util.cuh", "common.cuh"],
}


def record_traffic(spec):
    """--record-traffic KEY=BYTES[,SUMMARY]: write the DRAM bytes per launch read off an ncu capture of the kernel behind
    KEY into profiles/ncu_traffic.json, with the current commit and the digest of the kernel's sources, so that a later
    bench line can tell whether the figure still belongs to the kernel it times.  Run it on the tree the capture used."""
    key, _, rest = spec.partition("=")
    val, _, summary = rest.partition(",")
    try:
        commit = subprocess.check_output(["git", "-C", ROOT, "rev-parse", "--short", "HEAD"], text=True).strip()
        if subprocess.check_output(["git", "-C", ROOT, "status", "--porcelain", "--", "paper_2510_20787_b200/csrc"], text=True).strip():
            commit += "+uncommitted"
    except (OSError, subprocess.CalledProcessError):
        commit = None
    try:
        rec = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        rec = {}
    rec[key] = {"dram_bytes_per_launch": float(val), "commit": commit, "summary": summary or None,
                "sources": TRAFFIC_SOURCES[key], "sources_sha256": sources_digest(TRAFFIC_SOURCES[key])}
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(rec, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(rec[key]))


def free_port():
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def spawn_ranks(n, argv):
    """`python bench.py --gpus N` outside a launcher: start N local ranks of this same command under
    torch.distributed.run (one process per GPU, rendezvous on 127.0.0.1) and return their exit code.  Inside a launcher
    (RANK / WORLD_SIZE in the environment) nothing is spawned and None is returned."""
    if n <= 1 or "RANK" in os.environ or "WORLD_SIZE" in os.environ:
        return None
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_rank_selftest(args):
    """The rank plumbing alone (process group, barrier, max over ranks, whole-job rate) on the given backend: what N > 1
    adds to the single-GPU run.  Used by the CPU test with gloo; rank r pretends its step took 1 + r ms."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group(args.backend)
    dev = "cuda" if args.backend == "nccl" else "cpu"
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(1.0 + rank, dist if world > 1 else None, dev)
    if world > 1:
        dist.barrier(); dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"selftest": "ranks", "n_gpus": world, "ms_per_step": ms, "value": whole_job_rate(1000, world, ms)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="lte", choices=["lte", "reference"])
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--section", default=None, choices=["C3", "C4", "C5", "P", "S", "K"],
                    help="time only this extra section (long prefill / decode / forward+backward) after the main loop")
    ap.add_argument("--skip-main", action="store_true", help="with --section: skip the main C2 loop")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"], help="process-group backend for N > 1")
    ap.add_argument("--selftest-ranks", action="store_true", help="run only the rank plumbing (barrier, max over ranks)")
    ap.add_argument("--record-traffic", default=None, metavar="KEY=BYTES[,SUMMARY]",
                    help="no benchmark: store an ncu DRAM-bytes figure with its provenance (see record_traffic)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.record_traffic:
        record_traffic(args.record_traffic)
        return
    if args.impl == "reference" and not args.selftest_ranks:
        run_reference(args)                   # host only: rank 0 works, nothing to spawn
        return
    rc = spawn_ranks(args.gpus, sys.argv[1:])
    if rc is not None:
        sys.exit(rc)
    if args.selftest_ranks:
        run_rank_selftest(args)
    else:
        run_lte(args)


if __name__ == "__main__":
    main()
