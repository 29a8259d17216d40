#!/usr/bin/env python
"""Benchmark of the HashAttention decode path on B200.

A "step" is one layer-step of the whole hot path (ENCODE of the queries and of the appended key,
SCORE, TOPK, GATHER-ATT) on the Llama-3.1-8B decode shape at 32K context and 32x sparsity
(config c2).  To keep every step L2-cold the steps rotate over R independent layer replicas
(own K, V, signature cache, q and mapping weights), like the 32 layers of a model; the replicas'
touched bytes exceed the 126 MB L2.  Steps are captured into CUDA graphs (the C-ABI calls only
enqueue kernels) so that host launch overhead does not hide the kernels.

Prints ONE JSON line: `value` = microseconds per layer-step with the inputs resident in HBM, `e2e` the same
step driven from pinned host buffers, `roofline` (algorithmic bytes of the step over its time, against the
measured HBM peak), `breakdown_us` of the stand-alone entry points, `dense_same_run`, `supplementary`
(larger batches, longer and ragged contexts, always-kept windows, the prompt encoders, the SCORE latency
against the signature width) and `cpu_baseline`
(the oracle on the host cores).  `--impl reference` times the CPU oracle instead (the only reference this
method has here).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sparse_decode_attn_us_per_layer_step"
UNIT = "us"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the step's kernel on this workload: NOT measured by this
# run (a number taken under a profiler is never a bench value) but copied from the ncu capture named beside it
TRAFFIC_FROM_PROFILE = {"bytes": 6555553, "source": "profiles/launch_list_bench_c2.md", "captured_at_commit": "220b429"}
GATHER_TRAFFIC_FROM_PROFILE = {"bytes": 4275000, "source": "profiles/launch_list_bench_c2.md", "captured_at_commit": "aed5e69"}
MIN_TIMED_MS = 50.0                 # the timed region of `steps` steps is repeated until this much has been measured
WORKLOAD = "c2: B=1, Hq=32, Hkv=8, d=128, ctx=32768, k=1024 (32x), 1% planted keys"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if not self.nv:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {
                "hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80,
            }
            for k, bit in names.items():
                if r & bit:
                    self.reasons.add(k)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.002)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self.sample()
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ----------------------------------------------------------------------------- device state

class Replica:
    """One layer's resident state on the device plus the per-step inputs and outputs."""

    def __init__(self, cfg, seed, device, ha, wl, torch, windows=(0, 0), shard=None):
        w = wl.make_workload(cfg, device, seed=seed)
        if shard is not None:                                      # (rank, world): this rank's KV heads of the workload
            w = wl.shard_heads(w, shard[0], shard[1])
        w["k_max"] += windows[0] + windows[1]                     # index rows hold the always-kept tokens too
        self.w = w
        c = w["cfg"]
        B, Hq, Hkv = c.batch, c.n_q_heads, c.n_kv_heads
        self.shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=windows[0], n_local=windows[1])
        self.mq, self.mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
        n_pad = (w["n_cap"] + 3) // 4 * 4
        self.kc = torch.zeros(B, Hkv, n_pad, dtype=torch.int32, device=device)
        ha.ha_encode(self.mk, 1, w["K"], self.kc)                 # signature cache of the prompt (not timed)
        self.qc = torch.zeros(B, Hq, dtype=torch.int32, device=device)
        self.idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=device)
        self.cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=device)
        self.out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=device)
        self.host = None
        self.host_step = None

    def pin_host(self, torch):
        w = self.w
        self.host = tuple(w[x].cpu().pin_memory() for x in ("q", "k_new", "v_new")) + \
            (torch.zeros(tuple(self.out.shape), dtype=torch.bfloat16).pin_memory(),)
        self.host_step = None


class Bench:
    def __init__(self, cfg_name, n_replicas, device, seed_base=None, windows=(0, 0), shard=None):
        import torch
        from paper_2412_14468_b200 import binding as ha
        from paper_2412_14468_b200 import workloads as wl
        self.torch, self.ha, self.wl = torch, ha, wl
        self.device = device
        cfg = wl.CONFIGS[cfg_name] if isinstance(cfg_name, str) else cfg_name
        self.cfg = cfg
        base = (wl.BASE_SEED + cfg.index) if seed_base is None else seed_base
        self.reps = [Replica(cfg, base + 100003 * r, device, ha, wl, torch, windows, shard) for r in range(n_replicas)]
        r0 = self.reps[0]
        self.ws = ha.alloc_workspace(r0.shape, max(r.w["n_cap"] for r in self.reps), max(r.w["k_max"] for r in self.reps),
                                     device=device)
        torch.cuda.synchronize()

    # --- the entry points on replica r (all enqueue on the current stream)
    def step(self, r):
        ha, w = self.ha, r.w
        ha.ha_sparse_decode(r.shape, r.mq, r.mk, w["q"], w["k_new"], w["K"], w["V"], r.kc, w["seq_lens"], w["k_per_seq"],
                            0, w["n_cap"], w["k_max"], r.qc, r.idx, r.cnt, r.out, self.ws)

    def step_host(self, r):
        """One layer-step from pinned host buffers: a prepared ha_sparse_decode_host call (arguments marshalled
        once per replica, as a decode loop that reuses its staging buffers would)."""
        if r.host_step is None:
            ha, w = self.ha, r.w
            hq, hk, hv, ho = r.host
            r.host_step = ha.SparseDecodeHostStep(r.shape, r.mq, r.mk, hq, hk, hv, w["K"], w["V"], r.kc, w["seq_lens"],
                                                  w["k_per_seq"], 0, w["n_cap"], w["k_max"], r.idx, r.cnt, ho, self.ws)
        r.host_step()

    def encode(self, r):
        ha, w = self.ha, r.w
        ha.ha_encode(r.mq, r.w["cfg"].n_q_heads // r.w["cfg"].n_kv_heads, w["q"], r.qc.unsqueeze(2))

    def score_topk(self, r):
        ha, w = self.ha, r.w
        ha.ha_score_topk(r.shape, r.qc, r.kc, w["seq_lens"], w["k_per_seq"], 0, w["n_cap"], w["k_max"], r.idx, r.cnt, self.ws)

    def gather(self, r):
        ha, w = self.ha, r.w
        ha.ha_gather_attn(r.shape, w["q"], w["K"], w["V"], w["seq_lens"], r.idx, r.cnt, w["k_max"], r.out, self.ws)

    def dense(self, r):
        ha, w = self.ha, r.w
        ha.ha_dense_decode(r.shape, w["q"], w["K"], w["V"], w["seq_lens"], w["n_cap"], r.out, self.ws)

    # --- graphs
    def capture(self, fn, n_steps, start=0):
        """CUDA graph of n_steps consecutive calls of fn, rotating over the replicas.
        Returns (graph, kernel launches inside it)."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        before = self.ha.ha_kernel_launches()
        with torch.cuda.graph(g):
            for i in range(n_steps):
                fn(self.reps[(start + i) % len(self.reps)])
        return g, self.ha.ha_kernel_launches() - before

    def time_steps(self, fn, steps, warmup, sampler=None, barrier=None, min_ms=MIN_TIMED_MS, stats=None):
        """Times regions of exactly `steps` calls of fn (graph replays of R steps + a tail graph).  The region is
        repeated, back to back on the stream with an event between two regions, until at least `min_ms` have been
        measured (5 regions at least), so that a short `steps` never yields a single sub-millisecond sample.
        Returns (MEDIAN ms per region, kernel launches in one region); `stats`, if given, receives min / median /
        max ms per region and the number of regions."""
        torch = self.torch
        R = len(self.reps)
        fn(self.reps[0])                     # eager run first: surfaces errors outside capture
        torch.cuda.synchronize()
        g_full, l_full = self.capture(fn, R)
        n_full, tail = divmod(steps, R)
        g_tail, l_tail = (self.capture(fn, tail) if tail else (None, 0))
        wf, wt = divmod(max(warmup, 0), R)
        g_wtail = self.capture(fn, wt)[0] if wt else None

        def region():
            for _ in range(n_full):
                g_full.replay()
            if g_tail:
                g_tail.replay()

        for _ in range(wf):
            g_full.replay()
        if g_wtail:
            g_wtail.replay()
        # one untimed region: warms the graphs of the region itself and sizes the number of repeats
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        region()
        e1.record()
        torch.cuda.synchronize()
        est = max(e0.elapsed_time(e1), 1e-3)
        n_regions = int(min(4000, max(5, math.ceil(min_ms / est))))
        if barrier:
            barrier()
        if sampler:
            sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_regions + 2)]
        torch.cuda.synchronize()
        ev[0].record()
        region()                             # absorbs the host's launch latency on an idle GPU; not counted
        for i in range(n_regions):
            ev[i + 1].record()
            region()
        ev[n_regions + 1].record()
        if sampler:
            sampler.sample()
        torch.cuda.synchronize()
        if sampler:
            sampler.stop()
        if barrier:
            barrier()
        ts = sorted(ev[i + 1].elapsed_time(ev[i + 2]) for i in range(n_regions))
        med = ts[len(ts) // 2]
        if stats is not None:
            stats.update({"regions": n_regions, "ms_min": ts[0], "ms_median": med, "ms_max": ts[-1]})
        return med, n_full * l_full + l_tail


def aggregate_over_ranks(elapsed_ms: float, units: float, dist=None, device=None):
    """Multi-GPU bookkeeping: the step time is the MAX over ranks, the work is the SUM.
    Returns (max elapsed ms, total units).  Works with any torch.distributed backend."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device or "cpu")
    u = torch.tensor([units], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def rank_env():
    """(world size, rank, local rank) as the launcher (torch.distributed.run) exports them."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")))


def check_gpus_flag(gpus: int, world: int) -> str:
    """What `--gpus N` asks for against the job this process is part of: "ok" (they agree), "spawn" (a plain
    `python bench.py --gpus N` with N > 1: the ranks have to be launched first) or an error message."""
    if gpus < 1:
        return f"--gpus must be >= 1, got {gpus}"
    if gpus == world:
        return "ok"
    if world == 1:
        return "spawn"
    return f"--gpus {gpus} disagrees with the launcher's WORLD_SIZE={world}: start N ranks for --gpus N"


def init_ranks(backend: str, device=None):
    """Joins the process group the launcher described in the environment (MASTER_ADDR / MASTER_PORT / RANK /
    WORLD_SIZE); returns torch.distributed, or None for a single process."""
    world, rank, _ = rank_env()
    if world == 1:
        return None
    import torch.distributed as dist
    kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
    dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return dist


def job_value(ms_region_local: float, steps: int, shard: str, dist=None, device=None):
    """Whole-job figure of a multi-rank run from every rank's own time for `steps` layer-steps.
    shard = "replicas": every rank runs its own copy of the workload (weak scaling); the job completes `world`
    layer-steps per step time, so the job's us per layer-step is the slowest rank's step time / world.
    shard = "heads": the ranks split the KV heads of ONE workload (strong scaling; no exchange on the data path);
    a layer-step is complete when the slowest rank is, so the job's us per layer-step is that rank's step time.
    Returns dict(us_per_step_rank_max, value, scaling, world)."""
    world = dist.get_world_size() if (dist is not None and dist.is_initialized()) else 1
    ms_max, total_steps = aggregate_over_ranks(ms_region_local, float(steps), dist, device)
    us_rank = ms_max * 1e3 / steps
    if shard == "heads":
        return {"us_per_step_rank_max": us_rank, "value": us_rank, "scaling": "strong", "world": world,
                "rank_steps_total": total_steps}
    return {"us_per_step_rank_max": us_rank, "value": us_rank / world, "scaling": "weak", "world": world,
            "rank_steps_total": total_steps}


# ----------------------------------------------------------------------------- CPU oracle leg

def oracle_time(cfg_name, reps, budget_s=20.0, seed=None):
    """Times the oracle's decode step (as it stands) on the host cores for the same workload.
    Returns (us per layer-step, threads used, description of the sample)."""
    import numpy as np
    import oracle
    from paper_2412_14468_b200 import workloads as wl
    w = wl.make_workload(cfg_name, "cpu", seed=seed)
    mq, mk = wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"])
    q, k_new, K, V = (wl.as_u16(w[x]) for x in ("q", "k_new", "K", "V"))
    B, Hkv, n_cap = K.shape[0], K.shape[1], K.shape[2]
    codes = np.zeros((B, Hkv, n_cap), np.uint32)
    for b in range(B):
        for g in range(Hkv):
            codes[b, g] = oracle.encode(K[b, g], mk["w1"][g], mk["w2"][g], mk["w3"][g], mk["b1"][g], mk["b2"][g], mk["b3"][g])
    threads = max(1, min(oracle.max_threads(), len(os.sched_getaffinity(0))))
    oracle.decode_step(q, k_new, K, V, codes, mq, mk, w["lens"], w["ks"], sm_scale=w["sm_scale"], n_threads=threads)
    t0 = time.perf_counter()
    n = 0
    while n < reps and (time.perf_counter() - t0) < budget_s:
        oracle.decode_step(q, k_new, K, V, codes, mq, mk, w["lens"], w["ks"], sm_scale=w["sm_scale"], n_threads=threads)
        n += 1
    dt = time.perf_counter() - t0
    return dt / n * 1e6, threads, f"{n} full layer-steps of {cfg_name} (all {B * Hkv} (sequence, KV head) units, signature cache prebuilt)"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, args.steps)
    for _ in range(min(max(args.warmup, 0), 3)):
        oracle_time("c2", 1, budget_s=5.0)
    us, threads, sample = oracle_time("c2", steps, budget_s=120.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle (plain C, OpenMP over (sequence, KV head)) on the host cores"},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32768)
    ap.add_argument("--warmup", type=int, default=4096)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--replicas", type=int, default=32)
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: every rank runs its own copy of the workload (weak scaling, the default), or the ranks "
                         "split the KV heads of one workload (strong scaling; the path has no exchange step either way)")
    ap.add_argument("--no-supplementary", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    world, rank, local = rank_env()
    if args.impl == "reference":                            # rank 0 alone runs the oracle; nothing to launch
        return run_reference(args)
    verdict = check_gpus_flag(args.gpus, world)
    if verdict == "spawn":
        # `python bench.py --gpus N` without a launcher: start the N ranks the way the driver does, one per GPU
        port = 29000 + os.getpid() % 2000
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                   f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
                                   os.path.abspath(__file__)] + sys.argv[1:])
    elif verdict != "ok":
        sys.exit("bench.py: " + verdict)

    import torch
    from paper_2412_14468_b200 import binding as ha
    from paper_2412_14468_b200 import workloads as wl

    if torch.cuda.device_count() < (local + 1):
        sys.exit(f"bench.py: rank {rank} wants cuda:{local} but only {torch.cuda.device_count()} device(s) are visible")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    dist = init_ranks("nccl", torch.device(device))
    barrier = (lambda: dist.barrier()) if dist is not None else None
    if args.shard == "heads" and wl.CONFIGS["c2"].n_kv_heads % world != 0:
        sys.exit(f"bench.py: --shard heads needs a rank count that divides the {wl.CONFIGS['c2'].n_kv_heads} KV heads")

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    peak, peak_kind = _peaks()
    R = args.replicas
    by_heads = args.shard == "heads" and world > 1
    # replicas: every rank its own seeds; heads: the same workload on every rank, each keeps its KV heads
    bench = Bench("c2", R, device, seed_base=wl.BASE_SEED + 1 + (0 if by_heads else 7919 * rank),
                  shard=(rank, world) if by_heads else None)
    cfg = bench.reps[0].w["cfg"]
    lens, ks = bench.reps[0].w["lens"], bench.reps[0].w["ks"]
    alg_bytes = wl.algorithmic_bytes(lens, ks, cfg.n_q_heads, cfg.n_kv_heads)

    # ---- headline: regions of K layer-steps of the whole path, device-resident inputs
    sampler = ClockSampler(local)
    tstats = {}
    ms, launches = bench.time_steps(bench.step, steps, warmup, sampler=sampler, barrier=barrier, stats=tstats)
    job = job_value(ms, steps, args.shard if world > 1 else "replicas", dist, device)
    us_per_step = job["us_per_step_rank_max"]               # per rank (max over ranks)
    value = job["value"]                                    # whole job
    us_min = tstats["ms_min"] * 1e3 / steps

    # ---- the same step as a decode loop sees it: every layer-step behind an ordinary kernel that writes its q
    # (a copy kernel without programmatic launch attributes standing in for the QKV projection), so that no part
    # of a step can run under its predecessor.  `value` above is the steady state of back-to-back independent
    # steps, whose prologues (weight fetch, signature requests) overlap the step in front.
    q_src = [r.w["q"].clone() for r in bench.reps]

    def q_writer(r):
        r.w["q"].copy_(q_src[bench.reps.index(r)])

    def isolated_step(r):
        q_writer(r)
        bench.step(r)

    iso_steps = min(steps, 4096)
    istats, wstats = {}, {}
    t_iso, _ = bench.time_steps(isolated_step, iso_steps, min(warmup, 256), stats=istats)
    t_wr, _ = bench.time_steps(q_writer, iso_steps, min(warmup, 256), stats=wstats)
    latency_isolated_us = (t_iso - t_wr) * 1e3 / iso_steps
    isolated = {"latency_isolated_us": latency_isolated_us, "step_plus_q_writer_us": t_iso * 1e3 / iso_steps,
                "q_writer_alone_us": t_wr * 1e3 / iso_steps, "steps": iso_steps, "regions": istats["regions"],
                "min_us": (istats["ms_min"] - wstats["ms_median"]) * 1e3 / iso_steps,
                "how": "graph of [ordinary copy kernel writing q -> ha_sparse_decode] per layer-step, minus the same graph "
                       "with the copy kernels alone"}

    # ---- per entry point (graphs over the same replicas), for the roofline of the dominant kernel
    sub_steps = min(steps, 8192)
    parts = {}
    for name, fn in (("ha_encode[q]", bench.encode), ("ha_score_topk", bench.score_topk), ("ha_gather_attn", bench.gather)):
        t, _ = bench.time_steps(fn, sub_steps, min(warmup, 1024))
        parts[name] = t * 1e3 / sub_steps
    gather_bytes = sum(cfg.n_kv_heads * 512 * min(k, n) + cfg.n_q_heads * 512 for n, k in zip(lens, ks))
    scan_bytes = sum(cfg.n_kv_heads * 4 * n for n in lens)
    launches_per_step = launches / steps
    # At this batch size the whole layer-step is ONE kernel (fused_step_kernel: one 8-CTA cluster per
    # (sequence, KV head)), so the timed region contains launches of that kernel only and its average
    # launch duration is the step time itself.
    achieved = alg_bytes / (us_per_step * 1e-6) / 1e9
    achieved_isolated = alg_bytes / (latency_isolated_us * 1e-6) / 1e9
    g_us = parts["ha_gather_attn"]
    roofline = {
        "bound": "hbm",
        "kernel": ("fused_step_kernel<4,1> (the one kernel of ha_sparse_decode at this batch size)"
                   if launches_per_step < 1.5 else "kernels of ha_sparse_decode (multi-kernel path)"),
        "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
        # dram__bytes_read.sum + dram__bytes_write.sum per launch of this kernel on this workload, from the
        # ncu launch list of this very command (profiles/launch_list_bench_c2.md)
        "traffic": TRAFFIC_FROM_PROFILE["bytes"] if (launches_per_step < 1.5 and world == 1) else None,
        "traffic_source": TRAFFIC_FROM_PROFILE if (launches_per_step < 1.5 and world == 1) else None,
        "algorithmic_bytes_per_launch": alg_bytes, "us_per_launch": us_per_step,
        "launches_per_step": launches_per_step,
        "isolated": {"us_per_launch": latency_isolated_us, "achieved": achieved_isolated, "frac": achieved_isolated / peak},
        "standalone_entry_points": {
            "ha_gather_attn (gather_cluster_kernel<4,8>)": {"algorithmic_bytes": gather_bytes, "us": g_us,
                                                      "achieved": gather_bytes / (g_us * 1e-6) / 1e9,
                                                      "frac": gather_bytes / (g_us * 1e-6) / 1e9 / peak,
                                                      "traffic": GATHER_TRAFFIC_FROM_PROFILE["bytes"],
                                                      "traffic_source": GATHER_TRAFFIC_FROM_PROFILE},
            "ha_score_topk (score_select_cluster_kernel<4,8>)": {"algorithmic_bytes": scan_bytes, "us": parts["ha_score_topk"],
                                                                    "achieved": scan_bytes / (parts["ha_score_topk"] * 1e-6) / 1e9},
            "ha_encode[q] (encode_vec_kernel<1>)": {"us": parts["ha_encode[q]"]},
        },
    }

    # ---- end to end through the host-buffer entry point (H2D of q/k_new/v_new, D2H of out, sync per step)
    for r in bench.reps:
        r.pin_host(torch)
        bench.step_host(r)            # builds the replica's prepared call (untimed)
    torch.cuda.synchronize()
    e_steps = min(steps, 2048)
    for i in range(min(warmup, 64)):
        bench.step_host(bench.reps[i % R])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = bench.ha.ha_kernel_launches()
    e0.record()
    for i in range(e_steps):
        bench.step_host(bench.reps[i % R])
    e1.record()
    torch.cuda.synchronize()
    e2e_ms, _ = aggregate_over_ranks(e0.elapsed_time(e1), float(e_steps), dist, device)
    e2e_launches = bench.ha.ha_kernel_launches() - l0
    B = cfg.batch
    e2e = {"value": e2e_ms * 1e3 / e_steps / (1 if by_heads else world), "unit": UNIT, "steps": e_steps,
           "h2d_bytes_per_step": B * (cfg.n_q_heads + 2 * cfg.n_kv_heads) * 128 * 2,
           "d2h_bytes_per_step": B * cfg.n_q_heads * 128 * 2, "gpu_launches": e2e_launches}

    # ---- same-run dense decode kernel at full context
    d_steps = min(steps, 2048)
    t_dense, _ = bench.time_steps(bench.dense, d_steps, min(warmup, 256))
    dense_us = t_dense * 1e3 / d_steps
    dbytes = wl.dense_bytes(lens, cfg.n_q_heads, cfg.n_kv_heads)
    dense = {"us_per_layer_step": dense_us, "bytes": dbytes, "achieved_gbs": dbytes / (dense_us * 1e-6) / 1e9,
             "frac": dbytes / (dense_us * 1e-6) / 1e9 / peak, "speedup_sparse_vs_dense": dense_us / us_per_step}

    supplementary = {}
    if not args.no_supplementary and world == 1:
        del bench
        torch.cuda.empty_cache()
        cases = [("c3", wl.CONFIGS["c3"], 2, 400), ("c4", wl.CONFIGS["c4"], 2, 400), ("c5", wl.CONFIGS["c5"], 2, 200)]
        for bsz in (4, 8, 16, 32, 64):   # batch sweep at the headline shape: 32K context, 32x
            cases.append((f"sweep_B{bsz}_32K_32x", wl.Config(f"sweep{bsz}", 10 + bsz, bsz, 32768, 1024, 0.01), 2 if bsz >= 16 else 8, 400))
        for name, cfg_s, reps_n, st in cases:
            try:
                b2 = Bench(cfg_s, reps_n, device)
                l2, k2 = b2.reps[0].w["lens"], b2.reps[0].w["ks"]
                ab = wl.algorithmic_bytes(l2, k2)
                t_all, _ = b2.time_steps(b2.step, st, 20)
                qs2 = [r.w["q"].clone() for r in b2.reps]           # the step behind an ordinary kernel that writes q

                def wr2(r, b2=b2, qs2=qs2):
                    r.w["q"].copy_(qs2[b2.reps.index(r)])

                def iso2(r, b2=b2, wr2=wr2):
                    wr2(r)
                    b2.step(r)
                t_iso2, _ = b2.time_steps(iso2, st, 20)
                t_wr2, _ = b2.time_steps(wr2, st, 20)
                t_sc, _ = b2.time_steps(b2.score_topk, st, 20)
                t_ga, _ = b2.time_steps(b2.gather, st, 20)
                t_de, _ = b2.time_steps(b2.dense, 40, 4)
                us = t_all * 1e3 / st
                gb = sum(8 * 512 * min(kk, nn) + 32 * 512 for nn, kk in zip(l2, k2))
                supplementary[name] = {
                    "us_per_layer_step": us, "algorithmic_bytes": ab, "achieved_gbs": ab / (us * 1e-6) / 1e9,
                    "frac": ab / (us * 1e-6) / 1e9 / peak, "latency_isolated_us": (t_iso2 - t_wr2) * 1e3 / st,
                    "frac_isolated": ab / ((t_iso2 - t_wr2) * 1e3 / st * 1e-6) / 1e9 / peak,
                    "score_topk_us": t_sc * 1e3 / st, "gather_attn_us": t_ga * 1e3 / st,
                    "gather_attn_frac": gb / (t_ga * 1e3 / st * 1e-6) / 1e9 / peak,
                    "dense_us": t_de * 1e3 / 40, "dense_frac": wl.dense_bytes(l2) / (t_de * 1e3 / 40 * 1e-6) / 1e9 / peak,
                    "replicas": reps_n,
                }
                if name in ("sweep_B64_32K_32x", "c5"):   # the other schedule of the step: scoring ahead of the row fetch in one kernel
                    def step_pipelined(r, b2=b2):
                        w = r.w
                        ha.ha_sparse_decode_pipelined(r.shape, r.mq, r.mk, w["q"], w["k_new"], w["K"], w["V"], r.kc, w["seq_lens"],
                                                      w["k_per_seq"], 0, w["n_cap"], w["k_max"], r.qc, r.idx, r.cnt, r.out, b2.ws)
                    t_pp, _ = b2.time_steps(step_pipelined, st, 20)
                    supplementary[name]["pipelined_step_us"] = t_pp * 1e3 / st
                if name == "c3":   # the same lists over a paged copy of K/V (pages of 16 tokens scattered over a pool)
                    ps, pools = 16, []
                    for r in b2.reps:
                        K, V = r.w["K"], r.w["V"]
                        Bn, Hk, N, _ = K.shape
                        pps = (N + ps - 1) // ps
                        perm = torch.randperm(Bn * pps, device=device).to(torch.int32).reshape(Bn, pps)
                        pool = []
                        for X in (K, V):
                            Xp = torch.zeros(Bn * pps, Hk, ps, 128, dtype=X.dtype, device=device)
                            Xp[perm.reshape(-1).long(), :, :, :] = torch.nn.functional.pad(X, (0, 0, 0, pps * ps - N)) \
                                .reshape(Bn, Hk, pps, ps, 128).permute(0, 2, 1, 3, 4).reshape(Bn * pps, Hk, ps, 128)
                            pool.append(Xp)
                        pools.append((pool[0], pool[1], perm))

                    def gather_paged(r):
                        Kp, Vp, perm = pools[b2.reps.index(r)]
                        ha.ha_gather_attn_paged(r.shape, r.w["q"], Kp, Vp, perm, ps, r.w["seq_lens"], r.idx, r.cnt, r.w["k_max"],
                                                r.out, b2.ws)
                    t_pg, _ = b2.time_steps(gather_paged, st, 20)
                    supplementary[name]["gather_attn_paged16_us"] = t_pg * 1e3 / st
                    # ... and the signatures in pages of 16 behind the same block tables (one 64-byte segment per page and head)
                    cpools = []
                    for r, (_, _, perm) in zip(b2.reps, pools):
                        Bn, Hk, Np = r.kc.shape
                        pps = perm.shape[1]
                        Cp = torch.zeros(Bn * pps, Hk, ps, dtype=torch.int32, device=device)
                        Cp[perm.reshape(-1).long()] = torch.nn.functional.pad(r.kc, (0, pps * ps - Np)) \
                            .reshape(Bn, Hk, pps, ps).permute(0, 2, 1, 3).reshape(Bn * pps, Hk, ps)
                        cpools.append(Cp)

                    def score_paged(r):
                        i = b2.reps.index(r)
                        ha.ha_score_topk_paged(r.shape, r.qc, cpools[i], pools[i][2], r.w["seq_lens"], r.w["k_per_seq"], 0,
                                               r.w["n_cap"], r.w["k_max"], r.idx, r.cnt, b2.ws)
                    t_sp, _ = b2.time_steps(score_paged, st, 20)
                    supplementary[name]["score_topk_paged16_us"] = t_sp * 1e3 / st
                    del pools, cpools
                del b2
                torch.cuda.empty_cache()
            except Exception as ex:   # supplementary numbers never take the headline down
                supplementary[name] = {"error": repr(ex)[:200]}
        try:   # the step before the path: signature cache of a 32K-token prompt, 8 KV heads (not part of `value`)
            gq = torch.Generator(device).manual_seed(wl.BASE_SEED + 99)
            mp = wl.make_mapping(8, gq, device)
            mm = ha.Mapping(mp)
            xk = torch.randn(1, 8, 32768, 128, device=device, generator=gq).to(torch.bfloat16)
            ck = torch.zeros(1, 8, 32768, dtype=torch.int32, device=device)
            res = {}
            f_sync = lambda m_, h_, x_, o_: ha.ha_encode_prefill(m_, h_, x_, o_, path=ha.HA_PREFILL_MMA_SYNC)
            for nm, fn in (("chain_exact_us", ha.ha_encode), ("mma_sync_us", f_sync), ("tcgen05_us", ha.ha_encode_prefill)):
                for _ in range(3):
                    fn(mm, 1, xk, ck)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(10):
                    fn(mm, 1, xk, ck)
                e1.record()
                torch.cuda.synchronize()
                res[nm] = e0.elapsed_time(e1) * 100.0
            res["algorithmic_tflops_tcgen05"] = 8 * 32768 * 2 * (128 * 128 * 2 + 128 * 32) / res["tcgen05_us"] / 1e6
            res["input_gbs_tcgen05"] = 8 * 32768 * 256 / res["tcgen05_us"] / 1e3
            supplementary["prefill_encode_32K_tokens_8_heads"] = res
            del xk, ck
            torch.cuda.empty_cache()
        except Exception as ex:
            supplementary["prefill_encode_32K_tokens_8_heads"] = {"error": repr(ex)[:200]}
        try:   # the headline shape with the first and the most recent 128 tokens always in context, budget on top
            b3 = Bench("c2", R, device, windows=(128, 128))
            t_w, _ = b3.time_steps(b3.step, 640, 64)
            l3, k3 = b3.reps[0].w["lens"], [k + 256 for k in b3.reps[0].w["ks"]]
            ab = wl.algorithmic_bytes(l3, k3)
            us = t_w * 1e3 / 640
            supplementary["c2_sink128_local128"] = {"us_per_layer_step": us, "algorithmic_bytes": ab,
                                                    "achieved_gbs": ab / (us * 1e-6) / 1e9,
                                                    "frac": ab / (us * 1e-6) / 1e9 / peak, "replicas": len(b3.reps)}
            del b3
            torch.cuda.empty_cache()
        except Exception as ex:
            supplementary["c2_sink128_local128"] = {"error": repr(ex)[:200]}

        try:   # the paper's table "Latency of SCORE computation": one query against n tokens, signatures of 64 .. 512 bits
            #      (packed 64-bit words) against the inner product with keys of 128 16-bit floats; every timed launch is
            #      L2-cold (a 256 MB buffer is rewritten in front of it)
            paper_ms = {262144: (0.13, 0.085, 0.084, 0.087, 0.112), 2097152: (1.698, 0.144, 0.247, 0.445, 0.85),
                        33554432: (16.61, 2.188, 3.817, 7.005, 13.48)}   # inner product, 64, 128, 256, 512 bit (hardware not stated)
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

            def cold_us(fn, iters=7):
                ts = []
                for _ in range(iters + 2):
                    flush.fill_(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1) * 1e3)
                return float(sorted(ts[2:])[len(ts[2:]) // 2])

            def cold_kernel_us(fn, iters=9):
                ts = []
                for _ in range(iters + 2):
                    flush.fill_(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda._sleep(300000)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1) * 1e3)
                return float(sorted(ts[2:])[len(ts[2:]) // 2])

            table = {}
            gs = torch.Generator(device).manual_seed(wl.BASE_SEED + 77)
            for n_tok, pm in paper_ms.items():
                row = {}
                Kd = torch.randn(n_tok, 128, device=device, generator=gs, dtype=torch.float32).to(torch.bfloat16) \
                    if n_tok <= (1 << 21) else torch.empty(n_tok, 128, device=device, dtype=torch.bfloat16).normal_(generator=gs)
                qd = torch.randn(128, device=device, generator=gs).to(torch.bfloat16)
                dots = torch.empty(n_tok, device=device)
                us = cold_us(lambda: ha.ha_inner_products(qd, Kd, dots))
                row["inner_product_128xbf16"] = {"us": us, "gbs": n_tok * 260 / us / 1e3, "frac": n_tok * 260 / us / 1e3 / peak,
                                                 "paper_ms": pm[0]}
                del Kd, dots
                for j, bits in enumerate((64, 128, 256, 512)):
                    W = bits // 64
                    kc = torch.randint(-2**63, 2**63 - 1, (n_tok, W), dtype=torch.int64, device=device, generator=gs)
                    qc = torch.randint(-2**63, 2**63 - 1, (W,), dtype=torch.int64, device=device, generator=gs)
                    sc = torch.empty(n_tok, dtype=torch.int16, device=device)
                    us = cold_us(lambda: ha.ha_score_wide(qc, kc, bits, sc))
                    nbytes = n_tok * (8 * W + 2)
                    row[f"hamming_{bits}bit"] = {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak,
                                                 "paper_ms": pm[1 + j]}
                    del kc, sc
                table[f"{n_tok}_tokens"] = row
                torch.cuda.empty_cache()
            supplementary["score_latency_table"] = table

            # the same table through SCORE + TOPK (ha_score_topk_wide: one query head, k = n / 32, L2-cold launches): what a
            # decode step pays for selection at each signature width, beside the 32-bit selection of the layer-step
            sel = {}
            for n_tok in paper_ms:
                row = {}
                shp1 = ha.make_shape(1, 1, 1, 1.0)
                ln = torch.full((1,), n_tok, dtype=torch.int32, device=device)
                kq = n_tok // 32
                ix = torch.zeros(1, 1, kq, dtype=torch.int32, device=device)
                ct = torch.zeros(1, 1, dtype=torch.int32, device=device)
                kc32 = torch.randint(-2**31, 2**31 - 1, (1, 1, n_tok), dtype=torch.int32, device=device, generator=gs)
                qc32 = torch.randint(-2**31, 2**31 - 1, (1, 1), dtype=torch.int32, device=device, generator=gs)
                ws32 = ha.alloc_workspace(shp1, n_tok, kq, device=device)
                us = cold_kernel_us(lambda: ha.ha_score_topk(shp1, qc32, kc32, ln, None, kq, n_tok, kq, ix, ct, ws32))
                row["hamming_32bit"] = {"us": us, "gbs": n_tok * 4 / us / 1e3, "frac": n_tok * 4 / us / 1e3 / peak}
                del kc32, ws32
                wsw = ha.alloc_workspace_wide(shp1, n_tok, device=device)
                for bits in (64, 128, 256, 512):
                    W = bits // 64
                    kcw = torch.randint(-2**63, 2**63 - 1, (1, 1, n_tok, W), dtype=torch.int64, device=device, generator=gs)
                    qcw = torch.randint(-2**63, 2**63 - 1, (1, 1, W), dtype=torch.int64, device=device, generator=gs)
                    us = cold_kernel_us(lambda: ha.ha_score_topk_wide(shp1, bits, qcw, kcw, ln, None, kq, n_tok, kq, ix, ct, wsw))
                    nbytes = n_tok * 8 * W
                    row[f"hamming_{bits}bit"] = {"us": us, "signature_gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak}
                    del kcw
                sel[f"{n_tok}_tokens"] = row
                del wsw
                torch.cuda.empty_cache()
            supplementary["score_topk_latency_by_signature_width"] = sel

            # SCORE + TOPK alone with the two group reductions (maximum: the layer-step's contract; sum: the stand-alone
            # alternative), random signatures, L2-cold launches; the GPU is kept busy while the host enqueues, so the
            # events bracket the kernels only
            red = {}
            for name, (Bq, n_tok, kq) in {"c2": (1, 32768, 1024), "c3": (16, 32768, 2048), "batch64_32K": (64, 32768, 1024),
                                          "c4": (1, 524288, 16384)}.items():
                kc = torch.randint(-2**31, 2**31 - 1, (Bq, 8, n_tok), dtype=torch.int32, device=device, generator=gs)
                qc = torch.randint(-2**31, 2**31 - 1, (Bq, 32), dtype=torch.int32, device=device, generator=gs)
                shp = ha.make_shape(Bq, 32, 8, 1.0)
                wsq = ha.alloc_workspace(shp, n_tok, kq, device=device)
                ln = torch.full((Bq,), n_tok, dtype=torch.int32, device=device)
                ix = torch.zeros(Bq, 8, kq, dtype=torch.int32, device=device)
                ct = torch.zeros(Bq, 8, dtype=torch.int32, device=device)
                nbytes = Bq * 8 * (n_tok * 4 + kq * 4)
                t_max = cold_kernel_us(lambda: ha.ha_score_topk(shp, qc, kc, ln, None, kq, n_tok, kq, ix, ct, wsq))
                t_sum = cold_kernel_us(lambda: ha.ha_score_topk_sum(shp, qc, kc, ln, None, kq, kq, ix, ct))
                ixh = torch.zeros(Bq, 32, kq, dtype=torch.int32, device=device)     # one list per query head
                cth = torch.zeros(Bq, 32, dtype=torch.int32, device=device)
                t_head = cold_kernel_us(lambda: ha.ha_score_topk_per_head(shp, qc, kc, ln, None, kq, kq, ixh, cth))
                nbytes_head = Bq * 32 * (n_tok * 4 + kq * 4)                        # every query head scans its KV head's row
                red[name] = {"algorithmic_bytes": nbytes,
                             "max_over_heads": {"us": t_max, "frac": nbytes / t_max / 1e3 / peak},
                             "sum_over_heads": {"us": t_sum, "frac": nbytes / t_sum / 1e3 / peak},
                             "per_query_head": {"us": t_head, "bytes_read_by_the_sms": nbytes_head}}
                if name == "c2":   # GATHER-ATT through the per-head lists against the grouped lists (4x the K/V rows)
                    Kr = torch.empty(Bq, 8, n_tok, 128, device=device, dtype=torch.bfloat16).normal_(generator=gs)
                    Vr = torch.empty(Bq, 8, n_tok, 128, device=device, dtype=torch.bfloat16).normal_(generator=gs)
                    qr = torch.randn(Bq, 32, 128, device=device, generator=gs).to(torch.bfloat16)
                    orr = torch.zeros(Bq, 32, 128, device=device, dtype=torch.bfloat16)
                    wsh = ha.alloc_workspace(ha.make_shape(Bq, 32, 32, 1.0), n_tok, kq, device=device)
                    ha.ha_score_topk(shp, qc, kc, ln, None, kq, n_tok, kq, ix, ct, wsq)
                    t_gg = cold_kernel_us(lambda: ha.ha_gather_attn(shp, qr, Kr, Vr, ln, ix, ct, kq, orr, wsq))
                    t_gh = cold_kernel_us(lambda: ha.ha_gather_attn_per_head(shp, qr, Kr, Vr, ln, ixh, cth, kq, orr, wsh))
                    rows = Bq * 32 * kq * 512
                    red[name]["gather_attn_grouped_lists_us"] = t_gg
                    red[name]["gather_attn_per_head_lists"] = {"us": t_gh, "row_bytes": rows, "frac": rows / t_gh / 1e3 / peak}
                    del Kr, Vr, wsh
                del kc, ix, wsq, ixh
            supplementary["score_topk_group_reductions"] = red
            del flush
            torch.cuda.empty_cache()
        except Exception as ex:
            supplementary["score_latency_table"] = {"error": repr(ex)[:200]}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        us, threads, sample = oracle_time("c2", 200, budget_s=15.0)
        cpu_baseline = {"value": us, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": us_per_step / 1e3, "higher_is_better": False, "scaling": job["scaling"], "vs_baseline": None,
            "value_kind": "steady state of back-to-back independent layer-steps (median over the timed regions); "
                          "latency_isolated_us is one step behind an ordinary kernel",
            "latency_isolated_us": latency_isolated_us, "isolated": isolated,
            "timing": {"regions": tstats["regions"], "steps_per_region": steps, "us_per_step_median": us_per_step,
                       "us_per_step_min": us_min, "us_per_step_max": tstats["ms_max"] * 1e3 / steps,
                       "timed_ms_total": tstats["ms_median"] * tstats["regions"]},
            "dtype": "bf16 in/out, fp32 accumulate; u32 signatures", "data": "synthetic",
            "config": {"workload": WORKLOAD, "replicas": R,
                       "l2": f"steps rotate over {R} layer replicas ({R * alg_bytes / 1e6:.0f} MB touched per rotation > 126 MB L2)",
                       "launch": "CUDA graphs of ha_sparse_decode calls (one fused cluster kernel per step at this batch size); `value`: steps "
                                 "back to back (their prologues overlap the step in front), `latency_isolated_us`: every step behind an "
                                 "ordinary kernel that writes its q",
                       "parallelism": (f"KV heads split over {world} ranks" if by_heads else f"replicas x{world}")},
            "clocks": sampler.summary(), "gpu_launches": launches, "e2e": e2e, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "breakdown_us": parts, "dense_same_run": dense, "supplementary": supplementary,
            "paper_context": "A100: up to 4.3x (GPT-FAST) / 2.54x (FlashDecode) attention latency reduction at 32x",
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
