"""The N>1 bookkeeping of bench.py on CPU: two gloo ranks, step time = MAX over ranks, work = SUM
(the path itself shards by replicas only: no data-path collective exists)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    elapsed, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist, "cpu")
    dist.barrier()
    q.put((rank, elapsed, units))
    dist.destroy_process_group()


def test_max_time_and_summed_units_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 15.0, 300.0), (1, 15.0, 300.0)]


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0) == (3.5, 7.0)
    assert bench.job_value(2.0, 100, "replicas") == {"us_per_step_rank_max": 20.0, "value": 20.0, "scaling": "weak",
                                                     "world": 1, "rank_steps_total": 100.0}


def test_gpus_flag_against_the_launchers_world_size():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.check_gpus_flag(1, 1) == "ok" and bench.check_gpus_flag(8, 8) == "ok"
    assert bench.check_gpus_flag(4, 1) == "spawn"                    # plain `python bench.py --gpus 4`: ranks must be started
    assert "disagrees" in bench.check_gpus_flag(2, 4) and "disagrees" in bench.check_gpus_flag(1, 2)
    assert ">= 1" in bench.check_gpus_flag(0, 1)


def _job_worker(rank, world, port, q):
    """The world > 1 branch of bench.main() without CUDA: rank environment -> process group (gloo here, nccl on
    GPUs) -> whole-job value for both ways of sharding -> teardown."""
    sys.path.insert(0, ROOT)
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank), "LOCAL_RANK": str(rank),
                       "WORLD_SIZE": str(world)})
    import bench
    assert bench.rank_env() == (world, rank, rank)
    assert bench.check_gpus_flag(world, bench.rank_env()[0]) == "ok"
    d = bench.init_ranks("gloo")
    assert d is not None and d.get_world_size() == world
    ms_local = 4.0 + 2.0 * rank                                       # this rank's time for 200 steps
    weak = bench.job_value(ms_local, 200, "replicas", d, "cpu")
    strong = bench.job_value(ms_local, 200, "heads", d, "cpu")
    d.barrier()
    q.put((rank, weak, strong))
    d.destroy_process_group()


def test_whole_job_value_over_two_gloo_ranks_for_replicas_and_for_head_shards():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 27500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_job_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, weak, strong in res:
        # slowest rank: 6 ms for 200 steps = 30 us per step; two replicas complete two steps in that time
        assert weak == {"us_per_step_rank_max": 30.0, "value": 15.0, "scaling": "weak", "world": 2, "rank_steps_total": 400.0}
        # head shards: one layer-step is complete when the slowest rank is
        assert strong == {"us_per_step_rank_max": 30.0, "value": 30.0, "scaling": "strong", "world": 2, "rank_steps_total": 400.0}


def test_init_ranks_is_a_no_op_for_a_single_process(monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    assert bench.rank_env() == (1, 0, 0) and bench.init_ranks("gloo") is None


# ---- head-parallel split: every rank runs the whole step on its KV heads, nothing is exchanged on the data path

def _oracle_step(w):
    import oracle
    from paper_2412_14468_b200 import workloads as wl
    from tests._util import oracle_key_codes, u16
    Kc = oracle_key_codes(w["K"].contiguous(), w["map_k"], w["lens"])
    return oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"].contiguous()), u16(w["V"].contiguous()), Kc,
                              wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                              sm_scale=w["sm_scale"], n_threads=1)


def _head_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2412_14468_b200 import workloads as wl
    cfg = wl.Config("head-shards", 61, 2, [300, 77], None, 0.02, n_q_heads=8, n_kv_heads=4, sparsity=8)
    w = wl.make_workload(cfg, "cpu")                       # the same seeded inputs on every rank
    mine = _oracle_step(wl.shard_heads(w, rank, world))
    out = torch.from_numpy(mine["out"].astype("int32"))    # bf16 bit patterns [B, Hq / world, 128]
    idx = torch.from_numpy(mine["idx"].astype("int32"))
    outs = [torch.empty_like(out) for _ in range(world)]
    idxs = [torch.empty_like(idx) for _ in range(world)]
    dist.all_gather(outs, out)                             # assembling the result is the only communication
    dist.all_gather(idxs, idx)
    ok = None
    if rank == 0:
        whole = _oracle_step(w)
        ok = bool((torch.cat(outs, dim=1).numpy() == whole["out"].astype("int32")).all()
                  and (torch.cat(idxs, dim=1).numpy() == whole["idx"].astype("int32")).all())
    dist.barrier()
    q.put((rank, ok))
    dist.destroy_process_group()


def test_head_parallel_shards_over_two_gloo_ranks_reassemble_the_whole_step():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_head_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=240) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True), (1, None)]
