"""Host-side logic of the multi-GPU path, run as two gloo ranks on CPU: every rank plans its own
seeded batch of the same shape (the path shards by request, no collective on the data path) and
the whole-job figures are the slowest rank's time and the sum of the units all ranks processed."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from paper_2604_15464_b200 import binding, build
        from paper_2604_15464_b200 import workloads as wl

        build.build()
        # each rank: its own batch of the decode shape, planned on the host (no device in this test)
        meta = wl.workload_meta(2, seed=1000 + 2 + 7919 * rank)
        rapi = binding.Rpa.for_meta(meta, device=-1)
        rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        info = rapi.rpa_plan_info()
        units = bench.units_of("decode", info, meta)
        ms = 1.0 + rank  # rank 1 is the slow one
        total_ms, total_units = bench.aggregate_over_ranks(ms, units, dist, torch.device("cpu"))
        gathered = [None] * world
        dist.all_gather_object(gathered, (int(meta.kv_lens.sum()), units))
        q.put((rank, total_ms, total_units, gathered, info["batch_case_name"]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_request_and_aggregate():
    world, port = 2, 29500 + (os.getpid() % 2000)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=240) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    results.sort()
    (r0, ms0, u0, g0, c0), (r1, ms1, u1, g1, c1) = results
    assert ms0 == ms1 == 2.0  # max over ranks
    assert c0 == c1 == "decode"
    kv0, kv1 = g0[0][0], g0[1][0]
    assert kv0 != kv1  # different seeds: the ranks do not replay the same batch
    assert u0 == u1 == pytest.approx(g0[0][1] + g0[1][1])  # whole-job units = sum over ranks


def test_head_sharding_splits_the_work_without_overlap():
    import bench
    from paper_2604_15464_b200 import binding, build
    from paper_2604_15464_b200 import workloads as wl

    build.build()
    full = wl.workload_meta(2)
    rapi = binding.Rpa.for_meta(full, device=-1)
    rapi.rpa_plan(full.cu_q_lens, full.kv_lens)
    whole = rapi.rpa_plan_info()
    parts = []
    for rank in range(4):
        meta = bench.shard_heads(wl.workload_meta(2), rank, 4)
        assert (meta.num_q_heads, meta.num_kv_heads) == (8, 2) and np.array_equal(meta.kv_lens, full.kv_lens)
        r = binding.Rpa.for_meta(meta, device=-1)
        r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        parts.append(r.rpa_plan_info())
    assert sum(p["algorithmic_bytes"] for p in parts) == whole["algorithmic_bytes"]
    assert sum(p["algorithmic_flops"] for p in parts) == whole["algorithmic_flops"]
    with pytest.raises(ValueError):
        bench.shard_heads(wl.workload_meta(2), 0, 3)


def test_bench_gpus_n_starts_n_ranks_by_itself():
    """``python bench.py --gpus 2`` outside a torchrun environment must start two ranks (it re-executes
    itself under torch.distributed.run); checked here without a device through the planning-only
    mode, in which the ranks meet over gloo and rank 0 reports the size of the job."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--plan-only"], env=env,
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1  # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["plan_only"] is True
    # two different batches of the decode shape: about twice one batch's bytes
    one = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--plan-only"], env=env, capture_output=True,
                         text=True, timeout=600)
    single = json.loads([l for l in one.stdout.splitlines() if l.startswith("{")][0])
    assert single["n_gpus"] == 1
    assert 1.7 * single["units_per_step"] < line["units_per_step"] < 2.3 * single["units_per_step"]
