#!/usr/bin/env python
"""Benchmark of the ragged paged attention hot path on B200.

A step is one pass of the whole path over one synthetic batch: host plan (rpa_plan) plus attention
with the fused cache update (rpa_forward).  The default workload is the Llama-3-8B-shaped pure
decode batch (256 requests, kv_len ~ U{512..4096}, page 16); its metric is the achieved HBM
throughput in GB/s on the algorithmic bytes of the paper's decode-throughput formula (Section
4.1.1) generalised to ragged batches.  Other workloads: ``--workload prefill|mixed|skewed``.

By default one invocation times all three legs of the metric: the decode batch is the headline line
and the Llama-3-8B-shaped prefill (4 x 8192 tokens, TFLOP/s) and mixed (192 decode + 8 x 512-token
chunks, tokens/s) batches ride along under ``"legs"``, each with its own value, roofline, end-to-end
figure, CPU baseline and clock samples.  ``--workload NAME`` runs one workload only.

Timing: W warm-up steps, then blocks of exactly K steps, each bracketed by CUDA events (and, under
torchrun, a barrier); blocks are repeated until at least ``--min-seconds`` of GPU time has been timed,
and the median block is reported.  Clock samples are taken while those blocks run.  Per-kernel event
pairs are off during the timed blocks; the kernel durations of the roofline come from a second pass.

One JSON line is printed (rank 0).  ``--impl reference`` times the fp64 CPU oracle instead.
``--gpus N`` without a torchrun environment re-executes itself under ``torch.distributed.run``.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2604_15464_b200 import metrics
from paper_2604_15464_b200 import workloads as wl

WORKLOADS = {
    # name: (config id, metric, unit, bound)
    "decode": (2, "decode_hbm_throughput", "GB/s", "hbm"),
    "prefill": (3, "prefill_tensor_throughput", "TFLOP/s", "tensor"),
    "mixed": (4, "mixed_batch_tokens_per_s", "tokens/s", "hbm"),
    "mixed4b": ("4b", "mixed_batch_tokens_per_s", "tokens/s", "hbm"),  # chunks of 1000 tokens: 8192 new tokens
    "skewed": (5, "decode_hbm_throughput", "GB/s", "hbm"),
    # the paper's own uniform grids (Section 4.1.1 and 4.2.1: page 256, Llama-3-8B heads), --ctx / --seq
    "paper_decode": (0, "decode_hbm_throughput", "GB/s", "hbm"),
    "paper_prefill": (0, "prefill_tensor_throughput", "TFLOP/s", "tensor"),
}
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu
# capture of the same workload and seed; the summary file named here holds the command and figures
# (keys: workload, dominant kernel, FP8 cache)
NCU_TRAFFIC = {("decode", "row", False): (2.3820e9, "profiles/row_kernel_llama_decode.md"),
               ("decode", "row", True): (1.1994e9, "profiles/row_kernel_fp8_llama_decode.md"),
               ("prefill", "tile", False): (0.7680e9, "profiles/pair_kernel_llama_prefill.md"),
               ("mixed", "row", False): (3.3463e9, "profiles/mixed_llama_launch_list.md")}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self._stop = threading.Event()
        self._thread = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [x.strip() for x in out.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=6)

    def summary(self) -> dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(float(s[0]) for s in self.samples if s[0].replace(".", "").isdigit())
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(s[2 + k].lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": float(self.samples[0][1]),
                "reasons": reasons, "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        ids = [x for x in vis.split(",") if x.strip() != ""]
        if local < len(ids) and ids[local].strip().isdigit():
            return int(ids[local])
    return local


def shard_heads(meta, rank: int, world: int):
    """Tensor-parallel shard of a batch by KV head (the paper's TP sharding of h_kv, Section 3.1.1):
    every rank serves all requests for its own h_kv/world KV heads and their query heads, on its
    own slice of every cache page.  No exchange step: attention is independent per KV head."""
    if meta.num_kv_heads % world:
        raise ValueError(f"{meta.num_kv_heads} KV heads do not split over {world} ranks")
    h_g = meta.num_q_heads // meta.num_kv_heads
    meta.num_kv_heads //= world
    meta.num_q_heads = meta.num_kv_heads * h_g
    meta.name += f"_tp{world}r{rank}"
    return meta


def make_meta(workload: str, rank: int, pool_gb: float | None, args=None):
    cfg = WORKLOADS[workload][0]
    by_heads = args is not None and getattr(args, "shard", "requests") == "heads"
    # sharding by request: every rank draws its own batch of the same shape (weak scaling);
    # sharding by KV head: all ranks see the same requests and split the heads (strong scaling)
    seed = 1000 + (4 if cfg == "4b" else cfg) + (0 if by_heads else 7919 * rank)
    if workload == "paper_decode":  # n = 128 requests of identical context length, one new token each
        n, ctx = args.paper_n or 128, args.ctx
        shape = dict(wl.LLAMA3_8B, head_dim=args.head_dim)
        return wl.build_meta(f"paper_decode_ctx{ctx}_d{args.head_dim}", [1] * n, [ctx + 1] * n, page_size=args.page_size,
                             seed=seed, causal=not args.noncausal, **shape)
    if workload == "paper_prefill":  # one request of s new tokens, no cached context
        n, s_len = args.paper_n or 1, args.seq
        shape = dict(wl.LLAMA3_8B, head_dim=args.head_dim)
        return wl.build_meta(f"paper_prefill_s{s_len}_d{args.head_dim}", [s_len] * n, [s_len] * n, page_size=args.page_size,
                             seed=seed, causal=not args.noncausal, **shape)
    if cfg == 5:
        free, _ = torch.cuda.mem_get_info()
        page_bytes = 128 * 2 * 8 * 128 * 2
        want = 150e9 if pool_gb is None else pool_gb * 1e9
        pages = int(min(want, 0.8 * free) // page_bytes)
        return wl.workload_meta(5, seed, num_pages=pages)
    return wl.workload_meta(cfg, seed)


def aggregate_over_ranks(ms: float, units: float, dist, device) -> tuple:
    """Whole-job figures from per-rank ones: the slowest rank's time and the sum of the units all
    ranks processed.  ``dist`` is torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return ms, units
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    u = torch.tensor([units], device=device, dtype=torch.float64)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def units_of(workload: str, info: dict, meta) -> float:
    if workload in ("decode", "skewed", "paper_decode"):
        return info["algorithmic_bytes"] / 1e9  # GB
    if workload in ("prefill", "paper_prefill"):
        return info["algorithmic_flops"] / 1e12  # TFLOP
    return float(meta.num_tokens)  # tokens


def oracle_sample(meta, batch, budget_s: float = 15.0, rate: float | None = None):
    """Times the CPU oracle, as it stands, on a bounded sample of the batch's requests.  ``rate`` is
    the oracle's speed (nominal FLOP/s over all cores) used to size the sample; the time is measured.
    Returns (seconds, units-dict of the sample, description, cores, nominal FLOPs of the sample)."""
    from oracle import rpa_oracle as orc  # CPU-baseline leg only

    cost = meta.q_lens.astype(np.float64) * meta.kv_lens * meta.num_q_heads * meta.head_dim * 4  # ~flops
    cores = orc.threads()
    if rate is None:
        rate = 0.35e9 * cores  # conservative fp64 scalar rate for a first, short sample
    pick, acc = [], 0.0
    for r in np.random.default_rng(5).permutation(meta.num_seqs):
        if meta.q_lens[r] == 0:
            continue
        if pick and acc + cost[r] > budget_s * rate:
            continue
        pick.append(int(r))
        acc += cost[r]
        if acc > budget_s * rate:
            break
    pick.sort()
    host, n_pages, _, _ = wl.host_subset(batch, pick)
    shape = orc.OracleShape(meta.num_q_heads, meta.num_kv_heads, meta.head_dim, meta.page_size, n_pages,
                            meta.max_pages_per_seq, meta.sm_scale, meta.causal, meta.kv_fp8, meta.k_scale, meta.v_scale, meta.q_scale)
    triples = [(k, i, a) for k, r in enumerate(pick) for i in range(int(meta.q_lens[r])) for a in range(meta.num_q_heads)]
    frac = 1.0
    if acc > 1.5 * budget_s * rate:  # a single request may still be too long (full prefill): sample its rows
        total_rows = len(triples)
        keep = max(1, int(total_rows * budget_s * rate / acc))
        sel = np.random.default_rng(6).choice(total_rows, size=keep, replace=False)
        triples = [triples[i] for i in sorted(sel)]
        frac = keep / total_rows
    t0 = time.perf_counter()
    orc.update_cache(shape, host["new_k"], host["new_v"], host["kv_cache"], host["page_table"], host["cu_q_lens"],
                     host["kv_lens"])
    orc.attend_rows(shape, host["q"], host["kv_cache"], host["page_table"], host["cu_q_lens"], host["kv_lens"], triples)
    dt = time.perf_counter() - t0
    ql, kl = meta.q_lens[pick], meta.kv_lens[pick]
    units = {
        # (an FP8 cache moves one byte per cached element; Q and the output stay bf16)
        "GB": frac * (metrics.algorithmic_bytes(ql, kl, meta.num_q_heads, meta.num_kv_heads, meta.head_dim)
                      - (float((kl + ql).sum()) * 2 * meta.num_kv_heads * meta.head_dim if meta.kv_fp8 else 0.0)) / 1e9,
        "TFLOP": frac * metrics.attention_flops(ql, kl, meta.num_q_heads, meta.head_dim, meta.causal) / 1e12,
        "tokens": frac * float(ql.sum()),
    }
    n_live = int((meta.q_lens > 0).sum())
    whole = len(pick) == n_live and frac == 1.0
    what = f"{len(pick)} of {meta.num_seqs} requests" + (f", {len(triples)} sampled (token, head) rows" if frac < 1 else ", all rows")
    return dt, units, what, cores, (frac * acc, whole)


def cpu_baseline_of(meta, batch, unit, budget_s):
    """The oracle on a sample sized for about ``budget_s`` seconds of CPU work: a first short sample
    measures its speed on this machine and this workload, a second one is sized with that speed (unless
    the first already covered the whole batch)."""
    dt, units, what, cores, (flops, whole) = oracle_sample(meta, batch, budget_s=min(budget_s, 3.0))
    if not whole and dt < 0.6 * budget_s:
        dt, units, what, cores, _ = oracle_sample(meta, batch, budget_s=budget_s, rate=max(flops / max(dt, 1e-3), 1e6))
    return {"value": units[unit_key(unit)] / dt, "unit": unit, "cores": cores, "kind": "oracle", "sample": what, "seconds": dt}


def unit_key(unit: str) -> str:
    return {"GB/s": "GB", "TFLOP/s": "TFLOP", "tokens/s": "tokens"}[unit]


def run_reference(args):
    """The reference arm: the fp64 CPU oracle on the host cores, bounded samples of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg, metric, unit, _ = WORKLOADS[args.workload]
    if args.workload.startswith("paper_"):
        meta = make_meta(args.workload, 0, None, args)
    else:
        meta = wl.workload_meta(cfg, num_pages=None if cfg != 5 else 40000)
    batch = wl.materialize(meta, "cpu")
    times, total_units, what, cores, rate = [], 0.0, "", 1, None
    budget = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    for step in range(args.warmup + args.steps):
        dt, units, what, cores, (flops, _) = oracle_sample(meta, batch, budget_s=budget, rate=rate)
        if step == 0 and args.warmup > 0:  # the first warm-up sample calibrates the size of the later ones
            rate = max(flops / max(dt, 1e-3), 1e6)
        if step >= args.warmup:
            times.append(dt)
            total_units += units[unit_key(unit)]
    value = total_units / sum(times)
    line = {
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": meta.name, "sample": what},
        "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": what + " per step"},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def device_plan_launches(meta):
    """Kernels one device-planned step launches (fixed grids; the lists decide which of them work)."""
    group = meta.num_q_heads // meta.num_kv_heads
    rows = 2 if (meta.kv_fp8 and group <= 8) else 1
    tiles = (2 if meta.head_dim in (128, 256) else 0) if meta.kv_fp8 else 1  # FP8 tile paths exist at head_dim 128 and 256
    return 1 + rows + tiles


def median(xs):
    xs = sorted(xs)
    return xs[len(xs) // 2] if len(xs) % 2 else 0.5 * (xs[len(xs) // 2 - 1] + xs[len(xs) // 2])


def timed_blocks(run_block, steps, min_seconds, dist, device, max_blocks=4000):
    """Runs blocks of exactly ``steps`` steps until ``min_seconds`` of GPU time has been timed (at
    least one block, at most ``max_blocks``).  Every block is bracketed by a synchronize (and a barrier
    under torchrun) on both sides and timed with CUDA events on the launching stream; a block's time is
    the slowest rank's.  Returns the per-block times in ms."""
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times, total = [], 0.0
    while len(times) < max_blocks:
        if dist:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record(stream)
        run_block(steps)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if dist:  # all ranks must agree on the block's time, hence on when to stop
            t = torch.tensor([ms], device=device, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        times.append(ms)
        total += ms
        if total >= 1e3 * min_seconds:
            break
    return times


def run_leg(workload, args, rank, world, local, dist, peaks):
    """Everything bench.py reports for one workload; returns the dict of its JSON line (rank 0's view)."""
    from paper_2604_15464_b200 import binding

    device = torch.device("cuda", local)
    cfg, metric, unit, bound = WORKLOADS[workload]
    meta = make_meta(workload, rank, args.pool_gb, args)
    if args.shard == "heads" and world > 1:
        meta = shard_heads(meta, rank, world)
    if args.kv_fp8:
        meta.kv_fp8, meta.k_scale, meta.v_scale = True, 0.02, 0.02
        meta.name += "_fp8kv"
        if args.q_fp8:
            meta.q_scale = 0.02
            meta.name += "q"
    batch = wl.materialize(meta, device)
    rapi = binding.Rpa.for_meta(meta, device=local)
    if args.kv_chunk:
        rapi.rpa_set_kv_chunk(args.kv_chunk)
    if args.ablate:
        rapi.rpa_set_ablation(args.ablate)
    if args.tile_pair is not None:
        rapi.rpa_set_tile_pair(args.tile_pair)
    out = torch.zeros_like(batch.q)
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    cu_h, kl_h = meta.cu_q_lens, meta.kv_lens

    # Device-made plans: the plan of the step after this one is enqueued on a side stream as soon as
    # this step's kernels are (a serving loop knows the next lengths by then); the library orders the
    # two sets of lists with events.  Every step still launches one plan kernel and one forward.
    plan_stream = torch.cuda.Stream(priority=-1) if args.plan == "device" else None
    planned_ahead = [False]

    def step():
        if args.plan == "device":
            if not planned_ahead[0]:
                rapi.rpa_plan_device(batch.cu_q_lens, batch.kv_lens, plan_stream.cuda_stream)
        else:
            rapi.rpa_plan(cu_h, kl_h, sh)
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, sh)
        if args.plan == "device":
            rapi.rpa_plan_device(batch.cu_q_lens, batch.kv_lens, plan_stream.cuda_stream)
            planned_ahead[0] = True

    def run_steps(k):
        for _ in range(k):
            step()

    rapi.rpa_plan(cu_h, kl_h, sh)  # the counts reported below come from the host planner in either mode
    info = rapi.rpa_plan_info()
    planned_ahead[0] = False
    run_steps(args.warmup)
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, per-kernel events off, clocks sampled while it runs ----
    with ClockSampler(physical_gpu_index(local)) as clocks:
        block_ms = timed_blocks(run_steps, args.steps, args.min_seconds, dist, device)
    _, units_per_step = aggregate_over_ranks(0.0, units_of(workload, info, meta), dist, device)
    ms_per_step = median(block_ms) / args.steps
    value = units_per_step / (ms_per_step * 1e-3)

    # ---- roofline of the dominant kernel (this rank): a second pass with event pairs around each launch ----
    rapi.rpa_set_kernel_timing(True)
    run_steps(args.steps)
    torch.cuda.synchronize()
    kt = rapi.rpa_get_kernel_timing()
    rapi.rpa_set_kernel_timing(False)
    busy_ms = sum(block_ms)

    def kernel_roofline(kind):
        total_ms, launches = kt[kind]
        if launches == 0:
            return None
        k_ms = total_ms / launches
        if kind == "tile":  # dense contractions on the tensor cores
            achieved = info["tile_flops"] / 1e12 / (k_ms * 1e-3)
            # the cuBLAS burst figure: the larger (stricter) denominator; the sustained one is given beside it
            peak = float(peaks["bf16_tflops"])
            kbound, runit, nominal = "tensor", "TFLOP/s", NOMINAL_BF16_TFLOPS
        else:  # the split-KV row kernel streams the cache: HBM
            achieved = info["row_bytes"] / 1e9 / (k_ms * 1e-3)
            peak, kbound, runit, nominal = float(peaks["hbm_gbs"]), "hbm", "GB/s", NOMINAL_HBM_GBS
        kname = {"tile": {2: "rpa_tile1_kernel", 3: "rpa_tile2_kernel"}.get(info.get("tile_kernel", 1), "rpa_tile_kernel")}.get(kind, f"rpa_{kind}_kernel")
        r = {"bound": kbound, "kernel": kname, "achieved": achieved, "peak": peak, "unit": runit,
             "frac": achieved / peak, "peak_source": peaks["_source"], "traffic": None, "kernel_ms": k_ms,
             "kernel_launches": launches, "kernel_share_of_step": k_ms / max(1e-9, ms_per_step),
             "frac_of_nominal": achieved / nominal}
        if kind == "tile":
            r["frac_of_sustained_peak"] = achieved / float(peaks["bf16_tflops_sustained"])
        return r

    dom = max(("row", "tile", "combine"), key=lambda k: kt[k][0])
    roofline = kernel_roofline(dom)
    other = [kernel_roofline(k) for k in ("row", "tile") if k != dom and kt[k][1] > 0]
    traffic_key = (workload, dom, bool(meta.kv_fp8))
    if roofline and traffic_key in NCU_TRAFFIC and rank == 0 and meta.seed == 1000 + (4 if cfg == "4b" else cfg) and args.plan == "host":
        roofline["traffic"], roofline["traffic_source"] = NCU_TRAFFIC[traffic_key]

    # ---- end to end: host buffers through rpa_forward_host, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        T, n = meta.num_tokens, meta.num_seqs
        pin = lambda t: t.detach().cpu().pin_memory()
        hq, hk, hv = pin(batch.q), pin(batch.new_k), pin(batch.new_v)
        hpt, hcu, hkl = pin(batch.page_table), pin(batch.cu_q_lens), pin(batch.kv_lens)
        houts = [torch.zeros(batch.q.shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]

        def e2e_steps(k):
            # Two steps in flight, as a serving loop would keep them: step i+1 is submitted (planned,
            # its input copies enqueued) before step i's output is waited for, so the copies of one step
            # run beside the kernels of its neighbours.  Every step still copies all of its inputs from
            # pinned host memory and delivers its output rows to the host.
            for i in range(k):
                rapi.rpa_forward_host_submit(hq, hk, hv, batch.kv_cache, hpt, hcu, hkl, houts[i & 1], sh)
                if i > 0:
                    rapi.rpa_forward_host_wait()
            rapi.rpa_forward_host_wait()

        def e2e_serial(k):  # one at a time: rpa_forward_host returns with the output on the host
            for i in range(k):
                rapi.rpa_forward_host(hq, hk, hv, batch.kv_cache, hpt, hcu, hkl, houts[i & 1], sh)

        e2e_steps(3)
        ms_e2e = median(timed_blocks(e2e_steps, args.steps, 0.5 * args.min_seconds, dist, device, max_blocks=400)) / args.steps
        n_serial = max(3, args.steps // 4)
        ms_serial = median(timed_blocks(e2e_serial, n_serial, 0.25 * args.min_seconds, dist, device, max_blocks=400)) / n_serial
        row_q = meta.num_q_heads * meta.head_dim * 2
        row_k = meta.num_kv_heads * meta.head_dim * 2
        h2d = T * (row_q + 2 * row_k) + n * meta.max_pages_per_seq * 4 + (2 * n + 1) * 4 + info["num_row_items"] * 32
        e2e = {"value": units_per_step / (ms_e2e * 1e-3), "unit": unit, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(T * row_q), "ms_per_step": ms_e2e,
               "steps_in_flight": 2,
               "one_step_in_flight": {"value": units_per_step / (ms_serial * 1e-3), "ms_per_step": ms_serial,
                                      "steps": n_serial},
               "note": "rpa_forward_host_submit / rpa_forward_host_wait, two steps in flight: every step copies its "
                       "inputs from pinned host memory and its output back; the KV cache stays resident in HBM"}

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N=1 only ----
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = cpu_baseline_of(meta, batch, unit, args.cpu_budget)

    rapi.close()
    clock_summary = clocks.summary()
    # the same figure per GHz of the SM clock sampled during the timed blocks: under the power cap the
    # clock moves from run to run, and this tells a slower kernel from a slower clock
    per_ghz = value / (clock_summary["sm_mhz"] / 1e3) if clock_summary.get("sm_mhz") else None
    launches_per_step = device_plan_launches(meta) if args.plan == "device" else info["gpu_launches"]
    return {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if (args.shard == "heads" and world > 1) else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": meta.name, "kv_cache": "fp8_e4m3" if meta.kv_fp8 else "bf16",
                   "num_seqs": meta.num_seqs, "num_tokens": meta.num_tokens,
                   "kv_tokens": int(meta.kv_lens.sum()), "heads": f"{meta.num_q_heads}q/{meta.num_kv_heads}kv",
                   "head_dim": meta.head_dim, "page_size": meta.page_size, "num_pages": meta.num_pages,
                   "causal": bool(meta.causal), "batch_case": info["batch_case_name"], "row_items": info["num_row_items"],
                   "tile_items": info["num_tile_items"], "combine_groups": info["num_combine_groups"],
                   "kv_chunk_tokens": info["kv_chunk_tokens"], "parallelism": (f"tp{world}" if args.shard == "heads" and world > 1 else f"dp{world}"),
                   "step": ("rpa_plan_device (for the next step, on a side stream)" if args.plan == "device" else "rpa_plan") + " + rpa_forward",
                   "l2": ("KV working set %.2f GB per step exceeds the 126 MB L2; no flush needed" % (info["algorithmic_bytes"] / 1e9))
                         if bound == "hbm" else "compute-bound: K/V re-reads through L2 are part of the method; no flush"},
        "timing": {"blocks": len(block_ms), "steps_per_block": args.steps, "gpu_seconds_timed": busy_ms * 1e-3,
                   "block_ms_median": median(block_ms), "block_ms_min": min(block_ms), "block_ms_max": max(block_ms),
                   "per_kernel_events_in_timed_blocks": False},
        "clocks": clock_summary,
        "value_per_sm_ghz": per_ghz,
        "roofline": roofline,
        "roofline_other_kernels": other,
        "e2e": e2e,
        "cpu_baseline": cpu_baseline,
        # device-planned steps always launch the plan kernel and every attention kernel the handle
        # may need: with an FP8 cache the 8-row and the 16-row instantiation of the row kernel (when
        # there are at most 8 grouped heads) and the quantising pass before the tile kernel
        "gpu_launches": args.steps * launches_per_step,
        "gpu_launches_per_step": launches_per_step,
        "mbu_vs_nominal_8TBs": value / NOMINAL_HBM_GBS / world if unit == "GB/s" else None,
        "mfu_vs_nominal_2250": value / NOMINAL_BF16_TFLOPS / world if unit == "TFLOP/s" else None,
        "achieved_gbs": info["algorithmic_bytes"] / 1e9 / (ms_per_step * 1e-3),
        "achieved_tflops": info["algorithmic_flops"] / 1e12 / (ms_per_step * 1e-3),
    }


def run_plan_only(args):
    """No device: every rank plans its shard of the headline batch on the host (gloo for the
    aggregation) and rank 0 prints what the launch would cover.  Exercises the launch plumbing of
    ``--gpus N`` on a machine without GPUs; no throughput is reported."""
    from paper_2604_15464_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("gloo")
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()
    workload = "decode" if args.workload == "all" else args.workload
    meta = wl.workload_meta(WORKLOADS[workload][0], seed=1000 + 2 + 7919 * rank) if workload == "decode" else make_meta(workload, rank, 1.0, args)
    rapi = binding.Rpa.for_meta(meta, device=-1)
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    info = rapi.rpa_plan_info()
    _, units = aggregate_over_ranks(0.0, units_of(workload, info, meta), dist, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"plan_only": True, "metric": WORKLOADS[workload][1], "value": None, "unit": WORKLOADS[workload][2],
                          "n_gpus": world, "units_per_step": units, "config": {"workload": meta.name}}))
    if dist:
        dist.destroy_process_group()
    return 0


def respawn_under_torchrun(args) -> int:
    """``--gpus N`` outside a torchrun environment: start N ranks of this script, one per GPU."""
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=sorted(WORKLOADS) + ["all"],
                    help="all: the decode batch as the headline line with the prefill and mixed batches under \"legs\"")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="blocks of --steps steps are repeated until this much GPU time has been timed; the median block is reported")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of CPU work the oracle sample of each leg is sized for")
    ap.add_argument("--pool-gb", type=float, default=None, help="cache pool size for the skewed workload")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--plan-only", action="store_true", help="no device: plan the headline batch on every rank and print the launch's shape")
    ap.add_argument("--kv-chunk", type=int, default=0)
    ap.add_argument("--tile-pair", type=int, default=None, choices=[0, 1], help="rpa_set_tile_pair: tile items on the CTA-pair kernel (1) or the two-tile kernel (0)")
    ap.add_argument("--ablate", type=int, default=0, help="rpa_set_ablation mask (1: no cache update, 2: no kernel overlap, 4: no attention arithmetic, 8: no K/V loads)")
    ap.add_argument("--ctx", type=int, default=8192, help="context length of the paper_decode workload")
    ap.add_argument("--seq", type=int, default=8192, help="sequence length of the paper_prefill workload")
    ap.add_argument("--paper-n", type=int, default=0, help="requests in the paper_* workloads (default 128 / 1)")
    ap.add_argument("--page-size", type=int, default=256, help="page size of the paper_* workloads")
    ap.add_argument("--noncausal", action="store_true", help="paper_* workloads without the causal mask")
    ap.add_argument("--head-dim", type=int, default=128, help="head dimension of the paper_* workloads (128 or 256)")
    ap.add_argument("--kv-fp8", action="store_true", help="FP8 E4M3 cache with per-tensor scales (decode workloads)")
    ap.add_argument("--q-fp8", action="store_true", help="with --kv-fp8: Q is quantised to E4M3 with a per-tensor scale as well")
    ap.add_argument("--plan", default="host", choices=["host", "device"],
                    help="who builds the work lists each step: rpa_plan on the host, or rpa_plan_device on the GPU")
    ap.add_argument("--shard", default="requests", choices=["requests", "heads"],
                    help="how N ranks split the work: own requests each (weak scaling) or own KV heads each (strong)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return respawn_under_torchrun(args)
    if args.impl == "reference":
        if args.workload == "all":
            args.workload = "decode"
        return run_reference(args)
    if args.plan_only:
        return run_plan_only(args)

    from paper_2604_15464_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()
    binding.load_library()
    peaks = load_peaks()

    names = ["decode", "prefill", "mixed"] if args.workload == "all" else [args.workload]
    line = run_leg(names[0], args, rank, world, local, dist, peaks)
    if len(names) > 1:
        line["legs"] = {}
        for name in names[1:]:
            torch.cuda.empty_cache()
            line["legs"][name] = run_leg(name, args, rank, world, local, dist, peaks)
        line["gpu_launches_all_legs"] = line["gpu_launches"] + sum(l["gpu_launches"] for l in line["legs"].values())
    if dist:
        dist.barrier()
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
