#!/usr/bin/env python
"""Benchmark of the truncated-quantization hot path on B200.

A step is one full round over one batch of synthetic heavy-tailed gradients already resident in
HBM: statistics (default: one pass, g_min = mean|g| rounded down to a power of two, hinted by the
previous round's mean; --stats two-pass: moments, then the tail beyond g_min = mean|g|) ->
closed-form parameters (the 64-byte records are copied back and designed on the host: one sync per
round; --device-params designs them on the device instead, with no host round trip) -> fused
truncate + stochastic round + pack for all N workers -> fused unpack + dequantize + average.
Throughput is bytes of gradient input (N * d * elemsize) per second of step time.

The headline numbers (value, roofline, e2e, cpu_baseline) are those of --config (default: 25.6 M x 16
fp32).  On one GPU the line also carries, under "workloads", the per-kernel times (median, min, mean),
algorithmic bytes, fraction of the measured copy peak and sampled clocks of the other workloads with
d >= 25.6 M: 124 M x 8 stored as bf16 (uniform and non-uniform, 4 and 16 levels) and 10^9 x 4; each is
generated, timed and freed in turn (--no-workloads leaves them out).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With --gpus N > 1 (under torchrun) every rank runs its own replica
of the workload on its own GPU -- the path has no exchange step on one node, so there is no
collective in the data path -- and the value is the sum over ranks divided by the slowest rank's
time.  --impl reference times the CPU oracle (plain single-threaded C) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress & decompress-aggregate GB/s of fp32 gradient, % of B200 HBM peak"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/compress_kernel_resnet50-25.6M.md (valid for the kernel as it stands; None elsewhere)
NCU_DRAM_BYTES = {("resnet50-25.6M", "tq_compress"): 1_837_323_352}


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.index, self.period, self.samples, self.reasons, self.mem_samples = index, period_s, [], set(), []
        self.max_mhz, self.stop_flag, self.thread, self.err = None, False, None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if idx < len(ids) and ids[idx].isdigit():
                    idx = int(ids[idx])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:            # no NVML: report that instead of clocks
            self.err = repr(e)
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
        while not self.stop_flag:
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.mem_samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_MEM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for nm, bit in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
            except Exception as e:
                self.err = repr(e)
                break
            time.sleep(self.period)

    def stop(self):
        self.stop_flag = True
        if self.thread:
            self.thread.join(timeout=2)
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "mem_mhz": statistics.median(self.mem_samples) if self.mem_samples else None,
               "samples": len(self.samples), "reasons": sorted(self.reasons)}
        if self.err:
            out["error"] = self.err
        return out


def replica_workload(w, rank: int):
    """The workload rank `rank` runs: the same shapes with its own seeds (a replica, not a shard)."""
    from dataclasses import replace
    return replace(w, base_seed=w.base_seed + 1000 * rank)


def max_over_ranks(ms: float, world: int, device="cpu") -> float:
    """Slowest rank's time: the only cross-rank exchange of the benchmark (timing, not data)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(world: int, bytes_per_rank: int, ms: float) -> float:
    """Aggregate throughput of all ranks: every rank processes bytes_per_rank in the slowest rank's time."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def cpu_oracle_round(w, sample_d: int, seed: int = 0, stats_rule: str = "hinted"):
    """One round of the path by the CPU oracle on `sample_d` elements per worker.  Returns seconds."""
    import numpy as np
    import torch

    import oracle
    from paper_2402_01798_b200 import inputs
    oracle.lib()
    mode = oracle.NONUNIFORM if w.mode == "nonuniform" else oracle.UNIFORM
    grads = []
    for i in range(w.n_workers):
        t = inputs.powerlaw_gradient(sample_d, w.gamma, w.scale, w.base_seed + i, "cpu", w.dtype,
                                     w.outlier_frac, w.outlier_mult)
        raw = t.view(torch.int16).numpy().view(np.uint16) if w.dtype == torch.bfloat16 else t.numpy()
        grads.append(raw)
    t0 = time.perf_counter()
    ps, rows = [], []
    for i, raw in enumerate(grads):
        x = oracle.bf16_to_f32(raw) if w.dtype == torch.bfloat16 else raw
        st = oracle.stats_pow2(x) if stats_rule == "hinted" else oracle.stats(x)      # same g_min rule as the GPU arm
        p = oracle.params(st, w.num_levels, mode, w.gamma)
        ps.append(p)
        rows.append(oracle.compress(x, p, seed, i))
    out = oracle.decompress_aggregate(np.stack(rows), sample_d, ps)
    dt = time.perf_counter() - t0
    assert out.shape == (sample_d,)
    return dt


def run_reference(args, w):
    """--impl reference: the oracle as it stands, on host cores, each step a bounded sample."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    esz = 2 if w.dtype == torch.bfloat16 else 4
    # bounded sample: about 1.5e9 element-rounds over the whole run (a couple of minutes of one core)
    sample_d = min(w.d, max(1 << 16, int(1.5e9 / max(args.steps + args.warmup, 1)) // w.n_workers))
    for _ in range(args.warmup):
        cpu_oracle_round(w, sample_d, stats_rule=args.stats)
    times = [cpu_oracle_round(w, sample_d, stats_rule=args.stats) for _ in range(args.steps)]
    t = sum(times) / len(times)
    val = w.n_workers * sample_d * esz / t / 1e9
    sample = f"{w.n_workers} workers x {sample_d} elements of workload {w.name} per step (full round)"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "d": w.d, "n_workers": w.n_workers, "mode": w.mode, "levels": w.num_levels,
                   "gamma": w.gamma, "storage": str(w.dtype).split(".")[-1], "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_exchange(args, w, tq, rank, local_rank, world, dev):
    """The round with the N workers split over the ranks (strong scaling: the job is the same N x d whatever
    the number of ranks).  Each rank takes the statistics of, and compresses, the workers it owns; the
    64-byte statistics records and the packed rows are what crosses ranks; every rank forms the full update."""
    import torch
    import torch.distributed as dist
    from paper_2402_01798_b200 import exchange, inputs
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29531")
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    esz = 2 if w.dtype == torch.bfloat16 else 4
    mode = tq.NONUNIFORM if w.mode == "nonuniform" else tq.UNIFORM
    N, d, bits = w.n_workers, w.d, w.bits
    first, count = exchange.worker_slice(rank, world, N)
    from dataclasses import replace
    mine = replace(w, n_workers=max(count, 1), base_seed=w.base_seed + first)          # worker i's seed is base + i on any rank
    g, stride = inputs.make_worker_gradients(mine, dev)
    g = g[:count]
    words = tq.tq_packed_words(d, bits)
    stats_local = torch.zeros(max(count, 1) * 64, dtype=torch.uint8, device=dev)
    ws = torch.empty(tq.tq_stats_workspace_bytes(max(count, 1)), dtype=torch.uint8, device=dev)
    hint = tq.new_gmin_hint(max(count, 1), dev)
    params_dev = torch.empty(N * 176, dtype=torch.uint8, device=dev)
    out = torch.empty(d, dtype=torch.float32, device=dev)
    peer = exchange.PeerRows(N, words, dev) if args.exchange == "peer" else None
    packed_local = peer.local if peer else torch.empty((count, words), dtype=torch.int32, device=dev)

    def one_round():
        if count:
            if args.stats == "hinted":
                tq.tq_stats_hinted(g, hint, d, stats_dev=stats_local, workspace=ws)
            else:
                tq.tq_stats(g, d, stats_dev=stats_local, workspace=ws)
        stats_all = exchange.gather_worker_rows(stats_local[: count * 64].view(count, 64), N)
        tq.tq_params_device(stats_all.view(-1), N, w.num_levels, mode, w.gamma, params_dev=params_dev)
        if args.exchange == "allgather":
            if count:
                tq.tq_compress_device_params(g, params_dev[first * 176:], w.num_levels, mode, seed=1234, first_worker=first,
                                             d=d, packed=packed_local)
            packed_all = exchange.gather_worker_rows(packed_local, N)
            tq.tq_decompress_aggregate_device_params(packed_all, d, params_dev, w.num_levels, out=out)
        else:
            ps = tq.params_to_host(params_dev)                       # one host sync: the row-pointer call takes host records
            if count:
                tq.tq_compress(g, ps[first:first + count], seed=1234, first_worker=first, d=d, packed=packed_local)
            peer.ready()                                              # every rank's rows are written ...
            tq.tq_decompress_aggregate_rows(peer.row_addresses(), d, ps, out=out)
            peer.done()                                               # ... and read, before the next round overwrites them

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_round()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    l0 = tq.tq_kernel_launches()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    a.record()
    for _ in range(args.steps):
        one_round()
    b.record()
    barrier()
    launches = tq.tq_kernel_launches() - l0
    clocks = sampler.stop()
    ms = max_over_ranks(a.elapsed_time(b), world, dev) / args.steps
    checksum = float(out.double().sum().item())
    if rank == 0:
        peak, peak_kind = hbm_peak()
        in_bytes = N * d * esz
        line = {
            "metric": METRIC, "value": in_bytes / (ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "d": d, "n_workers": N, "mode": w.mode, "levels": w.num_levels, "bits": bits,
                       "gamma": w.gamma, "storage": str(w.dtype).split(".")[-1], "stats": args.stats,
                       "multi_gpu": f"workers split over {world} rank(s), exchange = {args.exchange}: "
                                    + ("statistics records and packed rows all-gathered over NCCL" if args.exchange == "allgather"
                                       else "statistics records all-gathered, packed rows read in place from the peers' memory"),
                       "exchanged_bytes_per_rank_per_step": int((N - count) * (words * 4 + 64))},
            "roofline": None, "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "clocks": clocks,
            "update_checksum": checksum, "peak": {"hbm_gbs": peak, "source": peak_kind},
        }
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def measure_round(args, tq, w, g, stride, dev, local_rank, world, steps, warmup, headline):
    """Times `steps` rounds of workload `w` on the gradients `g` already resident in HBM (CUDA events on the
    launching stream, clocks sampled meanwhile).  headline=True adds the roofline object, the end-to-end
    measurement with host buffers and the CPU oracle beside it."""
    import torch
    esz = 2 if w.dtype == torch.bfloat16 else 4
    mode = tq.NONUNIFORM if w.mode == "nonuniform" else tq.UNIFORM
    N, d, bits = w.n_workers, w.d, w.bits

    rank = int(os.environ.get("RANK", "0"))
    stats_t = lambda xs: {"ms": statistics.mean(xs), "ms_median": statistics.median(xs), "ms_min": min(xs)}
    words = tq.tq_packed_words(d, bits)
    packed = torch.empty((N, words), dtype=torch.int32, device=dev)
    out = torch.empty(d, dtype=torch.float32, device=dev)
    stats_dev = torch.empty(N * 64, dtype=torch.uint8, device=dev)
    stats_pin = torch.empty(N * 64, dtype=torch.uint8).pin_memory()
    ws = torch.empty(tq.tq_stats_workspace_bytes(N), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    params_dev = torch.empty(N * 176, dtype=torch.uint8, device=dev)
    hint = tq.new_gmin_hint(N, dev)

    def run_stats(grad):
        if args.stats == "hinted":
            tq.tq_stats_hinted(grad, hint, d, stats_dev=stats_dev, workspace=ws)
        else:
            tq.tq_stats(grad, d, stats_dev=stats_dev, workspace=ws)

    def one_round(ev=None):
        """Returns what tq_decompress_aggregate needs to run again on this round's packed rows."""
        if ev: ev[0].record()
        run_stats(g)
        if ev: ev[1].record()
        if args.host_params:
            stats_pin.copy_(stats_dev, non_blocking=True)
            stream.synchronize()                               # the one host sync of this variant of the round
            ps = tq.tq_params_batch(stats_pin, N, w.num_levels, mode, w.gamma)
            if ev: ev[2].record()
            tq.tq_compress(g, ps, seed=1234, d=d, packed=packed)
            if ev: ev[3].record()
            tq.tq_decompress_aggregate(packed, d, ps, out=out)
            if ev: ev[4].record()
            return lambda: tq.tq_decompress_aggregate(packed, d, ps, out=out)
        # --device-params: parameters designed on the device, nothing returns to the host inside the round
        tq.tq_params_device(stats_dev, N, w.num_levels, mode, w.gamma, params_dev=params_dev)
        if ev: ev[2].record()
        tq.tq_compress_device_params(g, params_dev, w.num_levels, mode, seed=1234, d=d, packed=packed)
        if ev: ev[3].record()
        tq.tq_decompress_aggregate_device_params(packed, d, params_dev, w.num_levels, out=out)
        if ev: ev[4].record()
        return lambda: tq.tq_decompress_aggregate_device_params(packed, d, params_dev, w.num_levels, out=out)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        one_round()
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    l0 = tq.tq_kernel_launches()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_start.record()
    for k in range(steps):
        one_round(evs[k])
    t_end.record()
    barrier()
    launches = tq.tq_kernel_launches() - l0
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)

    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / steps
    in_bytes = N * d * esz
    value = whole_job_gbs(world, in_bytes, ms_per_step)

    # per-kernel durations inside the timed region (CUDA events on the launching stream)
    t_stats = stats_t([e[0].elapsed_time(e[1]) for e in evs])       # two launches
    t_params = stats_t([e[1].elapsed_time(e[2]) for e in evs])      # device kernel, or copy + sync + host design
    t_comp = stats_t([e[2].elapsed_time(e[3]) for e in evs])
    t_dec = stats_t([e[3].elapsed_time(e[4]) for e in evs])
    peak, peak_kind = hbm_peak()
    stats_passes = 1 if args.stats == "hinted" else 2     # hinted: the second kernel returns at once when the hint holds
    stats_key = "tq_stats (hinted, 1 pass)" if args.stats == "hinted" else "tq_stats (2 passes)"
    alg = {
        stats_key: (stats_passes * N * d * esz, t_stats, 2),
        "tq_compress": (N * d * esz + N * d * bits // 8, t_comp, 1),
        "tq_decompress_aggregate": (N * d * bits // 8 + 4 * d, t_dec, 1),
    }
    kernels = {"tq_params": dict(t_params, where="host (one sync)" if args.host_params else "device kernel")}
    # gbs / frac_of_hbm_peak from the mean over the timed steps; *_best from the fastest step
    kernels.update({k: dict(t, launches_per_step=n, algorithmic_bytes=b, gbs=b / (t["ms"] * 1e-3) / 1e9,
                            input_gbs=in_bytes / (t["ms"] * 1e-3) / 1e9,      # bytes of gradient input of the round per second of this kernel
                            frac_of_hbm_peak=b / (t["ms"] * 1e-3) / 1e9 / peak,
                            frac_of_nominal_8tbs=b / (t["ms"] * 1e-3) / 1e9 / 8000.0,
                            frac_of_hbm_peak_median=b / (t["ms_median"] * 1e-3) / 1e9 / peak,
                            frac_of_hbm_peak_best=b / (t["ms_min"] * 1e-3) / 1e9 / peak) for k, (b, t, n) in alg.items()})

    result = {"ms_per_step": ms_per_step, "value": value, "kernels": kernels, "clocks": clocks, "launches": int(launches),
              "whole_round_frac": (sum(b for b, _, _ in alg.values()) / (ms_per_step * 1e-3) / 1e9) / peak,
              "roofline": None, "cpu": None, "e2e": None}
    if args.stats == "hinted":
        # what the statistics cost when the hint does not hold (first round, or the mean moved to another binade):
        # the tail kernel then reads the data a second time
        miss = []
        for _ in range(3):
            hint.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); run_stats(g); b.record()
            torch.cuda.synchronize()
            miss.append(a.elapsed_time(b))
        kernels[stats_key]["hint_miss_ms"] = statistics.mean(miss)
        result["round_ms_hint_miss"] = ms_per_step + statistics.mean(miss) - t_stats["ms"]
        run_stats(g)                                     # leave a valid hint behind

    # decompress-aggregate again with the packed rows evicted from L2 first (in the round above they
    # were just written by tq_compress, so part of them is still cache-resident)
    decompress_again = one_round()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    cold = []
    for _ in range(5):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); decompress_again(); b.record()
        torch.cuda.synchronize()
        cold.append(a.elapsed_time(b))
    t_cold = statistics.mean(cold)
    kb = alg["tq_decompress_aggregate"][0]
    kernels["tq_decompress_aggregate"]["cold_l2_ms"] = t_cold
    kernels["tq_decompress_aggregate"]["cold_l2_ms_min"] = min(cold)
    kernels["tq_decompress_aggregate"]["cold_l2_gbs"] = kb / (t_cold * 1e-3) / 1e9
    kernels["tq_decompress_aggregate"]["cold_l2_frac_of_hbm_peak"] = kb / (t_cold * 1e-3) / 1e9 / peak
    del flush
    result["checksum"] = float(out.double().sum().item())
    if not headline:
        return result

    # layer groups (Section 5): the round with the d elements cut into S equal groups, every step of it ONE launch
    # over all (worker, group) pairs with the parameters designed on the device; and, for 16 groups, the same
    # work as one set of calls per group
    def equal_groups(S):
        step = (d // S) // 16 * 16
        return [(k * step, step if k < S - 1 else d - k * step) for k in range(S)]

    def grouped_round(table, seg, sdev, wsd, pdev, pk, hnt=None):
        if hnt is not None:
            tq.tq_stats_hinted_segments(g, seg, hnt, stats_dev=sdev, workspace=wsd)
        else:
            tq.tq_stats_segments(g, seg, stats_dev=sdev, workspace=wsd)
        tq.tq_params_device(sdev, N * len(table), w.num_levels, mode, w.gamma, params_dev=pdev)
        tq.tq_compress_segments(g, seg, pdev, w.num_levels, mode, seed=1234, packed=pk)
        tq.tq_decompress_aggregate_segments(pk, seg, pdev, w.num_levels, out=out)

    def per_group_round(table, sdev, wsd, pdev, pk):
        col = 0
        for off, ln in table:
            gv = g[:, off:off + ln]
            wds = tq.tq_packed_words(ln, bits)
            tq.tq_stats(gv, ln, stats_dev=sdev, workspace=wsd)
            tq.tq_params_device(sdev, N, w.num_levels, mode, w.gamma, params_dev=pdev)
            tq.tq_compress_device_params(gv, pdev, w.num_levels, mode, seed=1234, d=ln, packed=pk[:, col:col + wds])
            tq.tq_decompress_aggregate_device_params(pk[:, col:col + wds], ln, pdev, w.num_levels, out=out[off:off + ln])
            col += wds

    def timed(fn, reps=20):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    groups = {"round_ms": {}, "round_ms_one_pass_stats": {}, "params": "device",
              "stats": "round_ms: two passes (g_min = mean|g| of the group); round_ms_one_pass_stats: one hinted pass (power-of-two g_min)"}
    for S in (1, 4, 16, 64):
        table = equal_groups(S)
        seg = tq.segments_array(table)
        sdev = torch.empty(N * S * 64, dtype=torch.uint8, device=dev)
        wsd = torch.empty(tq.tq_stats_workspace_bytes(N * S), dtype=torch.uint8, device=dev)
        pdev = torch.empty(N * S * 176, dtype=torch.uint8, device=dev)
        pk = torch.empty((N, tq.tq_segments_packed_words(seg, bits)), dtype=torch.int32, device=dev)
        groups["round_ms"][str(S)] = timed(lambda: grouped_round(table, seg, sdev, wsd, pdev, pk))
        hnt = tq.new_gmin_hint(N * S, dev)
        groups["round_ms_one_pass_stats"][str(S)] = timed(lambda: grouped_round(table, seg, sdev, wsd, pdev, pk, hnt))
        if S == 16:
            groups["one_call_per_group_16_ms"] = timed(lambda: per_group_round(table, sdev, wsd, pdev, pk))
        del sdev, wsd, pdev, pk
    result["layer_groups"] = groups

    # the whole round (one-pass statistics, device-made parameters: no host synchronisation inside) as ONE CUDA graph,
    # against the same round launched kernel by kernel
    def device_round():
        run_stats(g)
        tq.tq_params_device(stats_dev, N, w.num_levels, mode, w.gamma, params_dev=params_dev)
        tq.tq_compress_device_params(g, params_dev, w.num_levels, mode, seed=1234, d=d, packed=packed)
        tq.tq_decompress_aggregate_device_params(packed, d, params_dev, w.num_levels, out=out)

    try:
        if world > 1:
            raise RuntimeError("measured on one GPU only (a process group's watchdog thread may touch the device during a capture)")
        launched = timed(device_round)
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            device_round()                                   # every kernel loaded and configured before the capture
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            device_round()
        result["cuda_graph"] = {"round_ms": timed(graph.replay), "launched_round_ms": launched,
                                "what": "statistics (one pass) -> device parameters -> compress -> aggregate, captured once, replayed"}
        del graph
    except Exception as e:                                   # capture is an extra: report why it did not work
        result["cuda_graph"] = {"error": repr(e)[:300]}

    dom = "tq_compress"      # the single kernel with the largest share of the round (see profiles/launch_list_*)
    result["roofline"] = {"kernel": dom, "bound": "hbm", "achieved": kernels[dom]["gbs"], "peak": peak, "peak_source": peak_kind,
                          "unit": "GB/s", "frac": kernels[dom]["gbs"] / peak, "algorithmic_bytes": alg[dom][0],
                          "traffic": NCU_DRAM_BYTES.get((w.name, dom))}

    # end to end through the public API with HOST buffers: H2D of every worker's gradient, the round,
    # D2H of the aggregated update, all inside the timed region
    e2e = None
    if not args.no_e2e:
        host_g = torch.empty((N, stride), dtype=w.dtype).pin_memory()
        host_g.copy_(g)
        host_out = torch.empty(d, dtype=torch.float32).pin_memory()
        # two device buffers and a copy stream: step k+1's host->device copy runs while step k computes and
        # returns its result (every step still copies its own inputs in and its own result out)
        bufs = [torch.empty_like(g), torch.empty_like(g)]
        copy_stream = torch.cuda.Stream(device=dev)
        e2e_steps = max(2, min(steps, 5))

        def e2e_compute(g2):
            run_stats(g2)
            if args.host_params:
                stats_pin.copy_(stats_dev, non_blocking=True)
                stream.synchronize()
                pp = tq.tq_params_batch(stats_pin, N, w.num_levels, mode, w.gamma)
                tq.tq_compress(g2, pp, seed=1234, d=d, packed=packed)
                tq.tq_decompress_aggregate(packed, d, pp, out=out)
            else:
                tq.tq_params_device(stats_dev, N, w.num_levels, mode, w.gamma, params_dev=params_dev)
                tq.tq_compress_device_params(g2, params_dev, w.num_levels, mode, seed=1234, d=d, packed=packed)
                tq.tq_decompress_aggregate_device_params(packed, d, params_dev, w.num_levels, out=out)
            host_out.copy_(out, non_blocking=True)

        def e2e_run(steps):
            arrived = [torch.cuda.Event() for _ in range(steps)]
            consumed = [torch.cuda.Event() for _ in range(steps)]

            def copy_in(k):
                with torch.cuda.stream(copy_stream):
                    if k >= 2:
                        copy_stream.wait_event(consumed[k - 2])          # the buffer's previous step is finished
                    bufs[k % 2].copy_(host_g, non_blocking=True)
                    arrived[k].record(copy_stream)

            copy_in(0)
            for k in range(steps):
                if k + 1 < steps:
                    copy_in(k + 1)
                stream.wait_event(arrived[k])
                e2e_compute(bufs[k % 2])
                consumed[k].record(stream)

        e2e_run(2); barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        copy_stream.wait_event(a)                                        # no copy starts before the timed region
        e2e_run(e2e_steps)
        b.record()
        barrier()
        ems = a.elapsed_time(b)
        ems = max_over_ranks(ems, world, dev) / e2e_steps
        e2e = {"value": whole_job_gbs(world, in_bytes, ems), "unit": "GB/s", "ms_per_step": ems, "steps": e2e_steps,
               "h2d_bytes_per_step": int(N * stride * esz), "d2h_bytes_per_step": int(4 * d + 64 * N)}
        del host_g, host_out, bufs
    result["e2e"] = e2e

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_d = min(d, max(1 << 16, (1 << 26) // N))
        dt = cpu_oracle_round(w, sample_d, stats_rule=args.stats)
        cpu = {"value": N * sample_d * esz / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dt,
               "host_cores_available": os.cpu_count(),
               "sample": f"{N} workers x {sample_d} elements of workload {w.name}, one full round"}
    result["cpu"] = cpu
    return result



def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="index into the five workloads (default: 25.6M x 16)")
    ap.add_argument("--variant", type=int, default=None,
                    help="with --config 3: index 0..11 into the bf16 sweep (gamma x mode x levels)")
    ap.add_argument("--d", type=int, default=None,
                    help="override the workload's elements per worker (a reduced copy of a large workload, for profiler captures)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--device-params", action="store_true",
                    help="design the parameters on the device (tq_params_device): no host round trip inside the round")
    ap.add_argument("--stats", default="hinted", choices=["two-pass", "hinted"],
                    help="two-pass: g_min = mean|g| (tq_stats); hinted: g_min = mean|g| rounded down to a power of two, "
                         "one pass over the data with the previous round's mean as the hint (tq_stats_hinted)")
    ap.add_argument("--exchange", default="replicas", choices=["replicas", "allgather", "peer"],
                    help="replicas (default): every rank runs its own copy of the workload, nothing crosses ranks; "
                         "allgather: the N workers are split over the ranks and the packed rows are all-gathered (NCCL) "
                         "before the aggregation; peer: same split, the aggregation kernel reads the peers' rows in place")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="leave out the per-kernel measurements of the other d >= 25.6 M workloads")
    args = ap.parse_args()
    args.host_params = not args.device_params
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2402_01798_b200 import inputs
    w = inputs.WORKLOADS[args.config]
    if args.config == 3 and args.variant is not None:
        w = inputs.CONFIG4_SWEEP[args.variant]
    if args.d is not None:
        from dataclasses import replace
        w = replace(w, d=args.d, name=f"{w.name}-d{args.d}")
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_2402_01798_b200 import binding as tq

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    tq.lib()
    if args.exchange != "replicas":
        run_exchange(args, w, tq, rank, local_rank, world, dev)
        return

    wr = replica_workload(w, rank)                      # rank r uses its own seeds: a replica, not a shard
    g, stride = inputs.make_worker_gradients(wr, dev)
    head = measure_round(args, tq, wr, g, stride, dev, local_rank, world, args.steps, args.warmup, headline=True)
    del g

    # the other workloads with d >= 25.6 M (one GPU only: they would hold every rank for a while longer)
    workloads = None
    if world == 1 and not args.no_workloads:
        workloads = {}
        c4 = {(c.gamma, c.mode, c.num_levels): c for c in inputs.CONFIG4_SWEEP}
        groups = [[(inputs.WORKLOADS[2], 100)],
                  [(c4[(3.0, m, L)], 40) for m in ("nonuniform", "uniform") for L in (16, 4)],    # one set of gradients, four quantizers
                  [(inputs.WORKLOADS[4], 12)]]
        groups = [[(w2, k) for w2, k in grp if w2.name != w.name] for grp in groups]
        for group in (grp for grp in groups if grp):
            torch.cuda.empty_cache()
            g2, stride2 = inputs.make_worker_gradients(group[0][0], dev)
            for w2, steps2 in group:                    # same gradient data, different quantizers
                r = measure_round(args, tq, w2, g2, stride2, dev, local_rank, 1, steps2, 3, headline=False)
                workloads[w2.name] = {"d": w2.d, "n_workers": w2.n_workers, "mode": w2.mode, "levels": w2.num_levels,
                                      "storage": str(w2.dtype).split(".")[-1], "steps": steps2, "ms_per_step": r["ms_per_step"],
                                      "value_gbs": r["value"], "hbm_frac_of_peak_whole_round": r["whole_round_frac"],
                                      "kernels": r["kernels"], "clocks": r["clocks"]}
            del g2

    if rank == 0:
        d, N, bits = w.d, w.n_workers, w.bits
        words = tq.tq_packed_words(d, bits)
        in_bytes = N * d * (2 if w.dtype == torch.bfloat16 else 4)
        line = {
            "metric": METRIC, "value": head["value"], "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "d": d, "n_workers": N, "mode": w.mode, "levels": w.num_levels, "bits": bits,
                       "gamma": w.gamma, "scale": w.scale, "storage": str(w.dtype).split(".")[-1],
                       "g_min": ("mean|g| per worker rounded down to a power of two; one statistics pass, hinted by the previous round's mean "
                                 "(same data every round, so the hint always holds; when it does not, the tail pass runs again: "
                                 "kernels[...].hint_miss_ms and round_ms_hint_miss show that cost)" if args.stats == "hinted"
                                 else "mean|g| per worker (two statistics passes)"), "alpha_rule": "fixed point",
                       "params": "host" if args.host_params else "device (no host round trip inside the round)",
                       "l2": f"inputs ({in_bytes / 1e6:.0f} MB) exceed L2; packed rows ({N * words * 4 / 1e6:.0f} MB) are "
                             "re-read right after being written, see kernels.tq_decompress_aggregate.cold_l2_*",
                       "multi_gpu": "independent replica per rank, no data-path collective"},
            "hbm_frac_of_peak_whole_round": head["whole_round_frac"],
            "round_ms_hint_miss": head.get("round_ms_hint_miss"),
            "roofline": head["roofline"], "kernels": head["kernels"], "cpu_baseline": head["cpu"], "e2e": head["e2e"],
            "gpu_launches": head["launches"], "clocks": head["clocks"],
            "update_checksum": head["checksum"],      # rank 0's aggregated update, for comparing variants
            "layer_groups": head.get("layer_groups"), "cuda_graph": head.get("cuda_graph"),
            "workloads": workloads,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
