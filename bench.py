#!/usr/bin/env python
"""Benchmark of the table-lookup low-bit matmul path on B200.

Headline (value): decode mpGEMV weight-stream GB/s on the 2-bit Llama-3-8B MLP shapes, M = 1
(gate and up 4096 -> 14336, down 14336 -> 4096, group 64).  One step = the mpGEMVs of one MLP block
over one token: gate and up, which read the same activations, go through one grouped call (one
table build for both), down through a second call.  The packed weights rotate through several resident copies
whose total size exceeds L2, so every call streams from HBM.  Steps are replayed from a CUDA
graph and timed with CUDA events on the launching stream.

The graph of 60 steps is replayed at least 20 times whatever --steps says; every replay is timed by its
own pair of events, ms_per_step and value come from the median replay, and the line keeps the best
replay and the replay count.

Also reported on the same JSON line: under roofline.prefill the prefill mpGEMM rate (M = 1024,
K = 4096, N in {4096, 14336}, 4-bit, group 128) with its tensor roofline; under roofline.ceilings the
lookup-rate and instruction-issue ceilings of the decode kernel; under config one-line digests of
configs 1, 3 and 5 measured in the same run; the end-to-end rate through the C ABI with host
buffers; the CPU oracle's rate on a bounded sample; clocks sampled during the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
    python bench.py --leg {case,config1,config3,config5,ablation,ternary,microbench} [leg options]   # see bench_legs.py

With N > 1 (launched under torchrun) every rank runs an independent replica of the same step
(the path does not shard); value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mpGEMV weight-stream GB/s (decode, 2-bit Llama-3-8B MLP, M=1)"
UNIT = "GB/s"
WORKLOAD = "config2: decode mpGEMV M=1, 2-bit, group 64, Llama-3-8B MLP gate/up 4096x14336 + down 14336x4096"
MLP = [("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096)]
BITS, GROUP = 2, 64
NSETS = 6
GRAPH_STEPS = 60
MIN_REPLAYS = 20
NOMINAL_HBM_GBS = 8000.0
NOMINAL_FP16_TFLOPS = 2250.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TFLOPS = 1590.0


def weight_bytes(K, N, bits, group):
    """Algorithmic weight-stream bytes of one matrix: planes + fp16 scales + b-bit zero-points."""
    return K * N * bits // 8 + (K // group) * N * 2 + (K // group) * N * bits // 8


def total_bytes(M, K, N, bits, group):
    return weight_bytes(K, N, bits, group) + M * K * 2 + M * N * 2


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm": float(d["hbm_gbs"]), "tf_burst": float(d["bf16_tflops"]),
                "tf_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "src": "measured"}
    return {"hbm": FALLBACK_HBM_GBS, "tf_burst": FALLBACK_TFLOPS, "tf_sustained": 1400.0, "src": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, nm in names.items():
                    if r & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._t is not None:
            self._t.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---- reference arm: the CPU oracle, as it stands --------------------------------------------

def oracle_step_sample(cases, n_cols):
    """One oracle 'step' over the first n_cols output columns of each MLP matrix."""
    from oracle import tman_oracle as orc
    outs = []
    for c in cases:
        nc = min(n_cols, c.N)
        outs.append(orc.mpgemm(c.x, np.ascontiguousarray(c.codes[:, :nc]),
                               np.ascontiguousarray(c.scales[:, :nc]),
                               np.ascontiguousarray(c.zeros[:, :nc]), c.group))
    return outs


def time_oracle(cases, n_cols, steps, warmup):
    for _ in range(warmup):
        oracle_step_sample(cases, n_cols)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step_sample(cases, n_cols)
    dt = time.perf_counter() - t0
    wb = sum(weight_bytes(c.K, min(n_cols, c.N), c.bits, c.group) for c in cases)
    return dt / steps, wb


def host_cases(seed_offset=0):
    from paper_2511_11248_b200 import synth
    lo, hi = synth.scale_range(BITS)
    cases = [synth.make_case(f"c2_{nm}", 1, K, N, BITS, GROUP, synth.SEED_BASE + 200 + i + 10 * seed_offset, lo, hi)
             for i, (nm, K, N) in enumerate(MLP)]
    cases[1].x[:] = cases[0].x      # gate and up read the same activations
    return cases


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import tman_oracle as orc
    cases = host_cases()
    # size the per-step sample so that the whole run stays within a couple of minutes
    t_probe, _ = time_oracle(cases, 512, 1, 1)
    budget = 120.0 / max(1, args.steps + args.warmup)
    n_cols = int(max(8, min(14336, 512 * budget / max(t_probe, 1e-6)) // 8 * 8))
    n_cols = min(n_cols, 14336)
    sec, wb = time_oracle(cases, n_cols, args.steps, args.warmup)
    val = wb / sec / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": f"first {n_cols} output columns of each matrix per step"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                         "sample": f"first {n_cols} output columns of each of the 3 matrices, per step"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---- our arm ---------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2511_11248_b200 import binding as B, helpers as H, replicas, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    B.lib()   # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    peaks = measured_peaks()
    stream = torch.cuda.current_stream()

    # ---- decode workload: NSETS resident weight sets (> L2 in total) ---------------------------
    sets = []
    host0 = None
    for si in range(NSETS):
        cases = host_cases(seed_offset=si)
        if si == 0:
            host0 = cases
        entry = []
        for c in cases:
            dev = H.device_case(c)
            packed = H.pack_case(c, dev)
            y = torch.empty((1, c.N), dtype=torch.float16, device="cuda")
            ws = H.alloc_workspace(B.OP_GEMV, 1, c.K, 2 * c.N, BITS, GROUP)
            entry.append((c.K, c.N, packed, dev["x"], y, ws))
            del dev["codes"]
        sets.append(entry)
    torch.cuda.synchronize()
    resident_mb = sum(e[2].numel() for s in sets for e in s) / 1e6

    def step(si):
        gate, up, down = sets[si % NSETS]
        B.tman_mpgemv_grouped([gate[2], up[2]], gate[3], [gate[4], up[4]], 1, gate[0], [gate[1], up[1]],
                              BITS, GROUP, gate[5])
        B.tman_mpgemv(down[2], down[3], down[4], 1, down[0], down[1], BITS, GROUP, down[5])

    wbytes_step = sum(weight_bytes(K, N, BITS, GROUP) for _, K, N in MLP)
    abytes_step = sum(total_bytes(1, K, N, BITS, GROUP) for _, K, N in MLP)
    launches_per_step = 2          # grouped gate+up, down

    # graph of GRAPH_STEPS consecutive steps (launch-bound otherwise: a step is ~10 us of GPU time)
    for i in range(3):
        step(i)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(GRAPH_STEPS):
            step(i)
    n_replay = max(MIN_REPLAYS, -(-args.steps // GRAPH_STEPS))
    steps = n_replay * GRAPH_STEPS
    n_warm = max(1, -(-max(args.warmup, 3) // GRAPH_STEPS))
    for _ in range(n_warm):
        graph.replay()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_replay + 1)]
    barrier()
    with ClockSampler(physical_gpu_index(local_rank)) as clk:
        ev0.record()
        marks[0].record()
        for r in range(n_replay):
            graph.replay()
            marks[r + 1].record()
        ev1.record()
        torch.cuda.synchronize()
    barrier()
    # every replay's own duration: median for the headline, best and the whole region's mean beside it
    replay_ms = np.array([marks[r].elapsed_time(marks[r + 1]) for r in range(n_replay)])
    ms_median = replicas.max_over_ranks(float(np.median(replay_ms)), "cuda")
    ms_best = replicas.max_over_ranks(float(np.min(replay_ms)), "cuda")
    ms_total = replicas.max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    sec_step = ms_median / 1e3 / GRAPH_STEPS
    value = replicas.whole_job_rate(wbytes_step, sec_step, world) / 1e9
    st = [B.tman_read_status(e[5]) for s in sets for e in s]
    assert all(v == 0 for v in st), f"device status {st}"

    # ---- end to end through the C ABI with host buffers ---------------------------------------
    # one pinned input buffer (the activations of gate/up, then those of down) and one pinned output
    # buffer (gate, up, down results) per step: one copy in, one copy out
    kx, kd = host0[0].K, host0[2].K
    ng, nd = host0[0].N, host0[2].N
    x_host = torch.cat([torch.from_numpy(host0[0].x.view(np.int16)).view(torch.float16).reshape(-1),
                        torch.from_numpy(host0[2].x.view(np.int16)).view(torch.float16).reshape(-1)]).pin_memory()
    y_host = torch.empty(2 * ng + nd, dtype=torch.float16).pin_memory()
    x_dev = torch.empty(kx + kd, dtype=torch.float16, device="cuda")
    y_dev = torch.empty(2 * ng + nd, dtype=torch.float16, device="cuda")
    xg, xd = x_dev[:kx].view(1, kx), x_dev[kx:].view(1, kd)
    yg, yu, yd = y_dev[:ng].view(1, ng), y_dev[ng:2 * ng].view(1, ng), y_dev[2 * ng:].view(1, nd)
    h2d = x_host.numel() * 2
    d2h = y_host.numel() * 2

    def e2e_step(si, sync):
        gate, up, down = sets[si % NSETS]
        x_dev.copy_(x_host, non_blocking=True)
        B.tman_mpgemv_grouped([gate[2], up[2]], xg, [yg, yu], 1, kx, [ng, ng], BITS, GROUP, gate[5])
        B.tman_mpgemv(down[2], xd, yd, 1, kd, nd, BITS, GROUP, down[5])
        y_host.copy_(y_dev, non_blocking=True)
        if sync:
            torch.cuda.synchronize()

    # (a) the host waits for every step's result before it issues the next step
    e2e_steps = min(2000, max(50, steps // 10))
    for i in range(20):
        e2e_step(i, True)
    barrier()
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i, True)
    ev1.record()
    torch.cuda.synchronize()
    e2e_sync_ms = replicas.max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    e2e_sync_val = replicas.whole_job_rate(wbytes_step, e2e_sync_ms / 1e3 / e2e_steps, world) / 1e9
    # (b) the same calls and copies, every step, replayed from a CUDA graph (no host wait between
    # steps): host -> device copy of the activations, the two calls, device -> host copy of the results
    e2e_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(e2e_graph):
        for i in range(GRAPH_STEPS):
            e2e_step(i, False)
    e2e_replays = max(10, e2e_steps // GRAPH_STEPS)
    e2e_graph.replay()
    barrier()
    ev0.record()
    for _ in range(e2e_replays):
        e2e_graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    e2e_serial_ms = replicas.max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    e2e_serial_val = replicas.whole_job_rate(wbytes_step, e2e_serial_ms / 1e3 / (e2e_replays * GRAPH_STEPS), world) / 1e9

    # (c) as (b), with the copies on their own streams and two sets of device buffers: step i's
    # activations come in while step i-1 computes, its results go out while step i+1 computes
    # (independent requests served back to back).  Every step still copies its own input and output.
    xs_dev = [torch.empty(kx + kd, dtype=torch.float16, device="cuda") for _ in range(2)]
    ys_dev = [torch.empty(2 * ng + nd, dtype=torch.float16, device="cuda") for _ in range(2)]
    ys_host = [torch.empty(2 * ng + nd, dtype=torch.float16).pin_memory() for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    pipe_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(pipe_graph):
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        s_in.wait_event(fork)
        s_out.wait_event(fork)
        computed = [None, None]     # event: the step that last used buffer b has computed
        drained = [None, None]      # event: the results of the step that last used buffer b are on the host
        for i in range(GRAPH_STEPS):
            b = i % 2
            gate, up, down = sets[i % NSETS]
            if computed[b] is not None:
                s_in.wait_event(computed[b])            # x buffer b is free again
            with torch.cuda.stream(s_in):
                xs_dev[b].copy_(x_host, non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(s_in)
            main.wait_event(arrived)
            if drained[b] is not None:
                main.wait_event(drained[b])             # y buffer b is free again
            xg_b, xd_b = xs_dev[b][:kx].view(1, kx), xs_dev[b][kx:].view(1, kd)
            yb = ys_dev[b]
            B.tman_mpgemv_grouped([gate[2], up[2]], xg_b, [yb[:ng].view(1, ng), yb[ng:2 * ng].view(1, ng)], 1, kx,
                                  [ng, ng], BITS, GROUP, gate[5])
            B.tman_mpgemv(down[2], xd_b, yb[2 * ng:].view(1, nd), 1, kd, nd, BITS, GROUP, down[5])
            computed[b] = torch.cuda.Event()
            computed[b].record(main)
            s_out.wait_event(computed[b])
            with torch.cuda.stream(s_out):
                ys_host[b].copy_(yb, non_blocking=True)
                drained[b] = torch.cuda.Event()
                drained[b].record(s_out)
        for b in range(2):                              # join the side streams
            main.wait_event(drained[b])
        join_in = torch.cuda.Event()
        join_in.record(s_in)
        main.wait_event(join_in)
    pipe_graph.replay()
    torch.cuda.synchronize()
    barrier()
    ev0.record()
    for _ in range(e2e_replays):
        pipe_graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    e2e_ms = replicas.max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    e2e_val = replicas.whole_job_rate(wbytes_step, e2e_ms / 1e3 / (e2e_replays * GRAPH_STEPS), world) / 1e9
    # the last step's results, as they arrived on the host, against the device results
    assert torch.equal(ys_host[(GRAPH_STEPS - 1) % 2], ys_dev[(GRAPH_STEPS - 1) % 2].cpu()), "host results differ"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": n_warm * GRAPH_STEPS, "ms_per_step": sec_step * 1e3,
        "ms_per_step_best": ms_best / GRAPH_STEPS, "ms_per_step_mean": ms_total / steps,
        "replays": n_replay, "steps_per_replay": GRAPH_STEPS, "timing": "median over replays, each timed by its own events",
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "replicas": world,
                   "l2": f"inputs larger than L2: {NSETS} rotating weight sets, {resident_mb:.0f} MB resident",
                   "launch": f"CUDA graph of {GRAPH_STEPS} steps; per step one grouped call (gate+up) and one call (down)",
                   "total_bytes_gbs": world * abytes_step / sec_step / 1e9,
                   "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS},
        "clocks": clk.summary(),
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_replays * GRAPH_STEPS,
                "note": "weights resident; every step copies its activations in from pinned host memory and its "
                        "results back, all enqueued through the C ABI and replayed from a CUDA graph; copies run on "
                        "their own streams with two sets of device buffers, so a step's copies overlap its "
                        "neighbours' kernels",
                "one_stream": {"value": e2e_serial_val, "unit": UNIT, "steps": e2e_replays * GRAPH_STEPS},
                "host_waits_each_step": {"value": e2e_sync_val, "unit": UNIT, "steps": e2e_steps}},
        "gpu_launches": steps * launches_per_step,
    }
    avg_launch_s = sec_step / launches_per_step
    ach = (abytes_step / launches_per_step) / avg_launch_s / 1e9
    line["roofline"] = {"bound": "hbm", "kernel": "mpgemv_kernel (2-bit, M=1: BITS=2, MT=1, S=4, PRE, HALF, ROLL; grouped and single launches averaged)", "achieved": ach, "peak": peaks["hbm"],
                        "unit": "GB/s", "frac": ach / peaks["hbm"], "traffic": TRAFFIC_BYTES_PER_LAUNCH,
                        "peak_source": f"of {peaks['src']}", "algorithmic_bytes_per_launch": abytes_step / launches_per_step}

    if rank == 0:
        line["roofline"]["ceilings"] = decode_ceilings(torch, B, clk.summary(), abytes_step / launches_per_step, ach)
    if rank == 0 and not args.skip_gemm:
        line["roofline"]["prefill"] = bench_gemm(torch, B, H, synth, peaks)
    if rank == 0 and world == 1 and not args.skip_sweeps:
        import bench_legs
        line["config"].update(bench_legs.summaries(torch, B, H))
    if rank == 0 and world == 1 and not args.skip_cpu:
        line["cpu_baseline"] = cpu_baseline(host0, sets[0])
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/.  mpGEMV: one gate/up-sized launch moved 17.04 MB for 16.78 MB of algorithmic bytes
# (+1.5 %; counters re-taken on the present kernel build); traffic grows with the bytes streamed, so the step's mean launch (25.17 MB) is scaled
# by the same ratio.  mpGEMM: the M=1024, K=4096, N=14336 launch (the larger of the two timed shapes)
# read 39.2 MB and wrote 0.4 - 2.5 MB (the output mostly stays in L2).
TRAFFIC_BYTES_PER_LAUNCH = 25171968.0 * (17.04 / 16.78)
GEMM_TRAFFIC_BYTES_PER_LAUNCH = 40.6e6


# Warp instructions the decode kernel executes for one gate/up-sized launch (16.78 MB of algorithmic
# bytes), from the ncu capture summarised under profiles/ (smsp__inst_executed.sum).
DECODE_WARP_INSTRUCTIONS_PER_BYTE = 3.56e6 / 16.78e6
SCHEDULERS_PER_SM = 4


def decode_ceilings(torch, B, clocks, bytes_per_launch, achieved_gbs):
    """Two ceilings of the decode kernel other than HBM, in the units of roofline.achieved.
    lookup: the rate at which one SM performs the kernel's lookup (8-bit index, 256-entry fp32 table in
    shared memory, one add), measured now by the lookup microbenchmark; a lookup consumes one byte of a
    bit plane, and planes are 8/9 (2-bit, group 64) of the bytes streamed.
    issue: the kernel's warp instructions per byte (from its ncu capture) at one instruction per clock
    per scheduler."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    res = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        res.zero_()
        B.tman_debug_microbench(0, 512, res)
    torch.cuda.synchronize()
    clk = res[: sms * 8].view(torch.int64).cpu().numpy().astype(np.float64)
    lookups_per_clk = float((1 << 20) / np.median(clk))
    plane_share = (BITS / 8) / (BITS / 8 + (2 + BITS / 8) / GROUP)
    lookup_gbs = lookups_per_clk * sms * mhz * 1e6 / plane_share / 1e9
    issue_gbs = SCHEDULERS_PER_SM * sms * mhz * 1e6 / DECODE_WARP_INSTRUCTIONS_PER_BYTE / 1e9
    return {"unit": "GB/s", "sm_mhz": mhz,
            "lookup": {"lookups_per_clk_per_sm": round(lookups_per_clk, 2), "GBs": round(lookup_gbs, 1),
                       "achieved_frac": round(achieved_gbs / lookup_gbs, 3)},
            "issue": {"warp_instructions_per_byte": round(DECODE_WARP_INSTRUCTIONS_PER_BYTE, 4),
                      "GBs": round(issue_gbs, 1), "achieved_frac": round(achieved_gbs / issue_gbs, 3)}}


def bench_gemm(torch, B, H, synth, peaks):
    """Prefill mpGEMM, config 4: M=1024, K=4096, N in {4096, 14336}, 4-bit, group 128."""
    out = {"cases": []}
    tot_flops, tot_sec = 0.0, 0.0
    for spec in synth.config4_specs():
        c = synth.case_from_spec(spec)
        dev = H.device_case(c)
        packed = H.pack_case(c, dev)
        ncopies = 4
        xs = [dev["x"].clone() for _ in range(ncopies)]
        ys = [torch.empty((c.M, c.N), dtype=torch.float16, device="cuda") for _ in range(ncopies)]
        pks = [packed.clone() for _ in range(ncopies)]
        ws = H.alloc_workspace(B.OP_GEMM, c.M, c.K, c.N, c.bits, c.group)
        for i in range(4):
            B.tman_mpgemm(pks[i % ncopies], xs[i % ncopies], ys[i % ncopies], c.M, c.K, c.N, c.bits, c.group, ws)
        torch.cuda.synchronize()
        iters = 40
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            B.tman_mpgemm(pks[i % ncopies], xs[i % ncopies], ys[i % ncopies], c.M, c.K, c.N, c.bits, c.group, ws)
        e1.record()
        torch.cuda.synchronize()
        assert B.tman_read_status(ws) == 0
        sec = e0.elapsed_time(e1) / 1e3 / iters
        flops = 2.0 * c.M * c.K * c.N
        out["cases"].append({"M": c.M, "K": c.K, "N": c.N, "bits": c.bits, "group": c.group,
                             "us": sec * 1e6, "tflops": flops / sec / 1e12})
        tot_flops += flops
        tot_sec += sec
    tf = tot_flops / tot_sec / 1e12
    out.update({"bound": "tensor", "kernel": "mpgemm_kernel<4,2,true> (4-bit, CTA pairs, two row blocks per CTA)",
                "workload": "config4: prefill mpGEMM M=1024, K=4096, N in {4096, 14336}, 4-bit, group 128 "
                            "(sum of flops / sum of time; 4 rotating copies of inputs and outputs, 40 calls each)",
                "achieved": tf, "peak": peaks["tf_burst"], "unit": "TFLOP/s", "frac": tf / peaks["tf_burst"],
                "frac_of_nominal_fp16": tf / NOMINAL_FP16_TFLOPS, "traffic": GEMM_TRAFFIC_BYTES_PER_LAUNCH,
                "traffic_of": "the M=1024, K=4096, N=14336 launch",
                "peak_source": f"of {peaks['src']} (bf16 burst; fp16 has the same nominal rate)"})
    return out


def cpu_baseline(host0, set0):
    """The oracle, as it stands, on the host cores: a bounded sample of the same step; also the
    parity of the timed configuration against it."""
    from oracle import tman_oracle as orc
    import torch
    n_cols = 14336
    t_probe, _ = time_oracle(host0, 1024, 1, 0)
    reps = int(max(1, min(20, 10.0 / max(t_probe * 14, 1e-3))))
    sec, wb = time_oracle(host0, n_cols, reps, 1)
    outs = oracle_step_sample(host0, n_cols)
    errs = []
    for ref, (K, N, packed, x, y, ws) in zip(outs, set0):
        got = y.detach().cpu().to(torch.float64).numpy()
        errs.append(float(np.max(np.abs(got - ref)) / np.max(np.abs(ref))))
    return {"value": wb / sec / 1e9, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{reps} full steps (all columns of the 3 matrices), {sec * 1e3:.1f} ms per step",
            "parity_max_rel_err": max(errs)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12000)
    ap.add_argument("--warmup", type=int, default=600)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--skip-gemm", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-sweeps", action="store_true", help="leave the config 1/3/5 digests out of the line")
    ap.add_argument("--leg", default="headline", choices=["headline", "case", "config1", "config3", "config5", "ablation", "ternary", "stamps", "microbench"],
                    help="headline: the bench line (default); the others print their own JSON lines")
    args, rest = ap.parse_known_args()
    if args.leg != "headline":
        import bench_legs
        getattr(bench_legs, args.leg)(args, rest)
        return
    if rest:
        ap.error(f"unknown arguments {rest}")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
