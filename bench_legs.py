"""Measurement legs that `bench.py --leg NAME` runs besides the headline step: the design
microbenchmarks, a single shape (also the command line to profile), the decode batch sweep and the
prefill shape sweep.  Everything goes through the C ABI; one JSON line per result on stdout.
"""
from __future__ import annotations

import json

import numpy as np

L2_BYTES = 126e6
LLAMA3_8B_LAYER = [("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
                   ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096)]


def weight_bytes(K, N, bits, group):
    return K * N * bits // 8 + (K // group) * N * 2 + (K // group) * N * bits // 8


def event_us(torch, fn, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(reps):
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(ts)), float(np.min(ts))


# ---- design microbenchmarks ---------------------------------------------------------------------

LOOKUP_KINDS = [
    (0, "256-entry fp32 table, PRMT + LDS.32 + FADD", 8),
    (1, "256-entry fp16 table, PRMT + LDS.U16 + mixed add", 8),
    (2, "16-entry fp32 table (paper's shape), shift/mask + LDS.32 + FADD", 4),
    (3, "16-entry table in registers, SHFL + FADD", 4),
    (4, "256-entry table of 2 fp16 rows, PRMT + LDS.32 + HADD2", 8),
    (5, "256-entry table of 4 fp16 rows, PRMT + LDS.64 + 2 HADD2", 8),
    (6, "256-entry table of 8 fp16 rows, PRMT + LDS.128 + 4 HADD2", 8),
]


def microbench(args):
    """Lookup rates per SM, load-path bandwidths, cluster exchange and L2 latency (one B200)."""
    import torch
    from paper_2511_11248_b200 import binding as B

    res = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    index_bytes = 1 << 20          # index bytes a CTA looks up per launch (64 passes over a 16 KB pool)
    for kind, name, wpl in LOOKUP_KINDS:
        for threads in (256, 512):
            for _ in range(2):
                res.zero_()
                B.tman_debug_microbench(kind, threads, res)
            torch.cuda.synchronize()
            clk = res[: sms * 8].view(torch.int64).cpu().numpy().astype(np.float64)
            lookups = index_bytes * (8 // wpl)
            print(json.dumps({"leg": "microbench", "what": "lookup", "kind": kind, "table": name, "threads_per_cta": threads,
                              "lookups_per_clk_per_sm": round(float(lookups / np.median(clk)), 2),
                              "weight_bits_per_clk_per_sm": round(float(index_bytes * 8 / np.median(clk)), 1),
                              "clocks_median": float(np.median(clk)), "clocks_max": float(clk.max())}), flush=True)
    # load paths: a buffer larger than L2, read once per launch
    nbytes = 1 << 30
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    buf.zero_()
    for kind, arg, name in [(10, 0, "coalesced 16-byte loads (ld.global.cs.v4)"),
                            (11, 4096, "cp.async.bulk, 4 KB chunks"), (11, 16384, "cp.async.bulk, 16 KB chunks"),
                            (11, 32768, "cp.async.bulk, 32 KB chunks")]:
        res.zero_()
        B.tman_debug_microbench(kind, arg, res, buf)
        torch.cuda.synchronize()
        med, mn = event_us(torch, lambda: B.tman_debug_microbench(kind, arg, res, buf), 7)
        st = int(res[:4].view(torch.int32).item()) if kind == 11 else 0
        print(json.dumps({"leg": "microbench", "what": "load path", "path": name, "GBs_median": round(nbytes / med / 1e3, 1),
                          "GBs_best": round(nbytes / mn / 1e3, 1), "status": st}), flush=True)
    del buf
    # cluster exchange
    for cs in (1, 2, 4, 8):
        res.zero_()
        B.tman_debug_microbench(20, cs, res)
        torch.cuda.synchronize()
        v = res[: cs * 8 * 16].view(torch.int64).cpu().numpy().reshape(-1, 2)
        print(json.dumps({"leg": "microbench", "what": "cluster exchange", "cluster": cs,
                          "barrier_clocks": float(np.median(v[:, 0])),
                          "store_barrier_read_barrier_clocks": float(np.median(v[:, 1]))}), flush=True)
    # dependent loads that hit L2
    chain = torch.empty(8 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        res.zero_()
        B.tman_debug_microbench(21, 8 << 20, res, chain)
    torch.cuda.synchronize()
    print(json.dumps({"leg": "microbench", "what": "L2 load latency (dependent loads, 8 MB chain)",
                      "clocks": int(res[:8].view(torch.int64).item())}), flush=True)
    # how many clusters the device holds
    for threads, smem in ((512, 100 * 1024), (512, 200 * 1024), (544, 200 * 1024), (256, 100 * 1024)):
        caps = {str(cs): B.tman_debug_cluster_capacity(threads, smem, cs) for cs in (1, 2, 4, 8, 16)}
        print(json.dumps({"leg": "microbench", "what": "resident clusters", "threads": threads, "smem_bytes": smem,
                          "sms": sms, "clusters_by_size": caps}), flush=True)
