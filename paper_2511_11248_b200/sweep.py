"""Time the batch sweep of the decode path and the shape sweep of the prefill path through the C ABI.

    python -m paper_2511_11248_b200.sweep --config 3     # one decoder layer's projections, M in {1,2,4,8}
    python -m paper_2511_11248_b200.sweep --config 5     # prefill shapes, M in {128,512,2048,8192}

Config 3: the seven projections of a Llama-3-8B-shaped decoder layer run as four calls (q, k, v in one
grouped call, o, gate and up in one grouped call, down), replayed from a CUDA graph over rotating
weight sets larger than L2; reports weight-stream GB/s of the layer (sum of bytes / sum of time).
Config 5: one call per shape, rotating packed copies larger than L2; reports TFLOP/s.
Synthetic seeded inputs (value distributions of the parity tests); one JSON line per case.
With --dense every case also times the same product with fp16 weights through torch.matmul (the
library GEMM/GEMV: a yardstick for "what the low-bit weights buy or cost", not part of the path).
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B, helpers as H, synth

LLAMA3_8B_LAYER = [("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
                   ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096)]
L2_BYTES = 126e6


def weight_bytes(K, N, bits, group):
    return K * N * bits // 8 + (K // group) * N * 2 + (K // group) * N * bits // 8


def event_us(fn, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(reps):
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(ts))


def dense_layer_us(M, reps):
    """The layer's seven products with fp16 weights (torch.matmul), rotating weight sets > L2."""
    layer_bytes = sum(K * N * 2 for _, K, N in LLAMA3_8B_LAYER)
    nsets = max(2, int(2.2 * L2_BYTES // layer_bytes) + 1)
    sets = [[(torch.randn((M, K), dtype=torch.float16, device="cuda"),
              torch.randn((K, N), dtype=torch.float16, device="cuda") * 0.02) for _, K, N in LLAMA3_8B_LAYER]
            for _ in range(nsets)]

    def layer(e):
        for x, w in e:
            torch.matmul(x, w)

    for e in sets:
        layer(e)
    torch.cuda.synchronize()
    nrep = 4 * nsets
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(nrep):
            layer(sets[i % nsets])
    g.replay()
    torch.cuda.synchronize()
    return event_us(g.replay, reps) / nrep


def dense_case_us(M, K, N, reps):
    x = torch.randn((M, K), dtype=torch.float16, device="cuda")
    ncopy = max(2, int(2.2 * L2_BYTES // (K * N * 2)) + 1)
    ws = [torch.randn((K, N), dtype=torch.float16, device="cuda") * 0.02 for _ in range(ncopy)]
    y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    for w in ws[:2]:
        torch.matmul(x, w, out=y)
    torch.cuda.synchronize()

    def run():
        for w in ws:
            torch.matmul(x, w, out=y)

    return event_us(run, reps) / ncopy


def decode_layer(bits, group, M, reps):
    layer_bytes = sum(weight_bytes(K, N, bits, group) for _, K, N in LLAMA3_8B_LAYER)
    nsets = max(2, int(2.2 * L2_BYTES // layer_bytes) + 1)
    sets = []
    for s in range(nsets):
        entry = {}
        for i, (name, K, N) in enumerate(LLAMA3_8B_LAYER):
            c = synth.small_case(M, K, N, bits, group, seed=100 * s + i)
            dev = H.device_case(c)
            entry[name] = (H.pack_case(c, dev), dev["x"], torch.empty((M, N), dtype=torch.float16, device="cuda"))
        sets.append(entry)
    ws = {k: H.alloc_workspace(B.OP_GEMV, M, K, N, bits, group)
          for k, K, N in (("qkv", 4096, 6144), ("o", 4096, 4096), ("gu", 4096, 28672), ("down", 14336, 4096))}

    def layer(e):
        x = e["q"][1]
        B.tman_mpgemv_grouped([e["q"][0], e["k"][0], e["v"][0]], x, [e["q"][2], e["k"][2], e["v"][2]], M, 4096,
                              [4096, 1024, 1024], bits, group, ws["qkv"])
        B.tman_mpgemv(e["o"][0], e["o"][1], e["o"][2], M, 4096, 4096, bits, group, ws["o"])
        xg = e["gate"][1]
        B.tman_mpgemv_grouped([e["gate"][0], e["up"][0]], xg, [e["gate"][2], e["up"][2]], M, 4096, [14336, 14336],
                              bits, group, ws["gu"])
        B.tman_mpgemv(e["down"][0], e["down"][1], e["down"][2], M, 14336, 4096, bits, group, ws["down"])

    for e in sets:
        layer(e)
    torch.cuda.synchronize()
    nrep = 4 * nsets
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(nrep):
            layer(sets[i % nsets])
    g.replay()
    torch.cuda.synchronize()
    us = event_us(g.replay, reps) / nrep
    assert all(B.tman_read_status(w) == 0 for w in ws.values())
    return {"config": 3, "M": M, "bits": bits, "group": group, "layer_us": round(us, 2),
            "weight_stream_GBs": round(layer_bytes / us / 1e3, 1), "weight_sets": nsets, "launches_per_layer": 4}


def prefill_case(M, K, N, bits, group, reps):
    c = synth.small_case(M, K, N, bits, group, seed=5, outliers=True)
    dev = H.device_case(c)
    p0 = H.pack_case(c, dev)
    ncopy = max(2, int(2.2 * L2_BYTES // p0.numel()) + 1)
    pk = [p0] + [p0.clone() for _ in range(ncopy - 1)]
    ws = H.alloc_workspace(B.OP_GEMM, M, K, N, bits, group)
    ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
    x = dev["x"]
    for i in range(3):
        B.tman_mpgemm(pk[i % ncopy], x, ys[i % 2], M, K, N, bits, group, ws)
    torch.cuda.synchronize()

    def run():
        for i in range(ncopy):
            B.tman_mpgemm(pk[i], x, ys[i % 2], M, K, N, bits, group, ws)

    us = event_us(run, reps) / ncopy
    assert B.tman_read_status(ws) == 0
    plan = B.tman_debug_gemm_plan(M, K, N, bits, group)
    return {"config": 5, "M": M, "K": K, "N": N, "bits": bits, "group": group, "us": round(us, 1),
            "TFLOPs": round(2.0 * M * K * N / us / 1e6, 1), "split_tiles": 1 - plan["whole_tiles"],
            "column_tiles": plan["tiles_n"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, choices=[3, 5], required=True)
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--dense", action="store_true", help="also time the fp16-weight product (torch.matmul)")
    a = ap.parse_args()
    if a.config == 3:
        dense = {M: dense_layer_us(M, a.reps) for M in (1, 2, 4, 8)} if a.dense else {}
        torch.cuda.empty_cache()
        for bits in (2, 3, 4):
            for M in (1, 2, 4, 8):
                r = decode_layer(bits, 128, M, a.reps)
                if a.dense:
                    r["dense_fp16_layer_us"] = round(dense[M], 2)
                    r["speedup_vs_dense_fp16"] = round(dense[M] / r["layer_us"], 2)
                print(json.dumps(r), flush=True)
                torch.cuda.empty_cache()
    else:
        dense = {}
        for bits in (2, 4):
            for group in (64, 128):
                for M in (128, 512, 2048, 8192):
                    for _, K, N in synth.QWEN25_7B_PROJ:
                        r = prefill_case(M, K, N, bits, group, a.reps)
                        if a.dense:
                            if (M, K, N) not in dense:
                                dense[(M, K, N)] = dense_case_us(M, K, N, a.reps)
                                torch.cuda.empty_cache()
                            r["dense_fp16_us"] = round(dense[(M, K, N)], 1)
                            r["time_vs_dense_fp16"] = round(r["us"] / dense[(M, K, N)], 2)
                        print(json.dumps(r), flush=True)
                        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
