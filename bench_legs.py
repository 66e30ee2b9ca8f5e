"""Measurement legs that `bench.py --leg NAME` runs besides the headline step:

    python bench.py --leg case --op gemv --M 1 --K 4096 --N 14336 --bits 2 --group 64   # one shape (also the command to profile)
    python bench.py --leg config1                  # decode, M=1, 4096x4096, 4-bit, group 64
    python bench.py --leg config3 [--dense]        # one decoder layer's projections, bits {2,3,4} x M {1,2,4,8}
    python bench.py --leg config5 [--dense] [--all-groups]   # prefill shapes, M in {128,512,2048,8192}
    python bench.py --leg ternary                  # integer decode: ternary weights, 16-bit integer activations, BitNet sizes
    python bench.py --leg ablation                 # prefill with ConvertDQ / LoadFull / sequential in place of the product path
    python bench.py --leg microbench               # lookup rates, load paths, cluster exchange
    TMAN_LIBRARY=paper_2511_11248_b200/libtman_stamps.so python bench.py --leg stamps   # where the prefill roles wait

Everything goes through the C ABI; one JSON line per result on stdout.  Weights and activations are
seeded synthetic data drawn on the device (timing does not depend on the values; parity is the tests'
business).  Weight sets rotate through copies whose total size exceeds L2, so every call streams from
HBM.  With --dense a case also times the same product with fp16 weights through torch.matmul (the
library GEMM/GEMV: a yardstick for what the low-bit weights buy or cost, not part of the path).
The headline run calls summaries() for the one-line digests it carries.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

L2_BYTES = 126e6
LLAMA3_8B_LAYER = [("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
                   ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096)]
QWEN25_7B_PROJ = [("gateup", 3584, 18944), ("down", 18944, 3584), ("qkv", 3584, 4608)]


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


def device_problem(torch, B, H, M, K, N, bits, group, seed, with_fp16_weights=False):
    """Seeded synthetic weights (uniform codes and zero-points, scales in [0.005, 0.02]) packed by the
    library, and activations ~ N(0, 1), all drawn on the device.  with_fp16_weights: also the dequantized
    weights as fp16 [N][K] (what the LoadFull ablation variant reads)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    codes = torch.randint(0, 1 << bits, (K, N), dtype=torch.uint8, device="cuda", generator=g)
    zeros = torch.randint(0, 1 << bits, (K // group, N), dtype=torch.uint8, device="cuda", generator=g)
    scales = (0.005 + 0.015 * torch.rand((K // group, N), device="cuda", generator=g)).to(torch.float16)
    x = torch.randn((M, K), device="cuda", generator=g).to(torch.float16)
    packed = torch.empty(B.tman_packed_bytes(K, N, bits, group), dtype=torch.uint8, device="cuda")
    B.tman_pack_weights(codes, scales, zeros, K, N, bits, group, packed)
    if with_fp16_weights:
        w = scales.float().repeat_interleave(group, 0) * (codes.float() - zeros.float().repeat_interleave(group, 0))
        return packed, x, w.to(torch.float16).t().contiguous()
    return packed, x


def workspace(torch, B, op, M, K, N, bits, group):
    ws = torch.empty(B.tman_workspace_bytes(op, M, K, N, bits, group), dtype=torch.uint8, device="cuda")
    B.tman_workspace_init(ws)
    return ws


# ---- one shape -------------------------------------------------------------------------------------

def case(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    ap = argparse.ArgumentParser(prog="bench.py --leg case")
    ap.add_argument("--op", choices=["gemv", "gemm", "ternary", "ternary_i8"], default="gemv",
                    help="ternary: integer decode (M = 1); ternary_i8: integer prefill")
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=64)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--copies", type=int, default=1, help="rotate over this many packed copies")
    ap.add_argument("--graph", action="store_true", help="time the calls replayed from one CUDA graph")
    a = ap.parse_args(list(rest))
    if a.op in ("ternary", "ternary_i8"):
        a.bits = 2
    packed0, x = device_problem(torch, B, H, a.M, a.K, a.N, a.bits, a.group, seed=1)
    packed = [packed0] + [packed0.clone() for _ in range(a.copies - 1)]
    y = torch.empty((a.M, a.N), dtype=torch.float16, device="cuda")
    if a.op in ("ternary", "ternary_i8"):
        # the integer path reads only the planes of the packed buffer (codes 0..3 here: timing, not parity)
        ws = workspace(torch, B, B.OP_GEMV, 1, a.K, a.N, 2, a.group)
        sa = torch.empty(max(a.M, 64), dtype=torch.float32, device="cuda")
        if a.op == "ternary":
            q = torch.empty((1, a.K), dtype=torch.int16, device="cuda")
            B.tman_quantize_rows(x, 1, a.K, 32767, q, sa)
            fn = lambda pk, x_, y_, M, K, N, bits, group, ws_: B.tman_mpgemv_ternary(pk, q, sa, 0.02, y_, None, 1, K, N, group, ws_)
        else:
            q = torch.empty((a.M, a.K), dtype=torch.int8, device="cuda")
            B.tman_quantize_rows_i8(x, a.M, a.K, q, sa)
            fn = lambda pk, x_, y_, M, K, N, bits, group, ws_: B.tman_mpgemm_ternary_i8(pk, q, sa, 0.02, y_, M, K, N, group, ws_)
    else:
        op = B.OP_GEMV if a.op == "gemv" else B.OP_GEMM
        fn = B.tman_mpgemv if a.op == "gemv" else B.tman_mpgemm
        ws = workspace(torch, B, op, a.M, a.K, a.N, a.bits, a.group)
    def calls():
        for i in range(a.iters):
            fn(packed[i % a.copies], x, y, a.M, a.K, a.N, a.bits, a.group, ws)

    for i in range(3):
        fn(packed[i % a.copies], x, y, a.M, a.K, a.N, a.bits, a.group, ws)
    torch.cuda.synchronize()
    if a.graph:
        # back-to-back calls without host launch cost: what a call takes inside a decoding step
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            calls()
        g.replay()
        torch.cuda.synchronize()
        us = event_us(torch, g.replay, 7)[0] / a.iters
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        calls()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / a.iters
    assert B.tman_read_status(ws) == 0
    print(json.dumps({"leg": "case", "op": a.op, "M": a.M, "K": a.K, "N": a.N, "bits": a.bits, "group": a.group,
                      "us_per_call": round(us, 2), "iters": a.iters, "copies": a.copies, "graph": bool(a.graph)}))


# ---- decode: config 1 and the layer sweep (config 3) -------------------------------------------------

def decode_calls_us(torch, B, H, M, bits, group, calls, reps):
    """calls: list of lists of (K, N) that share activations (one grouped launch each).  Returns the
    median and best time of one pass over all calls, replayed from a CUDA graph over rotating sets."""
    pass_bytes = sum(weight_bytes(K, N, bits, group) for grp in calls for K, N in grp)
    nsets = max(2, int(2.2 * L2_BYTES // pass_bytes) + 1)
    sets = []
    for s in range(nsets):
        entry = []
        for ci, grp in enumerate(calls):
            K = grp[0][0]
            packed, x = [], None
            for gi, (_, N) in enumerate(grp):
                p, xx = device_problem(torch, B, H, M, K, N, bits, group, seed=1000 * s + 10 * ci + gi)
                packed.append(p)
                x = xx if x is None else x
            ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _, N in grp]
            entry.append((K, [N for _, N in grp], packed, x, ys))
        sets.append(entry)
    wss = [workspace(torch, B, B.OP_GEMV, M, grp[0][0], sum(N for _, N in grp), bits, group) for grp in calls]

    def one_pass(e):
        for (K, Ns, packed, x, ys), ws in zip(e, wss):
            if len(Ns) == 1:
                B.tman_mpgemv(packed[0], x, ys[0], M, K, Ns[0], bits, group, ws)
            else:
                B.tman_mpgemv_grouped(packed, x, ys, M, K, Ns, bits, group, ws)

    for e in sets:
        one_pass(e)
    torch.cuda.synchronize()
    nrep = 4 * nsets
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(nrep):
            one_pass(sets[i % nsets])
    g.replay()
    torch.cuda.synchronize()
    med, best = event_us(torch, g.replay, reps)
    assert all(B.tman_read_status(w) == 0 for w in wss)
    return med / nrep, best / nrep, pass_bytes, nsets


LAYER_CALLS = [[(4096, 4096), (4096, 1024), (4096, 1024)], [(4096, 4096)], [(4096, 14336), (4096, 14336)],
               [(14336, 4096)]]


def dense_layer_us(torch, M, reps):
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
    return event_us(torch, g.replay, reps)[0] / nrep


def config1_result(torch, B, H, reps=7):
    med, best, nbytes, nsets = decode_calls_us(torch, B, H, 1, 4, 64, [[(4096, 4096)]], reps)
    return {"leg": "config1", "M": 1, "K": 4096, "N": 4096, "bits": 4, "group": 64, "us": round(med, 2),
            "us_best": round(best, 2), "weight_stream_GBs": round(nbytes / med / 1e3, 1), "weight_sets": nsets}


def config1(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    print(json.dumps(config1_result(torch, B, H)), flush=True)


def config3_results(torch, B, H, reps=7, dense=False, bits_list=(2, 3, 4), Ms=(1, 2, 4, 8)):
    out = []
    dense_us = {M: dense_layer_us(torch, M, reps) for M in Ms} if dense else {}
    torch.cuda.empty_cache()
    for bits in bits_list:
        for M in Ms:
            med, best, nbytes, nsets = decode_calls_us(torch, B, H, M, bits, 128, LAYER_CALLS, reps)
            r = {"leg": "config3", "M": M, "bits": bits, "group": 128, "layer_us": round(med, 2),
                 "layer_us_best": round(best, 2), "weight_stream_GBs": round(nbytes / med / 1e3, 1),
                 "weight_sets": nsets, "launches_per_layer": len(LAYER_CALLS)}
            if dense:
                r["dense_fp16_layer_us"] = round(dense_us[M], 2)
                r["speedup_vs_dense_fp16"] = round(dense_us[M] / med, 2)
            out.append(r)
            torch.cuda.empty_cache()
    return out


def config3_projection_results(torch, B, H, reps=7, bits_list=(2, 3, 4), Ms=(1, 2, 4, 8)):
    """Each of the seven projections alone (one call per projection, rotating copies larger than L2)."""
    out = []
    for bits in bits_list:
        for M in Ms:
            for name, K, N in LLAMA3_8B_LAYER:
                med, best, nbytes, nsets = decode_calls_us(torch, B, H, M, bits, 128, [[(K, N)]], reps)
                out.append({"leg": "config3_projection", "proj": name, "M": M, "K": K, "N": N, "bits": bits, "group": 128,
                            "us": round(med, 2), "us_best": round(best, 2), "weight_stream_GBs": round(nbytes / med / 1e3, 1)})
                torch.cuda.empty_cache()
    return out


def config3(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    ap = argparse.ArgumentParser(prog="bench.py --leg config3")
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--per-projection", action="store_true", help="also time each of the seven projections alone")
    ap.add_argument("--reps", type=int, default=7)
    a = ap.parse_args(list(rest))
    for r in config3_results(torch, B, H, a.reps, a.dense):
        print(json.dumps(r), flush=True)
    if a.per_projection:
        for r in config3_projection_results(torch, B, H, a.reps):
            print(json.dumps(r), flush=True)


# ---- prefill shape sweep (config 5) --------------------------------------------------------------------

def dense_case_us(torch, M, K, N, reps):
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

    return event_us(torch, run, reps)[0] / ncopy


def prefill_case(torch, B, H, M, K, N, bits, group, reps):
    p0, x = device_problem(torch, B, H, M, K, N, bits, group, seed=5)
    ncopy = max(2, int(2.2 * L2_BYTES // p0.numel()) + 1)
    pk = [p0] + [p0.clone() for _ in range(ncopy - 1)]
    ws = workspace(torch, B, B.OP_GEMM, M, K, N, bits, group)
    ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
    for i in range(3):
        B.tman_mpgemm(pk[i % ncopy], x, ys[i % 2], M, K, N, bits, group, ws)
    torch.cuda.synchronize()

    def run():
        for i in range(ncopy):
            B.tman_mpgemm(pk[i], x, ys[i % 2], M, K, N, bits, group, ws)

    us = event_us(torch, run, reps)[0] / ncopy
    assert B.tman_read_status(ws) == 0
    plan = B.tman_debug_gemm_plan(M, K, N, bits, group)
    return {"leg": "config5", "M": M, "K": K, "N": N, "bits": bits, "group": group, "us": round(us, 1),
            "TFLOPs": round(2.0 * M * K * N / us / 1e6, 1), "split_tiles": 1 - plan["whole_tiles"],
            "column_tiles": plan["tiles_n"]}


def config5_results(torch, B, H, reps=7, dense=False, bits_list=(2, 4), groups=(128,), Ms=(128, 512, 2048, 8192)):
    out, dense_us = [], {}
    for bits in bits_list:
        for group in groups:
            for M in Ms:
                for _, K, N in QWEN25_7B_PROJ:
                    r = prefill_case(torch, B, H, M, K, N, bits, group, reps)
                    if dense:
                        if (M, K, N) not in dense_us:
                            dense_us[(M, K, N)] = dense_case_us(torch, M, K, N, reps)
                        r["dense_fp16_us"] = round(dense_us[(M, K, N)], 1)
                        r["time_vs_dense_fp16"] = round(r["us"] / dense_us[(M, K, N)], 2)
                    out.append(r)
                    torch.cuda.empty_cache()
    return out


def config5(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    ap = argparse.ArgumentParser(prog="bench.py --leg config5")
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--all-groups", action="store_true", help="group 64 as well as 128")
    ap.add_argument("--reps", type=int, default=7)
    a = ap.parse_args(list(rest))
    for r in config5_results(torch, B, H, a.reps, a.dense, groups=(64, 128) if a.all_groups else (128,)):
        print(json.dumps(r), flush=True)


# ---- integer path: ternary weights, 16-bit integer activations (paper Sec. 6.1, BitNet kernel sizes) --------

def ternary_results(torch, B, H, reps=7):
    out = []
    for K, N in ((2560, 2560), (2560, 6912), (6912, 2560), (6912, 6912)):
        g = torch.Generator(device="cuda")
        g.manual_seed(K + N)
        nbytes = K * N // 4                                   # the bit planes are all the kernel streams
        ncopy = max(2, int(2.2 * L2_BYTES // nbytes) + 1)
        group = 128
        packed = []
        for _ in range(ncopy):
            codes = torch.randint(0, 3, (K, N), dtype=torch.uint8, device="cuda", generator=g)
            pk = torch.empty(B.tman_packed_bytes(K, N, 2, group), dtype=torch.uint8, device="cuda")
            B.tman_pack_weights(codes, torch.ones((K // group, N), dtype=torch.float16, device="cuda"),
                                torch.ones((K // group, N), dtype=torch.uint8, device="cuda"), K, N, 2, group, pk)
            packed.append(pk)
        x = torch.randn((1, K), device="cuda", generator=g).to(torch.float16)
        a = torch.empty((1, K), dtype=torch.int16, device="cuda")
        sa = torch.empty(64, dtype=torch.float32, device="cuda")
        y = torch.empty((1, N), dtype=torch.float16, device="cuda")
        ws = workspace(torch, B, B.OP_GEMV, 1, K, N, 2, group)

        def one_pass(with_quant):
            for pk in packed:
                if with_quant:
                    B.tman_quantize_rows(x, 1, K, 32767, a, sa)
                B.tman_mpgemv_ternary(pk, a, sa, 0.02, y, None, 1, K, N, group, ws)

        res = {"leg": "ternary", "M": 1, "K": K, "N": N, "copies": ncopy, "plane_bytes": nbytes}
        for with_quant in (False, True):
            one_pass(True)
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr):
                for _ in range(4):
                    one_pass(with_quant)
            gr.replay()
            torch.cuda.synchronize()
            us = event_us(torch, gr.replay, reps)[0] / (4 * ncopy)
            key = "us_with_quantize" if with_quant else "us"
            res[key] = round(us, 2)
            if not with_quant:
                res["weight_stream_GBs"] = round(nbytes / us / 1e3, 1)
        assert B.tman_read_status(ws) == 0
        # the prefill side's dequantization step alone: packed planes -> INT8 [N][K]
        w8 = [torch.empty((N, K), dtype=torch.int8, device="cuda") for _ in range(min(ncopy, 16))]
        wsd = workspace(torch, B, B.OP_AUX, 1, K, N, 2, group)

        def dq():
            for i, pk in enumerate(packed):
                B.tman_dequant_ternary_int8(pk, K, N, group, w8[i % len(w8)], wsd)

        dq()
        torch.cuda.synchronize()
        gd = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gd):
            dq()
        gd.replay()
        torch.cuda.synchronize()
        us = event_us(torch, gd.replay, reps)[0] / ncopy
        assert B.tman_read_status(wsd) == 0
        res["dequant_int8_us"] = round(us, 2)
        res["dequant_int8_GBs"] = round((nbytes + K * N) / us / 1e3, 1)      # planes read + INT8 written
        out.append(res)
        del packed, w8
        torch.cuda.empty_cache()
    return out


def ternary_prefill_results(torch, B, H, reps=7):
    """INT8 prefill on the BitNet sizes: the fused kernel against fp16 torch.matmul on the same shape."""
    out = []
    group = 128
    for M in (128, 1024, 4096):
        for K, N in ((2560, 2560), (2560, 6912), (6912, 2560), (6912, 6912)):
            g = torch.Generator(device="cuda")
            g.manual_seed(M + K + N)
            codes = torch.randint(0, 3, (K, N), dtype=torch.uint8, device="cuda", generator=g)
            pk0 = torch.empty(B.tman_packed_bytes(K, N, 2, group), dtype=torch.uint8, device="cuda")
            B.tman_pack_weights(codes, torch.ones((K // group, N), dtype=torch.float16, device="cuda"),
                                torch.ones((K // group, N), dtype=torch.uint8, device="cuda"), K, N, 2, group, pk0)
            ncopy = max(2, int(2.2 * L2_BYTES // pk0.numel()) + 1)
            pk = [pk0] + [pk0.clone() for _ in range(ncopy - 1)]
            x = torch.randn((M, K), device="cuda", generator=g).to(torch.float16)
            a8 = torch.empty((M, K), dtype=torch.int8, device="cuda")
            sa = torch.empty(max(M, 64), dtype=torch.float32, device="cuda")
            B.tman_quantize_rows_i8(x, M, K, a8, sa)
            ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
            ws = workspace(torch, B, B.OP_AUX, 1, K, N, 2, group)

            def run():
                for i in range(ncopy):
                    B.tman_mpgemm_ternary_i8(pk[i], a8, sa, 0.02, ys[i % 2], M, K, N, group, ws)

            run()
            torch.cuda.synchronize()
            us = event_us(torch, run, reps)[0] / ncopy
            assert B.tman_read_status(ws) == 0
            qus = event_us(torch, lambda: B.tman_quantize_rows_i8(x, M, K, a8, sa), reps)[0]
            del pk
            torch.cuda.empty_cache()
            dus = dense_case_us(torch, M, K, N, reps)
            out.append({"leg": "ternary_prefill", "M": M, "K": K, "N": N, "us": round(us, 1),
                        "TOPs": round(2.0 * M * K * N / us / 1e6, 1), "quantize_rows_us": round(qus, 1),
                        "dense_fp16_torch_us": round(dus, 1), "time_vs_dense_fp16": round(us / dus, 2)})
            torch.cuda.empty_cache()
    return out


def ternary(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    for r in ternary_results(torch, B, H):
        print(json.dumps(r), flush=True)
    for r in ternary_prefill_results(torch, B, H):
        print(json.dumps(r), flush=True)


# ---- ablations (paper Sec. 6.5) --------------------------------------------------------------------------

ABLATION_SHAPES = [(128, 4096, 4096), (1024, 4096, 4096), (1024, 4096, 14336), (4096, 4096, 14336)]


def ablation_results(torch, B, H, reps=7, shapes=ABLATION_SHAPES, group=128):
    """4-bit prefill with one part replaced: ConvertDQ and LoadFull against the lookup dequantization,
    sequential against pipelined; LoadFull is also the kernel's own fp16 GEMM (no dequantization at all),
    so product / load_full is the overhead of fusing the dequantization.  torch.matmul with fp16 weights
    is the library yardstick."""
    out = []
    for M, K, N in shapes:
        p0, x, wt0 = device_problem(torch, B, H, M, K, N, 4, group, seed=9, with_fp16_weights=True)
        ncopy = max(2, int(2.2 * L2_BYTES // wt0.numel() // 2) + 1)
        pk = [p0] + [p0.clone() for _ in range(ncopy - 1)]
        wts = [wt0] + [wt0.clone() for _ in range(ncopy - 1)]
        ws = workspace(torch, B, B.OP_GEMM, M, K, N, 4, group)
        ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]
        row = {"leg": "ablation", "M": M, "K": K, "N": N, "bits": 4, "group": group, "copies": ncopy}
        for name in ("product", "convert_dq", "load_full", "sequential"):
            def run():
                for i in range(ncopy):
                    B.tman_debug_mpgemm_variant(name, pk[i], x, ys[i % 2], M, K, N, 4, group, ws, wts[i])
            run()
            torch.cuda.synchronize()
            row[name + "_us"] = round(event_us(torch, run, reps)[0] / ncopy, 1)
        assert B.tman_read_status(ws) == 0
        del pk, wts
        torch.cuda.empty_cache()
        row["dense_fp16_torch_us"] = round(dense_case_us(torch, M, K, N, reps), 1)
        row["convert_dq_over_product"] = round(row["convert_dq_us"] / row["product_us"], 2)
        row["sequential_over_product"] = round(row["sequential_us"] / row["product_us"], 2)
        row["product_over_load_full"] = round(row["product_us"] / row["load_full_us"], 2)
        row["product_TFLOPs"] = round(2.0 * M * K * N / row["product_us"] / 1e6, 1)
        out.append(row)
        torch.cuda.empty_cache()
    return out


def ablation(args, rest=()):
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    for r in ablation_results(torch, B, H):
        print(json.dumps(r), flush=True)


# ---- role time stamps of the prefill kernel (needs TMAN_LIBRARY=.../libtman_stamps.so) -------------------

def stamps(args, rest=()):
    """Where each role of the prefill pipeline waits (paper Sec. 4.2, Fig. 9).  Run as
    TMAN_LIBRARY=paper_2511_11248_b200/libtman_stamps.so python bench.py --leg stamps"""
    import torch
    from paper_2511_11248_b200 import binding as B, helpers as H
    for M, K, N, bits in ((1024, 4096, 14336, 4), (1024, 4096, 4096, 4), (2048, 3584, 18944, 4), (128, 3584, 18944, 4),
                          (1024, 4096, 14336, 2)):
        group = 128
        packed, x = device_problem(torch, B, H, M, K, N, bits, group, seed=3)
        ws = workspace(torch, B, B.OP_GEMM, M, K, N, bits, group)
        y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        for _ in range(3):
            B.tman_mpgemm(packed, x, y, M, K, N, bits, group, ws)
        torch.cuda.synchronize()
        assert B.tman_read_status(ws) == 0
        plan = B.tman_debug_gemm_plan(M, K, N, bits, group)
        ctas = plan["workers"] * (2 if plan["pair"] else 1)
        st = B.tman_debug_role_stamps(ws, ctas).astype(np.float64)
        role = lambda w0, w1, col: float(np.median(st[:, w0:w1, col] / st[:, w0:w1, 2]))
        lead = st[::2] if plan["pair"] else st                 # in a pair only the first CTA issues the MMAs
        print(json.dumps({
            "leg": "stamps", "M": M, "K": K, "N": N, "bits": bits, "group": group, "ctas": ctas, "pair": plan["pair"],
            "role_clocks_median": float(np.median(st[:, 0, 2])),
            "producer_waits_for_free_stage": round(role(0, 1, 0), 3),
            "mma_waits_for_free_accumulators": round(float(np.median(lead[:, 1, 0] / lead[:, 1, 2])), 3),
            "mma_waits_for_dequantized_stage": round(float(np.median(lead[:, 1, 1] / lead[:, 1, 2])), 3),
            "dequant_waits_for_loaded_stage": round(role(2, 18, 0), 3),
            "epilogue_waits_for_accumulators": round(role(18, 26, 0), 3)}), flush=True)


# ---- digests for the headline line ------------------------------------------------------------------

def summaries(torch, B, H):
    """One-line digests of configs 1, 3 and 5, measured now: config 1 as [us, GB/s]; config 3 as layer
    weight-stream GB/s per bits x M with the speed-up over fp16 weights through torch.matmul; config 5
    as TFLOP/s per M (sum of flops / sum of time over the three shapes, group 128) per bit width with
    the time relative to fp16 weights through torch.matmul."""
    c1 = config1_result(torch, B, H, reps=5)
    c3 = {}
    for r in config3_results(torch, B, H, reps=5, dense=True):
        c3.setdefault(f"b{r['bits']}", {})[f"M{r['M']}"] = [r["weight_stream_GBs"], r["speedup_vs_dense_fp16"]]
    c5 = {}
    rows = config5_results(torch, B, H, reps=3, dense=True)
    for bits in (2, 4):
        for M in (128, 512, 2048, 8192):
            sel = [r for r in rows if r["bits"] == bits and r["M"] == M]
            flops = sum(2.0 * r["M"] * r["K"] * r["N"] for r in sel)
            us = sum(r["us"] for r in sel)
            dus = sum(r["dense_fp16_us"] for r in sel)
            c5.setdefault(f"b{bits}", {})[f"M{M}"] = [round(flops / us / 1e6, 1), round(us / dus, 2)]
    return {"config1": {"us": c1["us"], "GBs": c1["weight_stream_GBs"]},
            "config3": {"what": "[layer weight-stream GB/s, speed-up over fp16 torch.matmul], group 128", **c3},
            "config5": {"what": "[TFLOP/s over the 3 shapes, time relative to fp16 torch.matmul], group 128", **c5}}


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


def microbench(args, rest=()):
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
