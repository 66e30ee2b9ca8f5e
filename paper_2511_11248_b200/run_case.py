"""Run one synthetic matmul case through the C ABI and print its device time.

    python -m paper_2511_11248_b200.run_case --op gemv --M 1 --K 4096 --N 14336 --bits 2 --group 64

Useful for timing a single shape and as the command line to profile (a few launches, one shape).
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B, helpers as H, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["gemv", "gemm"], default="gemv")
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=64)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--copies", type=int, default=1, help="rotate over this many packed copies")
    a = ap.parse_args()
    c = synth.small_case(a.M, a.K, a.N, a.bits, a.group, seed=1)
    dev = H.device_case(c)
    packed = [H.pack_case(c, dev)]
    for _ in range(a.copies - 1):
        packed.append(packed[0].clone())
    op = B.OP_GEMV if a.op == "gemv" else B.OP_GEMM
    fn = B.tman_mpgemv if a.op == "gemv" else B.tman_mpgemm
    ws = H.alloc_workspace(op, a.M, a.K, a.N, a.bits, a.group)
    y = torch.empty((a.M, a.N), dtype=torch.float16, device="cuda")
    for i in range(3):
        fn(packed[i % a.copies], dev["x"], y, a.M, a.K, a.N, a.bits, a.group, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.iters):
        fn(packed[i % a.copies], dev["x"], y, a.M, a.K, a.N, a.bits, a.group, ws)
    e1.record()
    torch.cuda.synchronize()
    assert B.tman_read_status(ws) == 0
    us = e0.elapsed_time(e1) * 1e3 / a.iters
    print(json.dumps({"op": a.op, "M": a.M, "K": a.K, "N": a.N, "bits": a.bits, "group": a.group,
                      "us_per_call": us, "iters": a.iters, "copies": a.copies}))


if __name__ == "__main__":
    main()
