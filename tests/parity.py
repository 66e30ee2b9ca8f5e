"""What the GPU parity tests share: running a case through the C ABI on guarded buffers, packed
either by the library or by the oracle, and comparing outputs with the oracle."""
import numpy as np
import torch

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import binding as B, helpers as H

TOL = 5e-3   # max|gpu - ref| / max|ref|, the bound stated for fp32 accumulation of fp16 inputs


def rel_err(got, ref):
    assert np.all(np.isfinite(got))
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


def oracle_packed(c):
    """The packed buffer as the oracle writes it, uploaded between guard bytes."""
    host = orc.pack(c.codes, c.scales, c.zeros, c.bits, c.group)
    dst = H.alloc_packed(c.K, c.N, c.bits, c.group)
    assert dst.numel() == host.size
    dst.copy_(torch.from_numpy(host))
    return dst


def run(op, c, dev=None, packed=None, pack="library"):
    """One call of tman_mpgemv (op 0) or tman_mpgemm (op 1) on guarded buffers; returns (y, ws, packed, dev)."""
    dev = dev or H.device_case(c)
    if packed is None:
        packed = oracle_packed(c) if pack == "oracle" else H.pack_case(c, dev)
    ws = H.alloc_workspace(op, c.M, c.K, c.N, c.bits, c.group)
    y = H.alloc_y(c.M, c.N)
    fn = B.tman_mpgemv if op == B.OP_GEMV else B.tman_mpgemm
    fn(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, ws)
    assert B.tman_read_status(ws) == 0
    H.check_guards()
    return y, ws, packed, dev


def dequantized(c):
    """s * (q - z) in fp64 (Sec. 2.2, the dequantization formula), for the library-matmul check below."""
    z = np.repeat(c.zeros.astype(np.float64), c.group, axis=0)
    s = np.repeat(c.scales.astype(np.float64), c.group, axis=0)
    return (c.codes.astype(np.float64) - z) * s


def check_every_output(c, y, oracle_rows, oracle_ref, tol=TOL, chunk=1024):
    """Compare EVERY element of y with an fp64 library matmul of the dequantized weights.  The library
    matmul is not trusted by itself: on the rows the oracle computed it must agree with the oracle to
    rounding.  Returns the largest error relative to max|ref|."""
    w = dequantized(c)
    x = c.x.astype(np.float64)
    at_rows = x[oracle_rows] @ w
    scale = float(np.max(np.abs(oracle_ref)))
    assert np.max(np.abs(at_rows - oracle_ref)) <= 1e-9 * scale
    worst = 0.0
    for r0 in range(0, c.M, chunk):
        ref = x[r0:r0 + chunk] @ w
        got = H.to_f64(y[r0:r0 + chunk])
        assert np.all(np.isfinite(got)), (c.name, r0)
        worst = max(worst, float(np.max(np.abs(got - ref))) / scale)
    assert worst <= tol, (c.name, worst)
    return worst


def block_rows(M, seed, block=128):
    """One row in every block of `block` rows (a different place in each), plus the corners."""
    rng = np.random.default_rng(seed)
    starts = np.arange(0, M, block)
    rows = starts + rng.integers(0, block, size=starts.size)
    rows = np.minimum(rows, M - 1)
    return np.unique(np.concatenate([rows, [0, M - 1, min(M - 1, 127), min(M - 1, 128)]])).astype(np.int64)
