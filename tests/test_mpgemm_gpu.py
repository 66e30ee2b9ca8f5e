"""Parity of tman_mpgemm (prefill path) with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import binding as B, helpers as H, synth

from parity import TOL, block_rows, check_every_output, rel_err, run

pytestmark = pytest.mark.gpu


def run_gemm(c, pack="library"):
    return run(B.OP_GEMM, c, pack=pack)[0]


def check_full(c, pack="library"):
    got = H.to_f64(run_gemm(c, pack))
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    e = rel_err(got, ref)
    assert e <= TOL, (c.name, e)


def check_sampled(c):
    """Full-size case.  The oracle computes one row in every block of 128 rows (the kernel's row tile),
    compared one by one; every other element of y is compared with an fp64 library matmul that must
    itself agree with the oracle on those rows."""
    y = run_gemm(c)
    rows = block_rows(c.M, c.seed)
    ref = orc.mpgemm_rows(c.x, c.codes, c.scales, c.zeros, c.group, rows)
    got = H.to_f64(y[torch.from_numpy(rows).cuda()])
    e = rel_err(got, ref)
    assert e <= TOL, (c.name, e)
    check_every_output(c, y, rows, ref)


SMALL = [
    # (M, K, N, bits, group): one tile, ragged M and N tiles, several k-blocks, every bit width
    (128, 128, 128, 4, 128), (128, 256, 128, 2, 64), (1, 256, 8, 4, 64), (100, 384, 136, 3, 128),
    (300, 512, 264, 4, 32), (257, 1024, 72, 2, 128), (129, 640, 392, 3, 64), (512, 2048, 256, 4, 64),
]


@pytest.mark.parametrize("M,K,N,bits,G", SMALL)
def test_small_cases(M, K, N, bits, G):
    check_full(synth.small_case(M, K, N, bits, G, seed=M + K + N + bits, outliers=(bits == 4)))


@pytest.mark.parametrize("M,K,N,bits,G", SMALL[::2] + [(600, 256, 7176, 2, 64), (300, 8192, 1024, 4, 128)])
def test_on_a_buffer_the_oracle_packed(M, K, N, bits, G):
    # the kernel reads a buffer that no GPU code produced
    check_full(synth.small_case(M, K, N, bits, G, seed=M + K + N + bits + 1), pack="oracle")


# Enough tokens and channels for the CTA-pair kernel (512-row tiles split over two SMs), with ragged
# row tiles, ragged channel ranges and every bit width; compared element by element.
PAIRED = [(600, 256, 7176, 2, 64), (1030, 128, 4744, 3, 128), (513, 256, 14344, 4, 64),
          (1024, 384, 3560, 4, 32)]


@pytest.mark.parametrize("M,K,N,bits,G", PAIRED)
def test_pair_kernel_cases(M, K, N, bits, G):
    check_full(synth.small_case(M, K, N, bits, G, seed=M + K + N + bits, outliers=(bits == 4)))


# Long K and few tiles: every tile's k-blocks go to several workers, which exchange fp32 chunks through
# the workspace and share the summing.  Pairs of CTAs with two and one row block, a single CTA, ragged
# M and N, every bit width; compared element by element.
SPLIT = [(300, 8192, 1024, 4, 128), (520, 8192, 1288, 2, 64), (200, 16384, 520, 3, 128), (100, 24576, 2560, 3, 128)]
# Slightly fewer tiles than workers (or a few more than a whole round): the last tiles' k-blocks are laid
# end to end and dealt in equal spans; a tile cut by a span boundary is summed by the worker that ends it.
SPANS = [(600, 8192, 5120, 4, 128), (1100, 4096, 6400, 2, 64)]


@pytest.mark.parametrize("M,K,N,bits,G", SPLIT)
def test_split_tile_cases(M, K, N, bits, G):
    plan = B.tman_debug_gemm_plan(M, K, N, bits, G)
    assert plan["pieces"] >= 2, plan               # the shape must take the path this test is about
    c = synth.small_case(M, K, N, bits, G, seed=M + K + N + bits)
    check_full(c)
    # the same call again on the same workspace: flags and partial tiles were left ready
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    ws = H.alloc_workspace(B.OP_GEMM, c.M, c.K, c.N, c.bits, c.group)
    ys = []
    for _ in range(3):
        y = H.alloc_y(c.M, c.N)
        B.tman_mpgemm(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, ws)
        ys.append(y)
    assert B.tman_read_status(ws) == 0
    assert torch.equal(ys[0], ys[1]) and torch.equal(ys[1], ys[2])   # fixed summation order: same bits


@pytest.mark.parametrize("M,K,N,bits,G", SPANS)
def test_span_cases(M, K, N, bits, G):
    plan = B.tman_debug_gemm_plan(M, K, N, bits, G)
    assert plan["span_tiles"] > 0, plan            # the shape must take the path this test is about
    c = synth.small_case(M, K, N, bits, G, seed=M + K + N + bits)
    y = run_gemm(c)
    rows = np.unique(np.concatenate([[255, 256, 511, 512], block_rows(M, M + N)]))
    ref = orc.mpgemm_rows(c.x, c.codes, c.scales, c.zeros, c.group, rows)
    got = H.to_f64(y[torch.from_numpy(rows).cuda()])
    assert rel_err(got, ref) <= TOL
    check_every_output(c, y, rows, ref)
    y2 = run_gemm(c)
    assert torch.equal(y, y2)                       # fixed summation order: same bits


def dequantized_fp16_nk(c):
    """fp16(s * (q - z)) as [N][K]: what the LoadFull variant reads in place of the packed weights."""
    z = np.repeat(c.zeros.astype(np.float32), c.group, axis=0)
    s_ = np.repeat(c.scales.astype(np.float32), c.group, axis=0)
    w = (s_ * (c.codes.astype(np.float32) - z)).astype(np.float16)           # one rounding, like the table's entries
    return torch.from_numpy(np.ascontiguousarray(w.T).view(np.int16)).cuda().view(torch.float16)


@pytest.mark.parametrize("variant", ["convert_dq", "load_full", "sequential"])
@pytest.mark.parametrize("M,K,N,G", [(100, 384, 136, 128), (600, 512, 7176, 64), (1024, 1024, 3560, 32)])
def test_ablation_variants_compute_the_same_numbers(variant, M, K, N, G):
    # Sec. 6.5: the variants replace how fp16 weights come about, or the pipelining; never the result
    if variant == "load_full" and N % 32:
        N = (N + 31) // 32 * 32        # the LoadFull variant takes whole 32-channel units only
    c = synth.small_case(M, K, N, 4, G, seed=M + K + N, outliers=True)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    ws = H.alloc_workspace(B.OP_GEMM, M, K, N, 4, G)
    want = H.alloc_y(M, N)
    B.tman_mpgemm(packed, dev["x"], want, M, K, N, 4, G, ws)
    wt = dequantized_fp16_nk(c) if variant == "load_full" else None
    got = H.alloc_y(M, N)
    B.tman_debug_mpgemm_variant(variant, packed, dev["x"], got, M, K, N, 4, G, ws, wt)
    assert B.tman_read_status(ws) == 0
    H.check_guards()
    assert torch.equal(got, want)                     # the same bits as the product path
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    assert rel_err(H.to_f64(got), ref) <= TOL
    if variant != "load_full":
        with pytest.raises(B.TmanError) as e:          # the variants exist for 4-bit weights
            B.tman_debug_mpgemm_variant(variant, packed, dev["x"], got, M, K, N, 2, G, ws, wt)
        assert e.value.status in (3, 4)


STAMPS_CHILD = """
import sys, numpy as np, torch
from paper_2511_11248_b200 import binding as B, helpers as H, synth
M, K, N, bits, G, out = [int(a) for a in sys.argv[1:6]] + [sys.argv[6]]
c = synth.small_case(M, K, N, bits, G, seed=M + K + N)
dev = H.device_case(c)
packed = H.pack_case(c, dev)
ws = H.alloc_workspace(B.OP_GEMM, M, K, N, bits, G)
y = H.alloc_y(M, N)
B.tman_mpgemm(packed, dev["x"], y, M, K, N, bits, G, ws)
assert B.tman_read_status(ws) == 0
H.check_guards()
plan = B.tman_debug_gemm_plan(M, K, N, bits, G)
ctas = plan["workers"] * (2 if plan["pair"] else 1)
np.save(out + ".y.npy", y.cpu().numpy().view(np.uint16))
np.save(out + ".stamps.npy", B.tman_debug_role_stamps(ws, ctas))
"""


@pytest.mark.parametrize("M,K,N,bits,G", [(1024, 1024, 3560, 4, 128), (300, 8192, 1024, 2, 64)])
def test_time_stamp_build_computes_the_same_bits(M, K, N, bits, G, tmp_path):
    # the library built with TMAN_ROLE_STAMPS reads the clock around every role's waits and nothing else:
    # its output must be bit-identical to the regular library's, and its stamps must be plausible
    import os
    import subprocess
    import sys
    from paper_2511_11248_b200 import build
    lib = build.build(stamps=True)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, TMAN_LIBRARY=lib, PYTHONPATH=root)
    out = str(tmp_path / "stamped")
    subprocess.run([sys.executable, "-c", STAMPS_CHILD, str(M), str(K), str(N), str(bits), str(G), out],
                   check=True, env=env, cwd=root, timeout=600)
    c = synth.small_case(M, K, N, bits, G, seed=M + K + N)
    want = run_gemm(c).cpu().numpy().view(np.uint16)
    assert np.array_equal(np.load(out + ".y.npy"), want)
    st = np.load(out + ".stamps.npy")                  # [ctas][26 warps][wait a, wait b, role, tag]
    assert np.all(st[:, :, 3] == 0x5354414D50)
    assert np.all(st[:, :, 2] > 0) and np.all(st[:, :, 0] >= 0) and np.all(st[:, :, 1] >= 0)
    assert np.all(st[:, :, 0] + st[:, :, 1] <= st[:, :, 2])      # a role cannot wait longer than it lives
    # the regular library says so when asked for stamps
    ws = H.alloc_workspace(B.OP_GEMM, M, K, N, bits, G)
    with pytest.raises(B.TmanError) as e:
        B.tman_debug_role_stamps(ws, 2)
    assert e.value.status == 3


def test_integer_case_is_exact():
    rng = np.random.default_rng(5)
    c = synth.small_case(130, 512, 136, 3, 64, seed=31)
    c.x[:] = rng.integers(-2, 3, size=c.x.shape).astype(np.float16)
    c.scales[:] = 1.0
    c.zeros[:] = 0
    got = H.to_f64(run_gemm(c))
    want = c.x.astype(np.int64) @ c.codes.astype(np.int64)
    assert np.array_equal(got, want.astype(np.float16).astype(np.float64))


def test_pair_kernel_refuses_a_foreign_buffer_and_a_small_workspace():
    """Enough tokens for CTA pairs: both CTAs of every cluster must leave cleanly on a header mismatch."""
    M, K, N, bits, G = 600, 512, 1024, 4, 128
    c = synth.small_case(M, K, N, bits, G, seed=77)
    dev = H.device_case(c)
    junk = torch.zeros(B.tman_packed_bytes(K, N, bits, G), dtype=torch.uint8, device="cuda")
    ws = H.alloc_workspace(B.OP_GEMM, M, K, N, bits, G)
    y = H.alloc_y(M, N, fill=3.0)
    B.tman_mpgemm(junk, dev["x"], y, M, K, N, bits, G, ws)
    assert B.tman_read_status(ws) == 5          # TMAN_ERR_BAD_PACKED
    assert bool((y == 3.0).all())
    H.check_guards()
    # the library is usable afterwards, on a freshly prepared workspace
    B.tman_workspace_init(ws)
    packed = H.pack_case(c, dev)
    B.tman_mpgemm(packed, dev["x"], y, M, K, N, bits, G, ws)
    assert B.tman_read_status(ws) == 0
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    assert float(np.max(np.abs(H.to_f64(y) - ref)) / np.max(np.abs(ref))) <= TOL
    # a workspace smaller than tman_workspace_bytes asks for is refused before any launch
    small = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TmanError) as e:
        B.tman_mpgemm(packed, dev["x"], y, M, K, N, bits, G, small)
    assert e.value.status == 4                  # TMAN_ERR_BUFFER_TOO_SMALL


def test_gemm_and_gemv_read_the_same_packed_buffer():
    c = synth.small_case(4, 1024, 264, 4, 64, seed=32)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    wsv = H.alloc_workspace(B.OP_GEMV, c.M, c.K, c.N, c.bits, c.group)
    wsm = H.alloc_workspace(B.OP_GEMM, c.M, c.K, c.N, c.bits, c.group)
    yv = H.alloc_y(c.M, c.N)
    ym = H.alloc_y(c.M, c.N)
    B.tman_mpgemv(packed, dev["x"], yv, c.M, c.K, c.N, c.bits, c.group, wsv)
    B.tman_mpgemm(packed, dev["x"], ym, c.M, c.K, c.N, c.bits, c.group, wsm)
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    scale = np.max(np.abs(ref))
    assert np.max(np.abs(H.to_f64(yv) - ref)) / scale <= TOL
    assert np.max(np.abs(H.to_f64(ym) - ref)) / scale <= TOL


@pytest.mark.parametrize("spec", synth.config4_specs(), ids=lambda s: s[0])
def test_config4(spec):
    c = synth.case_from_spec(spec)
    if c.N <= 4096:
        check_full(c)            # every element from the oracle itself
    else:
        check_sampled(c)


@pytest.mark.parametrize("spec", synth.config5_specs(), ids=lambda s: s[0])
def test_config5(spec):
    check_sampled(synth.case_from_spec(spec, outliers=True))
