"""Parity of tman_mpgemm (prefill path) with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import binding as B, helpers as H, synth

pytestmark = pytest.mark.gpu
TOL = 5e-3   # max|gpu - ref| / max|ref|


def run_gemm(c):
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    ws = H.alloc_workspace(B.OP_GEMM, c.M, c.K, c.N, c.bits, c.group)
    y = torch.full((c.M, c.N), float("nan"), dtype=torch.float16, device="cuda")
    B.tman_mpgemm(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, ws)
    assert B.tman_read_status(ws) == 0
    return y


def check_full(c):
    got = H.to_f64(run_gemm(c))
    assert np.all(np.isfinite(got)), c.name
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    e = float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
    assert e <= TOL, (c.name, e)


def check_sampled(c, n_rows=24):
    """Full-size case: every output must be finite; sampled rows are compared one by one."""
    y = run_gemm(c)
    assert bool(torch.isfinite(y).all()), c.name
    rng = np.random.default_rng(c.seed)
    rows = np.unique(np.concatenate([[0, c.M - 1, min(c.M - 1, 127), min(c.M - 1, 128)],
                                     rng.integers(0, c.M, size=n_rows)]))
    ref = orc.mpgemm_rows(c.x, c.codes, c.scales, c.zeros, c.group, rows)
    got = H.to_f64(y[torch.from_numpy(rows).cuda()])
    e = float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
    assert e <= TOL, (c.name, e)


SMALL = [
    # (M, K, N, bits, group): one tile, ragged M and N tiles, several k-blocks, every bit width
    (128, 128, 128, 4, 128), (128, 256, 128, 2, 64), (1, 256, 8, 4, 64), (100, 384, 136, 3, 128),
    (300, 512, 264, 4, 32), (257, 1024, 72, 2, 128), (129, 640, 392, 3, 64), (512, 2048, 256, 4, 64),
]


@pytest.mark.parametrize("M,K,N,bits,G", SMALL)
def test_small_cases(M, K, N, bits, G):
    check_full(synth.small_case(M, K, N, bits, G, seed=M + K + N + bits, outliers=(bits == 4)))


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
        y = torch.full((c.M, c.N), float("nan"), dtype=torch.float16, device="cuda")
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
    assert bool(torch.isfinite(y).all())
    rng = np.random.default_rng(M + N)
    rows = np.unique(np.concatenate([[0, M - 1, 255, 256, 511, 512], rng.integers(0, M, size=26)]))
    ref = orc.mpgemm_rows(c.x, c.codes, c.scales, c.zeros, c.group, rows)
    got = H.to_f64(y[torch.from_numpy(rows).cuda()])
    assert float(np.max(np.abs(got - ref)) / np.max(np.abs(ref))) <= TOL
    y2 = run_gemm(c)
    assert torch.equal(y, y2)                       # fixed summation order: same bits


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
    y = torch.full((M, N), 3.0, dtype=torch.float16, device="cuda")
    B.tman_mpgemm(junk, dev["x"], y, M, K, N, bits, G, ws)
    assert B.tman_read_status(ws) == 5          # TMAN_ERR_BAD_PACKED
    assert bool((y == 3.0).all())
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
    yv = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
    ym = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
    B.tman_mpgemv(packed, dev["x"], yv, c.M, c.K, c.N, c.bits, c.group, wsv)
    B.tman_mpgemm(packed, dev["x"], ym, c.M, c.K, c.N, c.bits, c.group, wsm)
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    scale = np.max(np.abs(ref))
    assert np.max(np.abs(H.to_f64(yv) - ref)) / scale <= TOL
    assert np.max(np.abs(H.to_f64(ym) - ref)) / scale <= TOL


@pytest.mark.parametrize("spec", synth.config4_specs(), ids=lambda s: s[0])
def test_config4(spec):
    check_sampled(synth.case_from_spec(spec), n_rows=48)


@pytest.mark.parametrize("spec", synth.config5_specs(), ids=lambda s: s[0])
def test_config5(spec):
    check_sampled(synth.case_from_spec(spec, outliers=True), n_rows=12)
