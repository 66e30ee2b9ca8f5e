"""Small conveniences over the binding for tests and the benchmark: buffer allocation and
host<->device marshalling of a whole problem.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def device_case(case, device="cuda"):
    """Upload a synth.Case; returns dict of device tensors."""
    return {
        "codes": torch.from_numpy(case.codes).to(device),
        "scales": torch.from_numpy(case.scales.view(np.int16)).to(device).view(torch.float16),
        "zeros": torch.from_numpy(case.zeros).to(device),
        "x": torch.from_numpy(case.x.view(np.int16)).to(device).view(torch.float16),
    }


# Every buffer a call may write sits between two runs of guard bytes; check_guards() tells whether a
# kernel wrote outside what it was given.
GUARD_BYTES = 256
GUARD_VALUE = 0xC3
_guarded = []   # (what, whole allocation, payload bytes)


def guarded_bytes(nbytes, what, device="cuda"):
    """nbytes of device memory (256-byte aligned) with guard bytes before and after."""
    pad = (-nbytes) % 256
    whole = torch.full((GUARD_BYTES + nbytes + pad + GUARD_BYTES,), GUARD_VALUE, dtype=torch.uint8, device=device)
    _guarded.append((what, whole, nbytes))
    return whole[GUARD_BYTES:GUARD_BYTES + nbytes]


def check_guards(forget=False):
    """Raise if any guard byte around a guarded buffer has changed."""
    for what, whole, nbytes in _guarded:
        front_ok = bool((whole[:GUARD_BYTES] == GUARD_VALUE).all())
        back_ok = bool((whole[GUARD_BYTES + nbytes:] == GUARD_VALUE).all())
        if not (front_ok and back_ok):
            raise AssertionError(f"write outside {what} ({nbytes} bytes): "
                                 f"{'before' if not front_ok else 'after'} the buffer")
    if forget:
        _guarded.clear()


def alloc_y(M, N, fill=float("nan"), device="cuda"):
    """Output matrix [M][N] fp16 between guard bytes, pre-filled so that unwritten elements show."""
    y = guarded_bytes(M * N * 2, f"y[{M}][{N}]", device).view(torch.float16).view(M, N)
    y.fill_(fill)
    return y


def alloc_packed(K, N, bits, group, device="cuda"):
    return guarded_bytes(B.tman_packed_bytes(K, N, bits, group), "packed buffer", device)


def alloc_workspace(op, M, K, N, bits, group, device="cuda"):
    ws = guarded_bytes(B.tman_workspace_bytes(op, M, K, N, bits, group), "workspace", device)
    B.tman_workspace_init(ws)
    return ws


def pack_case(case, dev=None, device="cuda"):
    dev = dev or device_case(case, device)
    packed = alloc_packed(case.K, case.N, case.bits, case.group, device)
    B.tman_pack_weights(dev["codes"], dev["scales"], dev["zeros"], case.K, case.N, case.bits,
                        case.group, packed)
    return packed


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()
