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


def alloc_packed(K, N, bits, group, device="cuda"):
    return torch.empty(B.tman_packed_bytes(K, N, bits, group), dtype=torch.uint8, device=device)


def alloc_workspace(op, M, K, N, bits, group, device="cuda"):
    ws = torch.empty(B.tman_workspace_bytes(op, M, K, N, bits, group), dtype=torch.uint8, device=device)
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
