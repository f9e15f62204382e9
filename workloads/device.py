"""Device-side (torch) allocation and filling of arenas for a workload.

Sizes are passed in by the caller (they come from the library's plan or from the
oracle); this module only allocates uint8 tensors and fills them by byte position
with the workload's counter-based value streams, or with a constant.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

from . import rng
from .configs import arena_key

FILL_BYTE = 0xCD


def alloc_filled(sizes: Sequence[int], seed: int, kind: int, device="cuda") -> List:
    """One uint8 tensor per rank, filled with the stream arena_key(seed, kind, rank)."""
    import torch
    out = []
    for r, n in enumerate(sizes):
        t = torch.empty(int(n), dtype=torch.uint8, device=device)
        if n:
            rng.torch_fill_bytes(t, arena_key(seed, kind, r))
        out.append(t)
    return out


def alloc_const(sizes: Sequence[int], value: int = FILL_BYTE, device="cuda") -> List:
    import torch
    return [torch.full((int(n),), value, dtype=torch.uint8, device=device) for n in sizes]


def host_slice(seed: int, kind: int, rank: int, start: int, nbytes: int) -> np.ndarray:
    """The bytes [start, start+nbytes) of the arena stream, regenerated on the host."""
    return rng.fill_bytes(arena_key(seed, kind, rank), nbytes, start_byte=start)
