"""Counter-based pseudo-random streams for synthetic inputs.

Everything here is a pure function of (key, counter): the value at position i
of a stream never depends on how many values were drawn before it, so the
host (numpy) and the device (torch) fill the same bytes independently.

This module holds no layout or re-sharding arithmetic: it only produces
numbers.  The 64-bit mixer is the published splitmix64 finaliser.
"""
from __future__ import annotations

import numpy as np

_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_GOLDEN = 0x9E3779B97F4A7C15
_MASK = (1 << 64) - 1


def mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrapping arithmetic)."""
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= np.uint64(_M1)
        z ^= z >> np.uint64(27)
        z *= np.uint64(_M2)
        z ^= z >> np.uint64(31)
    return z


def mix64_int(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * _M1) & _MASK
    z = ((z ^ (z >> 27)) * _M2) & _MASK
    return z ^ (z >> 31)


def stream_key(seed: int, *tags: int) -> int:
    """Derives the 64-bit key of one stream from a master seed and integer tags."""
    k = mix64_int(seed ^ _GOLDEN)
    for t in tags:
        k = mix64_int((k + _GOLDEN * (int(t) + 1)) & _MASK)
    return k


def hash_u64(key: int, start: int, count: int) -> np.ndarray:
    """h[i] = mix64(key + (start + i) * GOLDEN) for i in [0, count)."""
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return mix64(np.uint64(key) + idx * np.uint64(_GOLDEN))


def uniform01(key: int, start: int, count: int) -> np.ndarray:
    """53-bit uniform doubles in [0, 1)."""
    return (hash_u64(key, start, count) >> np.uint64(11)).astype(np.float64) * 2.0 ** -53


def permutation(key: int, n: int) -> np.ndarray:
    """Seeded permutation of 0..n-1: stable argsort of the hash stream."""
    return np.argsort(hash_u64(key, 0, n), kind="stable").astype(np.int64)


def bf16_bits(key: int, start: int, count: int) -> np.ndarray:
    """bf16 bit patterns of uniform values in [-1, 1).

    u24 = top 24 bits of the hash; f = u24 * 2^-23 - 1 is exact in fp32; the
    bf16 pattern is the upper 16 bits of that fp32 (truncation keeps [-1, 1)).
    """
    u24 = (hash_u64(key, start, count) >> np.uint64(40)).astype(np.float32)
    f = u24 * np.float32(2.0 ** -23) - np.float32(1.0)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def fill_bytes(key: int, nbytes: int, start_byte: int = 0) -> np.ndarray:
    """The byte range [start_byte, start_byte + nbytes) of the bf16 stream `key`
    (little-endian 16-bit elements), as a uint8 array."""
    first = start_byte // 2
    last = (start_byte + nbytes + 1) // 2
    raw = bf16_bits(key, first, last - first).view(np.uint8)
    off = start_byte - 2 * first
    return raw[off:off + nbytes].copy()


# ---- the same bf16 stream produced on a torch device --------------------------------

def _s64(x: int) -> int:
    x &= _MASK
    return x - (1 << 64) if x >= (1 << 63) else x


def torch_fill_bytes(out, key: int, chunk_elems: int = 1 << 26) -> None:
    """Fills the 1-D uint8 torch tensor `out` (any device, 2-byte aligned) with the bf16 stream `key`, bit-identical to fill_bytes(key, n)."""
    import torch

    n = out.numel()
    if n % 2:   # odd tail byte: the low byte of the last 16-bit element, made on the host
        out[n - 1:] = torch.from_numpy(fill_bytes(key, 1, start_byte=n - 1)).to(out.device)
        out = out[:n - 1]
        n -= 1
        if n == 0:
            return
    dst = out.view(torch.int16)
    n_el = n // 2
    dev = out.device
    m1, m2, g, k = _s64(_M1), _s64(_M2), _s64(_GOLDEN), _s64(key)
    for s in range(0, n_el, chunk_elems):
        c = min(chunk_elems, n_el - s)
        z = torch.arange(s, s + c, dtype=torch.int64, device=dev)
        z = z * g + k
        # logical right shifts on int64: arithmetic shift then mask off the sign fill
        z = (z ^ ((z >> 30) & ((1 << 34) - 1))) * m1
        z = (z ^ ((z >> 27) & ((1 << 37) - 1))) * m2
        z = z ^ ((z >> 31) & ((1 << 33) - 1))
        u24 = ((z >> 40) & ((1 << 24) - 1)).to(torch.float32)
        f = u24 * (2.0 ** -23) - 1.0
        bits = (f.view(torch.int32) >> 16).to(torch.int16)
        dst[s:s + c] = bits
        del z, u24, f, bits
