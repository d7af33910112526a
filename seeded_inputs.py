"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests/bench.

This module holds no allgather arithmetic: it only fills buffers.  The paper's workload is a
micro-benchmark allgather over fixed-size byte blocks whose content is irrelevant (Section IV-A:
block sizes 1 B .. 1 MiB, 5..320 processes, 5 warm-ups + 50 timed runs); the generators here give
blocks of those shapes whose every 32-bit word encodes where it came from, so that a block that
lands in the wrong slot, or a word that lands at the wrong offset, cannot compare equal.

    word(seed, r, i) = low 32 bits of splitmix64(seed XOR (r << 32 | i))

where r is the rank that owns the send block and i the word index inside the block.  A block of m
bytes is the first m bytes of that little-endian word stream.
"""
from __future__ import annotations

import numpy as np

SENTINEL = 0xA5          # receive buffers and workspaces are pre-filled with this byte
GUARD_BYTES = 4096       # guard band kept before and after every buffer handed to the library
BASE_SEED = 0x5BA4B170   # config k uses BASE_SEED + k; changing-data runs add the iteration

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 finaliser (uint64 in, uint64 out), the usual public constants."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += np.uint64(0x9E3779B97F4A7C15)
        x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        x = x ^ (x >> np.uint64(31))
    return x


def send_blocks(P: int, m: int, seed: int) -> np.ndarray:
    """Send buffers of all P ranks as one contiguous uint8 array of shape (P, m).

    Row r is rank r's send block (m bytes).  m may be any size >= 0; when m is not a multiple of
    4 the last word is truncated.
    """
    if P < 0 or m < 0:
        raise ValueError("P and m must be non-negative")
    words = (m + 3) // 4
    out = np.empty((P, m), dtype=np.uint8)
    if P == 0 or m == 0:
        return out
    idx = np.arange(words, dtype=np.uint64)
    # generate a bounded number of ranks at a time so large configurations stay cheap in memory
    rows_per_pass = max(1, (1 << 22) // max(words, 1))
    for r0 in range(0, P, rows_per_pass):
        r1 = min(P, r0 + rows_per_pass)
        ranks = np.arange(r0, r1, dtype=np.uint64)[:, None]
        key = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ ((ranks << np.uint64(32)) | idx[None, :])
        w32 = (splitmix64(key) & np.uint64(0xFFFFFFFF)).astype("<u4")
        out[r0:r1] = w32.view(np.uint8).reshape(r1 - r0, words * 4)[:, :m]
    return out


def send_blocks_v(counts, seed: int) -> np.ndarray:
    """Concatenated send blocks of different sizes: rank r contributes counts[r] bytes, taken
    from the same per-rank word stream as send_blocks."""
    counts = [int(c) for c in counts]
    out = np.empty(sum(counts), dtype=np.uint8)
    pos = 0
    for r, c in enumerate(counts):
        if c:
            words = (c + 3) // 4
            key = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ ((np.uint64(r) << np.uint64(32))
                                                           | np.arange(words, dtype=np.uint64))
            w32 = (splitmix64(key) & np.uint64(0xFFFFFFFF)).astype("<u4")
            out[pos:pos + c] = w32.view(np.uint8)[:c]
        pos += c
    return out


def block_counts(P: int, seed: int, kind: str = "mixed", unit: int = 16, scale: int = 64) -> list:
    """Seeded per-rank byte counts for allgatherv runs: multiples of `unit`, about `scale` units
    on average; "mixed" includes empty blocks and a few large ones."""
    key = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + np.arange(P, dtype=np.uint64)
    h = splitmix64(key)
    base = (h % np.uint64(2 * scale + 1)).astype(np.int64)
    if kind == "mixed":
        sel = ((h >> np.uint64(40)) % np.uint64(8)).astype(np.int64)
        base = np.where(sel == 0, 0, base)            # one in eight is empty
        base = np.where(sel == 1, base * 6, base)     # one in eight is several times larger
    return [int(b) * unit for b in base]


def sentinel_buffer(nbytes: int, value: int = SENTINEL) -> np.ndarray:
    """A uint8 buffer of nbytes filled with the sentinel byte."""
    return np.full(nbytes, value, dtype=np.uint8)


def sample_indices(count: int, n: int, seed: int) -> np.ndarray:
    """`count` pseudo-random indices in [0, n), reproducible from the seed (for sampled compares)."""
    if n <= 0:
        return np.empty(0, dtype=np.int64)
    key = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + np.arange(count, dtype=np.uint64)
    return (splitmix64(key) % np.uint64(n)).astype(np.int64)
