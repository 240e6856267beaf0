"""Seeded synthetic inputs for the bounded-state restore path.

This module only *draws inputs*: registration geometries, token ids, chunk payload
bytes and block tables.  It contains none of the method's arithmetic (no digest, key,
checksum, window or commit logic) so that both the CPU oracle and the CUDA path can
be fed from it without sharing any computation.

The shapes follow the paper's workloads (Section 4 "System topology", Appendix
"Measured Capacity Tables"): 256-token chunks, 64,096 bytes of registered state per
token per rank (so one chunk is 16,408,576 bytes), two TP rank slices, and prefixes of
32K..512K tokens.  KV values do not matter to a byte mover, so payload bytes are
uniform random.  Token ids are uniform in [0, 129280).

All draws come from numpy's SFC64 bit generator keyed by (master seed, tag, ...), so any
chunk, table or token range can be regenerated on demand without materialising the rest.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

CHUNK_TOKENS = 256
VOCAB = 129280
MASTER_SEED = 0xB5B5260817826

_TAG_TOK, _TAG_DATA, _TAG_BT, _TAG_SIZES, _TAG_FAULT = 1, 2, 3, 4, 5


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.SFC64(np.random.SeedSequence([int(k) for k in key])))


@dataclass
class Layout:
    """A registration geometry: allocator groups and the tensors registered in each.

    block_tokens: tokens per paged block of each group (pool sizes depend on the prefix length
                  and come from `pool_blocks`).
    tensors:      (group, bytes_per_token) in registration order, group-major.
    """

    name: str
    block_tokens: list[int]
    tensors: list[tuple[int, int]] = field(default_factory=list)

    @property
    def n_groups(self) -> int:
        return len(self.block_tokens)

    @property
    def bytes_per_token(self) -> int:
        return sum(e for _, e in self.tensors)

    @property
    def chunk_bytes(self) -> int:
        return CHUNK_TOKENS * self.bytes_per_token


def baseline_layout() -> Layout:
    """Two allocator groups: 56 tensors x 1,120 B/token and 43 tensors x 32 B/token,
    64-token blocks (64,096 B/token => 16,408,576 B/chunk, the paper's Eq. 5 coefficient)."""
    tensors = [(0, 1120)] * 56 + [(1, 32)] * 43
    return Layout("baseline-2group-99tensor", [64, 64], tensors)


def hetero_layout(seed: int = MASTER_SEED, bytes_per_token: int = 64096,
                  name: str = "hetero-3group-170tensor") -> Layout:
    """170 registered tensors of heterogeneous per-token sizes (multiples of 16 B) that sum
    to `bytes_per_token` (64,096 by default), in three allocator groups with 64-, 16- and
    64-token blocks.  Tensors [0,90) -> group 0, [90,140) -> group 1, [140,170) -> group 2."""
    assert bytes_per_token % 16 == 0
    n, units_total = 170, bytes_per_token // 16
    rng = _rng(seed, _TAG_SIZES)
    # skewed weights: a few wide tensors, many narrow ones
    w = 1.0 + rng.integers(0, 64, size=n).astype(np.float64) ** 2 / 64.0
    units = 1 + np.floor((units_total - n) * w / w.sum()).astype(np.int64)
    left = units_total - int(units.sum())
    assert 0 <= left < n
    units[:left] += 1
    assert int(units.sum()) == units_total
    groups = [0] * 90 + [1] * 50 + [2] * 30
    tensors = [(g, int(16 * u)) for g, u in zip(groups, units)]
    return Layout(name, [64, 16, 64], tensors)


def mtp_on_layout(seed: int = MASTER_SEED) -> Layout:
    """The paper's MTP-on registration size: 170 tensors accounting to 16,633,856 B per chunk
    (64,976 B/token; Section 6.4 reports 532,283,392 B = 32 x 16,633,856 at W = 32).  The paper
    gives only the tensor count and the total, so the individual sizes are seeded like `hetero_layout`."""
    return hetero_layout(seed=seed + 1, bytes_per_token=64976, name="mtp-on-3group-170tensor")


def short_run_layout() -> Layout:
    """A registration dominated by the shortest destination runs a paged cache can have: 1,600
    tensors of 16 B per token in 16-token blocks (256-byte runs, 80 % of the bytes) beside 50
    tensors of 128 B per token in 64-token blocks (8 KiB runs).  32,000 B/token, 8,192,000 B per
    chunk, 25,800 runs per chunk: the stress case for an install kernel's per-run overhead."""
    return Layout("short-runs-2group-1650tensor", [16, 64], [(0, 16)] * 1600 + [(1, 128)] * 50)


def tiny_layout() -> Layout:
    """A very small geometry for brute-force tests: 2 groups, 3 tensors, 16 and 64-token blocks."""
    return Layout("tiny", [16, 64], [(0, 48), (0, 16), (1, 32)])


def tokens(n_tokens: int, seed: int = MASTER_SEED) -> np.ndarray:
    """int32 token ids, uniform in [0, VOCAB)."""
    return _rng(seed, _TAG_TOK).integers(0, VOCAB, size=n_tokens, dtype=np.int32)


def chunk_payload(layout: Layout, rank: int, chunk: int, seed: int = MASTER_SEED,
                  out: np.ndarray | None = None) -> np.ndarray:
    """Uniform random payload bytes of chunk `chunk` of rank slice `rank` (uint8, chunk_bytes)."""
    nbytes = layout.chunk_bytes
    assert nbytes % 8 == 0
    words = _rng(seed, _TAG_DATA, rank, chunk).integers(0, 2**64, size=nbytes // 8, dtype=np.uint64)
    if out is None:
        return words.view(np.uint8)
    out.view(np.uint64)[:] = words
    return out


def blocks_per_chunk(layout: Layout, group: int) -> int:
    return CHUNK_TOKENS // layout.block_tokens[group]


def pool_blocks(layout: Layout, group: int, n_chunks: int) -> int:
    """Physical pool size of a group: the logical blocks of the prefix plus one spare per eight
    (at least one), so a scatter through a wrong table entry lands on a canary block."""
    n_logical = n_chunks * blocks_per_chunk(layout, group)
    return n_logical + max(1, -(-n_logical // 8))


def block_table(layout: Layout, rank: int, group: int, n_chunks: int,
                seed: int = MASTER_SEED) -> np.ndarray:
    """A seeded random injection of the prefix's logical blocks into the group's pool (int32)."""
    n_logical = n_chunks * blocks_per_chunk(layout, group)
    perm = _rng(seed, _TAG_BT, rank, group).permutation(pool_blocks(layout, group, n_chunks))
    return np.ascontiguousarray(perm[:n_logical].astype(np.int32))


def fault_site(n_ranks: int, n_groups: int, lo_chunk: int, hi_chunk: int, case: int,
               seed: int = MASTER_SEED) -> tuple[int, int, int, int]:
    """A seeded (rank, group, chunk, u32-word-fraction-in-1e6) site for failure injection."""
    rng = _rng(seed, _TAG_FAULT, case)
    return (int(rng.integers(0, n_ranks)), int(rng.integers(0, n_groups)),
            int(rng.integers(lo_chunk, hi_chunk)), int(rng.integers(0, 1_000_000)))


CANARY = 0xA5
