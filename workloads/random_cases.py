"""Seeded random reshard problems for stress tests: odd shapes, odd cuts, odd byte offsets.

Each side of a problem partitions every tensor's global shape by a random grid into local
boxes; a local box is stored whole or as several flat ranges of its C-order flattening
(irregular shards); entries land in random buffers, in random order, with random gaps, so
byte offsets have arbitrary residues.  Metadata only.
"""
from __future__ import annotations

from itertools import product
from typing import List, Sequence, Tuple

import numpy as np

from .layouts import ReshardCase
from .meta import BOX, FLAT_SLICE, ShardMeta, ShardedState, prod


def _cuts(rng: np.random.Generator, n: int, max_parts: int) -> List[int]:
    parts = int(rng.integers(1, min(max_parts, n) + 1)) if n > 0 else 1
    inner = sorted(rng.choice(np.arange(1, n), size=parts - 1, replace=False).tolist()) if parts > 1 else []
    return [0] + inner + [n]


def random_side(rng: np.random.Generator, tensors: Sequence[Tuple[str, Tuple[int, ...], int]], n_bufs: int,
                *, max_parts: int = 3, flat_prob: float = 0.5, replicas: int = 1, gap_mod: int = 0,
                shuffle: bool = True, element_aligned: bool = False) -> ShardedState:
    """tensors: (fqn, global shape, itemsize).  gap_mod > 0 inserts random gaps of
    0..gap_mod-1 elements between entries so that offsets are not 16-byte aligned.
    element_aligned: every entry starts on a multiple of its item size (entries of different
    item sizes share buffers, so this does not follow from the gaps)."""
    entries: List[ShardMeta] = []
    for rep in range(replicas):
        for fqn, shape, isz in tensors:
            cuts = [_cuts(rng, n, max_parts) for n in shape]
            for idx in product(*[range(len(c) - 1) for c in cuts]):
                off = tuple(cuts[d][i] for d, i in enumerate(idx))
                ln = tuple(cuts[d][i + 1] - cuts[d][i] for d, i in enumerate(idx))
                n = prod(ln)
                if n > 1 and rng.random() < flat_prob:
                    fc = _cuts(rng, n, 3)
                    for a, b in zip(fc[:-1], fc[1:]):
                        entries.append(ShardMeta(fqn, isz, isz, shape, off, ln, kind=FLAT_SLICE,
                                                 flat_begin=a, flat_end=b))
                else:
                    entries.append(ShardMeta(fqn, isz, isz, shape, off, ln))
    order = rng.permutation(len(entries)) if shuffle else np.arange(len(entries))
    fill = [0] * n_bufs
    for i in order:
        e = entries[int(i)]
        b = int(rng.integers(0, n_bufs))
        gap = int(rng.integers(0, gap_mod)) * e.itemsize if gap_mod else 0
        start = fill[b] + gap
        if element_aligned:
            start = -(-start // e.itemsize) * e.itemsize
        e.buf_index, e.byte_offset = b, start
        fill[b] = e.byte_offset + e.byte_length
    return ShardedState(entries, [f + int(rng.integers(0, 64)) for f in fill])


def random_case(seed: int, *, n_tensors: int = 4, max_ndim: int = 3, max_dim: int = 7, gap_mod: int = 5,
                itemsizes: Sequence[int] = (1, 2, 4, 8), dst_replicas: int = 1) -> ReshardCase:
    rng = np.random.default_rng(seed)
    tensors = []
    for t in range(n_tensors):
        nd = int(rng.integers(0, max_ndim + 1))
        shape = tuple(int(rng.integers(1, max_dim + 1)) for _ in range(nd))
        tensors.append((f"t{t}.w", shape, int(rng.choice(list(itemsizes)))))
    src = random_side(rng, tensors, int(rng.integers(1, 4)), gap_mod=gap_mod)
    dst = random_side(rng, tensors, int(rng.integers(1, 4)), gap_mod=gap_mod, replicas=dst_replicas)
    return ReshardCase(f"random-{seed}", src, dst, "index", seed)


def big_random_case(seed: int, *, itemsize: int = 2, gap_mod: int = 7) -> ReshardCase:
    """Larger odd-shaped tensors (several tiles, ragged tails) with misaligned offsets."""
    rng = np.random.default_rng(seed)
    tensors = [
        ("big.a", (1000, 517), itemsize),
        ("big.b", (50257, 24), itemsize),
        ("big.c", (9, 130, 67), itemsize),
        ("big.d", (300_001,), itemsize),
        ("big.e", (4, 3, 33, 65), itemsize),
        ("big.s", (), itemsize),
    ]
    src = random_side(rng, tensors, 3, max_parts=4, gap_mod=gap_mod)
    dst = random_side(rng, tensors, 2, max_parts=3, gap_mod=gap_mod, replicas=2)
    return ReshardCase(f"big-random-{seed}-i{itemsize}", src, dst, "index", seed)


def many_tiny_case(n_tensors: int = 100_000, seed: int = 7) -> ReshardCase:
    """10^5 tiny tensors (4..512 bytes each, odd sizes), saved on 2 ranks and wanted on 3:
    stresses FQN grouping in the planner and the one-warp-per-unit path of the kernel."""
    rng = np.random.default_rng(seed)
    sizes = rng.integers(1, 129, n_tensors)
    isz = rng.choice([1, 2, 4], n_tensors)
    src, dst = ShardedState([], [0, 0]), ShardedState([], [0, 0, 0])
    for t in range(n_tensors):
        n, w = int(sizes[t]), int(isz[t])
        cut = int(rng.integers(0, n + 1))
        name = f"tiny.{t}"
        for st, parts in ((src, [(0, cut), (cut, n)]), (dst, [(0, n)])):
            for a, b in parts:
                if b > a:
                    r = int(rng.integers(0, len(st.buf_bytes)))
                    st.metas.append(ShardMeta(name, w, w, (n,), (a,), (b - a,), r, st.buf_bytes[r]))
                    st.buf_bytes[r] += (b - a) * w
    return ReshardCase(f"many-tiny-{n_tensors}", src, dst, "index", seed)


def random_convert_case(seed: int, *, narrow: bool = True, big: bool = False, dst_replicas: int = 1) -> ReshardCase:
    """Random problem in which about half of the tensors change their element type on the way
    (4-byte saved, 2-byte wanted when `narrow`, else the reverse; dtype tag = item size) and the
    rest are moved unchanged.  Fill them with bit patterns, not values: every pattern is legal."""
    rng = np.random.default_rng(seed)
    a, b = (4, 2) if narrow else (2, 4)
    if big:
        shapes = [(1000, 517), (50257, 6), (9, 130, 67), (300_001,), (4, 3, 33, 65), ()]
    else:
        shapes = [tuple(int(rng.integers(1, 8)) for _ in range(int(rng.integers(0, 4)))) for _ in range(5)]
    saved, wanted = [], []
    for t, shape in enumerate(shapes):
        if t % 2 == 0 or rng.random() < 0.3:
            saved.append((f"c{t}.w", shape, a))
            wanted.append((f"c{t}.w", shape, b))
        else:
            isz = int(rng.choice([1, 2, 4, 8]))
            saved.append((f"c{t}.w", shape, isz))
            wanted.append((f"c{t}.w", shape, isz))
    parts = 4 if big else 3
    src = random_side(rng, saved, int(rng.integers(1, 4)), max_parts=parts, gap_mod=7, element_aligned=True)
    dst = random_side(rng, wanted, int(rng.integers(1, 4)), max_parts=3, gap_mod=7, replicas=dst_replicas, element_aligned=True)
    return ReshardCase(f"random-convert-{seed}-{'narrow' if narrow else 'widen'}{'-big' if big else ''}", src, dst, "index", seed,
                       convert=(1 if narrow else 2, a, b))
