"""Shared test helpers: fixture parsing, buffer conversion, brute-force element mapping."""
from __future__ import annotations

import os
from typing import List, Sequence

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_irregular_example():
    shape, recs = None, []
    with open(os.path.join(GOLDEN, "irregular_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("shape"):
                shape = tuple(int(x) for x in line.split()[1:])
                continue
            parts = [p.strip() for p in line.split("|")]
            rank = int(parts[0])
            a, b = (int(x) for x in parts[1].split())
            boxes = []
            for p in parts[2:]:
                o, l = p.split(";")
                boxes.append((tuple(int(x) for x in o.split()), tuple(int(x) for x in l.split())))
            recs.append((rank, a, b, boxes))
    return shape, recs


def np_bufs(torch_bufs) -> List[np.ndarray]:
    return [b.cpu().numpy() for b in torch_bufs]


def _coords(i: int, lengths: Sequence[int]):
    out = []
    for n in reversed(lengths):
        out.append(i % n)
        i //= n
    return tuple(reversed(out))


def _lin(c: Sequence[int], lengths: Sequence[int]) -> int:
    i = 0
    for x, n in zip(c, lengths):
        i = i * n + x
    return i


def brute_force_reshard(src_metas, src_blobs, dst_metas, dst_buf_bytes, fill_byte=0, first_wins=False):
    """Element-by-element definition, written independently of the oracle: for every element
    of every wanted entry find the one saved entry that holds its global coordinate and copy
    its bytes (first_wins: several may hold it, the first in input order supplies the bytes).
    Pure Python loops: tiny inputs only."""
    out = [np.full(int(n), fill_byte, dtype=np.uint8) for n in dst_buf_bytes]
    for d in dst_metas:
        base = d.flat_begin if d.kind == 1 else 0
        for i in range(d.numel):
            local = _coords(base + i, d.lengths)
            g = tuple(o + c for o, c in zip(d.offsets, local))
            hits = []
            for s in src_metas:
                if s.fqn != d.fqn:
                    continue
                rel = tuple(x - o for x, o in zip(g, s.offsets))
                if any(r < 0 or r >= n for r, n in zip(rel, s.lengths)):
                    continue
                pos = _lin(rel, s.lengths)
                if s.kind == 1:
                    if not (s.flat_begin <= pos < s.flat_end):
                        continue
                    pos -= s.flat_begin
                hits.append((s, pos))
            assert len(hits) == 1 or (first_wins and len(hits) > 1), (d.fqn, g, len(hits))
            s, pos = hits[0]
            sb = s.byte_offset + pos * s.itemsize
            db = d.byte_offset + i * d.itemsize
            out[d.buf_index][db:db + d.itemsize] = src_blobs[s.buf_index][sb:sb + s.itemsize]
    return out
