"""Plain description of one checkpoint entry, shared by every consumer of the synthetic inputs.

A `ShardMeta` carries what the paper's global metadata file records for one saved (or
wanted) tensor shard (Sec. 3.2): the FQN and global shape, the ShardMeta index tuple
(nD offsets, nD lengths), the dtype identity, and the ByteMeta (buffer, byte offset, byte
length).  An irregular shard is given as a flat element range of its enclosing local box
(`kind == FLAT_SLICE`); nothing in this module decomposes, intersects or copies anything.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

BOX = 0
FLAT_SLICE = 1


def prod(xs: Sequence[int]) -> int:
    p = 1
    for x in xs:
        p *= int(x)
    return p


@dataclass
class ShardMeta:
    fqn: str
    itemsize: int
    dtype_tag: int
    global_shape: Tuple[int, ...]
    offsets: Tuple[int, ...]
    lengths: Tuple[int, ...]
    buf_index: int = 0
    byte_offset: int = 0
    kind: int = BOX
    flat_begin: int = 0
    flat_end: int = 0

    @property
    def ndim(self) -> int:
        return len(self.global_shape)

    @property
    def numel(self) -> int:
        if self.kind == FLAT_SLICE:
            return self.flat_end - self.flat_begin
        return prod(self.lengths)

    @property
    def byte_length(self) -> int:
        return self.numel * self.itemsize


@dataclass
class ShardedState:
    """All entries of one side (saved or wanted) of a reshard problem."""

    metas: List[ShardMeta] = field(default_factory=list)
    buf_bytes: List[int] = field(default_factory=list)  # size of every rank buffer

    @property
    def total_bytes(self) -> int:
        return sum(m.byte_length for m in self.metas)


# dtype identities used by the generators (opaque to the engine)
DTYPE_BF16 = 1
DTYPE_F32 = 2
DTYPE_U8 = 3
DTYPE_I64 = 4
