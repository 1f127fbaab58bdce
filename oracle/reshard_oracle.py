"""CPU oracle for load-time checkpoint resharding and save-blob packing.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition the CUDA library is
checked against; it shares no code with the library and must never be imported by the
product path (only by tests/, the smoke check and the CPU-baseline leg of the benchmark).

What it computes follows the paper's representation (arXiv 2407.20143):
  * a tensor is named by its FQN and has a global shape; a shard is the box
    (nD_offsets, nD_lengths) of that shape (Sec. 3.2, "Model and optimizer states");
  * a ByteMeta locates the shard's bytes in a storage file (Sec. 3.2, "Checkpoint
    representation"); bytes are the shard's elements densely in C order;
  * an irregular shard is a contiguous range of the C-order flattening of a rank's local
    tensor (Sec. 3.2, "Decomposing irregular tensors");
  * loading under a new parallelism gives every new shard the elements of the saved
    shards that fall into it (Sec. 3.3, Step 2 and Step 5).
The method reaches exactly the result with a plain definition, so the oracle is that
definition: per FQN, ASSEMBLE the full global tensor from the saved shards by slice
assignment, then SLICE it once per wanted shard.  Irregular shards go through `ravel()` of
their local box; the oracle never decomposes them into boxes.  Everything is moved as
unsigned integers of the element size, never as floats.

Entries are duck-typed objects with the attributes fqn, itemsize, dtype_tag, global_shape,
offsets, lengths, kind (0 box, 1 flat slice), flat_begin, flat_end, buf_index, byte_offset,
byte_length.

Element conversion while resharding (binary32 <-> bfloat16) is not in the paper, which moves
bytes only; it is an extension of the library, and the oracle states it from the definition
of rounding (`f32_to_bf16`: search the two neighbouring bfloat16 values, pick the nearer,
the even one on a tie), not from a bit trick.

Pins (tests/test_oracle_pins.py): the paper's worked example of an irregular shard, the
identity / round-trip / exact-cover invariants, textbook reductions to numpy concatenate
and split, a brute-force per-element index map on tiny inputs (also with replicated saved
shards, where the first holder in input order supplies the bytes), and the closed-form
index-pattern fill; for the conversions, hand-worked bit patterns (tests/golden/
f32_to_bf16_examples.txt), torch's own cast on everything but NaN, and the half-ulp error
bound.  No function here is "parity unpinned".
"""
from __future__ import annotations

from collections import defaultdict
from typing import Dict, Iterable, List, Sequence, Tuple

import numpy as np

_UINT = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}
FLAT_SLICE = 1
F32_TO_BF16, BF16_TO_F32 = 1, 2  # conversion kinds


class OracleError(ValueError):
    pass


def _box(e) -> Tuple[slice, ...]:
    return tuple(slice(int(o), int(o) + int(l)) for o, l in zip(e.offsets, e.lengths))


def _payload(blob: np.ndarray, e) -> np.ndarray:
    """The entry's bytes, viewed as a 1-D array of unsigned integers of the element size."""
    raw = blob[e.byte_offset:e.byte_offset + e.byte_length]
    if raw.size != e.byte_length:
        raise OracleError(f"{e.fqn}: byte range outside its buffer")
    return np.ascontiguousarray(raw).view(_UINT[e.itemsize])


def f32_to_bf16(bits: np.ndarray) -> np.ndarray:
    """binary32 bit patterns (uint32) -> bfloat16 bit patterns (uint16), round to nearest, ties
    to even.  A bfloat16 is a binary32 whose low 16 bits are zero, and for non-negative floats
    the order of bit patterns is the order of values, so the two candidates for |x| are the
    pattern with its low half cleared (`below`) and the next bfloat16 pattern (`above`; past
    the largest finite one it stands for 2^128, as IEEE 754 rounding prescribes before
    overflow turns it into infinity).  Distances are taken in float64, where they are exact.
    NaN (any payload, either sign) -> 0x7FC0."""
    bits = np.asarray(bits, dtype=np.uint32)
    sign = bits & np.uint32(0x80000000)
    mag = bits & np.uint32(0x7FFFFFFF)
    nan = mag > np.uint32(0x7F800000)
    below = mag & np.uint32(0xFFFF0000)
    above = (below.astype(np.uint64) + 0x10000).astype(np.uint32)  # at most 0x7F800000 for finite input
    value = lambda pattern: pattern.view(np.float32).astype(np.float64)  # noqa: E731
    with np.errstate(invalid="ignore", over="ignore"):
        x = value(mag)
        v_above = np.where(above == np.uint32(0x7F800000), 2.0 ** 128, value(above))
        d_below, d_above = x - value(below), v_above - x
        below_is_odd = ((below >> np.uint32(16)) & np.uint32(1)) == 1
        up = (d_above < d_below) | ((d_above == d_below) & below_is_odd)
    up &= mag < np.uint32(0x7F800000)  # infinity stays
    out = np.where(up, above, below) | sign
    out = np.where(nan, np.uint32(0x7FC00000), out)
    return (out >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> binary32 bit patterns (uint32): a bfloat16 IS the upper
    half of a binary32, so the value is unchanged when 16 zero bits are appended."""
    return np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)


def check_family(entries: Sequence) -> Tuple[Tuple[int, ...], int]:
    """All entries of one FQN must agree on global shape and dtype (Sec. 3.2)."""
    e0 = entries[0]
    for e in entries:
        if (tuple(e.global_shape) != tuple(e0.global_shape) or e.itemsize != e0.itemsize
                or e.dtype_tag != e0.dtype_tag):
            raise OracleError(f"{e.fqn}: entries disagree on global shape or dtype")
        for o, l, g in zip(e.offsets, e.lengths, e.global_shape):
            if o < 0 or l < 0 or o + l > g:
                raise OracleError(f"{e.fqn}: box outside the global shape")
    return tuple(int(g) for g in e0.global_shape), int(e0.itemsize)


def _held(global_shape: Sequence[int], e) -> np.ndarray:
    """Which elements of the global tensor the entry holds (boolean array of the global shape)."""
    m = np.zeros(tuple(global_shape), dtype=bool)
    b = _box(e)
    if e.kind == FLAT_SLICE:
        flat = m[b].ravel()
        flat[int(e.flat_begin):int(e.flat_end)] = True
        m[b] = flat.reshape(m[b].shape)
    else:
        m[b] = True
    return m


def assemble(global_shape: Sequence[int], itemsize: int, entries: Sequence, payloads: Sequence[np.ndarray],
             first_wins: bool = False):
    """Full global tensor from saved shards, plus how many shards supplied each element.

    Sec. 3.2: shard i covers the box offsets_i + lengths_i of the global shape; an irregular
    shard covers elements [flat_begin, flat_end) of the flattened local box.
    first_wins: replicated shards are allowed and the earliest entry supplies the value
    (entries are assigned last to first, so the first one overwrites the rest).  Replicas are
    whole shards stored more than once: two entries that share an element must hold exactly the
    same elements; entries that overlap only partly are an error, with or without first_wins.
    """
    T = np.zeros(tuple(global_shape), dtype=_UINT[itemsize])
    cover = np.zeros(tuple(global_shape), dtype=np.uint8)
    pairs = list(zip(entries, payloads))
    if first_wins:
        held = [_held(global_shape, e) for e in entries]
        for i in range(len(held)):
            for j in range(i):
                if (held[i] & held[j]).any() and not np.array_equal(held[i], held[j]):
                    raise OracleError(f"{entries[i].fqn}: two saved shards overlap only partly")
    for e, data in (reversed(pairs) if first_wins else pairs):
        b = _box(e)
        if e.kind == FLAT_SLICE:
            a, z = int(e.flat_begin), int(e.flat_end)
            # values: flatten the local box, overwrite [a, z), put the box back
            tmp = T[b].ravel()
            tmp[a:z] = data
            T[b] = tmp.reshape(T[b].shape)
            # the same for the coverage count
            cnt = cover[b].ravel()
            cnt[a:z] += 1
            cover[b] = cnt.reshape(cover[b].shape)
        else:
            T[b] = data.reshape(tuple(int(l) for l in e.lengths))
            cover[b] += 1
    return T, cover


def take(T: np.ndarray, cover: np.ndarray, e, replicas_ok: bool = False) -> np.ndarray:
    """Bytes of the wanted shard e cut out of the assembled tensor (uint8, C order)."""
    b = _box(e)
    if e.kind == FLAT_SLICE:
        a, z = int(e.flat_begin), int(e.flat_end)
        vals, cov = T[b].ravel()[a:z], cover[b].ravel()[a:z]
    else:
        vals, cov = T[b].ravel(), cover[b].ravel()
    if cov.size and cov.min() < 1:
        raise OracleError(f"{e.fqn}: wanted element held by no saved shard")
    if cov.size and cov.max() > 1 and not replicas_ok:
        raise OracleError(f"{e.fqn}: element held by more than one saved shard")
    return np.ascontiguousarray(vals).view(np.uint8)


def group_by_fqn(entries: Iterable) -> Dict[str, List]:
    g: Dict[str, List] = defaultdict(list)
    for e in entries:
        g[e.fqn].append(e)
    return g


def reshard_fqn(src_entries: Sequence, src_payloads: Sequence[np.ndarray], dst_entries: Sequence,
                allow_replicas: bool = False, convert=None) -> List[np.ndarray]:
    """Bytes of every wanted shard of ONE FQN, given the payloads of its saved shards.
    convert = (kind, saved dtype_tag, wanted dtype_tag): a tensor saved with the first tag and
    wanted with the second is converted element by element after it has been assembled."""
    s0, d0 = src_entries[0], dst_entries[0]
    if (s0.itemsize, s0.dtype_tag) == (d0.itemsize, d0.dtype_tag):
        shape, itemsize = check_family(list(src_entries) + list(dst_entries))
        T, cover = assemble(shape, itemsize, src_entries, src_payloads, first_wins=allow_replicas)
        return [take(T, cover, d, replicas_ok=allow_replicas) for d in dst_entries]
    sizes = {F32_TO_BF16: (4, 2), BF16_TO_F32: (2, 4)}
    if (convert is None or (s0.dtype_tag, d0.dtype_tag) != tuple(convert[1:])
            or (s0.itemsize, d0.itemsize) != sizes[convert[0]]):
        raise OracleError(f"{s0.fqn}: saved and wanted entries disagree on dtype")
    shape, itemsize = check_family(list(src_entries))
    if check_family(list(dst_entries))[0] != shape:
        raise OracleError(f"{s0.fqn}: entries disagree on global shape or dtype")
    T, cover = assemble(shape, itemsize, src_entries, src_payloads, first_wins=allow_replicas)
    T = f32_to_bf16(T) if convert[0] == F32_TO_BF16 else bf16_to_f32(T)
    return [take(T, cover, d, replicas_ok=allow_replicas) for d in dst_entries]


def reshard(src_metas: Sequence, src_blobs: Sequence[np.ndarray], dst_metas: Sequence,
            dst_buf_bytes: Sequence[int], fill_byte: int = 0, allow_replicas: bool = False,
            convert=None) -> List[np.ndarray]:
    """Every target rank buffer (uint8 arrays); bytes no entry names keep `fill_byte`.
    allow_replicas: saved shards may be stored more than once (a checkpoint written without
    de-duplication); the first entry in input order supplies the bytes."""
    out = [np.full(int(n), fill_byte, dtype=np.uint8) for n in dst_buf_bytes]
    src_by, dst_by = group_by_fqn(src_metas), group_by_fqn(dst_metas)
    for fqn, dsts in dst_by.items():
        srcs = src_by.get(fqn, [])
        if not srcs:
            if all(d.byte_length == 0 for d in dsts):
                continue
            raise OracleError(f"{fqn}: wanted but never saved")
        payloads = [_payload(src_blobs[s.buf_index], s) for s in srcs]
        for d, data in zip(dsts, reshard_fqn(srcs, payloads, dsts, allow_replicas, convert)):
            buf = out[d.buf_index]
            if d.byte_offset + d.byte_length > buf.size:
                raise OracleError(f"{fqn}: target byte range outside its buffer")
            buf[d.byte_offset:d.byte_offset + d.byte_length] = data
    return out


# --------------------------------------------------------------------------- pack / unpack
def pack_layout(sizes: Sequence[int], align: int = 256) -> Tuple[List[int], int]:
    """ByteMeta table of a save blob (Sec. 3.2): tensor i starts at the end of tensor i-1
    rounded up to `align`; the blob ends at the last end rounded up."""
    offs, pos = [], 0
    for n in sizes:
        pos = -(-pos // align) * align
        offs.append(pos)
        pos += int(n)
    return offs, -(-pos // align) * align


def pack(tensors: Sequence[np.ndarray], align: int = 256):
    """One contiguous blob: tensor bytes at the table's offsets, zero bytes elsewhere."""
    raws = [np.ascontiguousarray(t).reshape(-1).view(np.uint8) for t in tensors]
    offs, total = pack_layout([r.size for r in raws], align)
    blob = np.zeros(total, dtype=np.uint8)
    for r, o in zip(raws, offs):
        blob[o:o + r.size] = r
    return blob, [(o, r.size) for r, o in zip(raws, offs)]


def unpack(blob: np.ndarray, table: Sequence[Tuple[int, int]]) -> List[np.ndarray]:
    return [blob[o:o + n].copy() for (o, n) in table]


# --------------------------------------------------------------------------- save-side de-duplication
def worst_fit(shard_bytes: Sequence[int], holders: Sequence[Sequence[int]], n_ranks: int, initial_load=None):
    """Owner of every shard (Sec. 4.1, "Balancing saving workload"): walk the shards in order
    and give each to the holder with the smallest cumulative size so far (lowest rank on ties).
    The paper states the procedure, so this follows its steps; pinned by a hand-worked example
    and by the list-scheduling bound (tests/test_dedup.py)."""
    load = list(initial_load) if initial_load is not None else [0] * n_ranks
    owners = []
    for size, hs in zip(shard_bytes, holders):
        if not hs:
            raise OracleError("a shard needs at least one holder")
        smallest = min(load[r] for r in hs)
        owner = min(r for r in hs if load[r] == smallest)
        load[owner] += int(size)
        owners.append(owner)
    return owners, load
