"""Seeded, random-access fill values for synthetic checkpoints.

Every element value is a function of (key id k of its FQN, global linear index g of the
element in C order over the tensor's global shape, fill kind, seed), so any consumer can
regenerate any element without the others:

  index    4- and 8-byte dtypes: bits = (g + salt(k)) mod 2^32 (8-byte: no modulus);
           2-byte: (g + salt(k)) mod 65521; 1-byte: (g + salt(k)) mod 251.
           A wrong byte decodes back to the global index it came from.
  uniform  value = pool[(g + salt(k)) mod P], pool = P draws of uniform[-1, 1)
  normal   value = pool[(g + salt(k)) mod P], pool = P draws of normal(0, 0.02)
           (P = 16777213, prime; fp32 bits, or bf16 bits rounded to nearest even).

This module knows how a box or a flat range of a local tensor maps to global indices only
in order to write the values; it holds no resharding logic.  It runs on any torch device.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from .meta import FLAT_SLICE, ShardMeta, ShardedState, prod

POOL = 16_777_213
_CHUNK = 1 << 26  # elements generated at a time

_pool_cache: Dict[tuple, torch.Tensor] = {}


def salt(k: int) -> int:
    return (int(k) * 1_000_003 + 12_345) % (1 << 31)


def _pool(fill: str, seed: int, itemsize: int, device) -> torch.Tensor:
    key = (fill, seed, itemsize, str(device))
    t = _pool_cache.get(key)
    if t is None:
        rng = np.random.default_rng(seed)
        if fill == "uniform":
            v = rng.uniform(-1.0, 1.0, POOL).astype(np.float32)
        elif fill == "normal":
            v = rng.normal(0.0, 0.02, POOL).astype(np.float32)
        else:
            raise ValueError(fill)
        bits = v.view(np.uint32)
        if itemsize == 4:
            t = torch.from_numpy(bits.astype(np.int64))
        elif itemsize == 2:  # bf16, round to nearest even on the fp32 bit pattern
            b = bits.astype(np.uint64)
            b = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
            t = torch.from_numpy(b.astype(np.int64))
        elif itemsize == 8:
            t = torch.from_numpy(bits.astype(np.int64) * 0x100000001 % (1 << 62))
        else:
            t = torch.from_numpy((bits >> 24).astype(np.int64))
        t = t.to(device)
        _pool_cache[key] = t
    return t


def _strides(shape: Sequence[int]) -> List[int]:
    s, out = 1, []
    for n in reversed(shape):
        out.append(s)
        s *= int(n)
    return list(reversed(out))


def global_indices(m: ShardMeta, lo: int, hi: int, device) -> torch.Tensor:
    """Global linear indices (int64) of elements [lo, hi) of the entry, in the entry's byte order."""
    gs = _strides(m.global_shape)
    base = (m.flat_begin if m.kind == FLAT_SLICE else 0)
    idx = torch.arange(base + lo, base + hi, dtype=torch.int64, device=device)
    g = torch.zeros_like(idx)
    ls = _strides(m.lengths)
    for d in range(len(m.lengths)):
        c = idx // ls[d] if d == 0 else (idx // ls[d]) % int(m.lengths[d])
        g += (c + int(m.offsets[d])) * gs[d]
    return g


def values_for(g: torch.Tensor, k: int, itemsize: int, fill: str, seed: int) -> torch.Tensor:
    """Fill bits (int64, low `itemsize` bytes significant) of the elements with global indices g."""
    x = g + salt(k)
    if fill == "index":
        if itemsize == 4:
            return x % (1 << 32)
        if itemsize == 2:
            return x % 65521
        if itemsize == 1:
            return x % 251
        return x
    return _pool(fill, seed, itemsize, g.device)[x % POOL]


_INT = {1: torch.uint8, 2: torch.int16, 4: torch.int32, 8: torch.int64}


def _to_bytes(bits: torch.Tensor, itemsize: int) -> torch.Tensor:
    if itemsize == 1:
        return bits.to(torch.uint8)
    if itemsize == 2:
        bits = torch.where(bits >= (1 << 15), bits - (1 << 16), bits)
    elif itemsize == 4:
        bits = torch.where(bits >= (1 << 31), bits - (1 << 32), bits)
    return bits.to(_INT[itemsize]).view(torch.uint8)


def entry_bytes(m: ShardMeta, k: int, fill: str, seed: int, device, lo: int = 0,
                hi: Optional[int] = None) -> torch.Tensor:
    """uint8 tensor: the bytes of elements [lo, hi) of entry m under the given fill."""
    hi = m.numel if hi is None else hi
    g = global_indices(m, lo, hi, device)
    return _to_bytes(values_for(g, k, m.itemsize, fill, seed), m.itemsize)


def write_entry(buf: torch.Tensor, m: ShardMeta, k: int, fill: str, seed: int) -> None:
    n = m.numel
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        b = m.byte_offset + lo * m.itemsize
        buf[b:b + (hi - lo) * m.itemsize] = entry_bytes(m, k, fill, seed, buf.device, lo, hi)


def make_buffers(state: ShardedState, device, poison: int = 0) -> List[torch.Tensor]:
    return [torch.full((n,), poison, dtype=torch.uint8, device=device) for n in state.buf_bytes]


def fill_state(state: ShardedState, key_ids: Dict[str, int], fill: str, seed: int, device,
               poison: int = 0) -> List[torch.Tensor]:
    """Rank buffers of `state` with every entry written under the fill; other bytes = poison."""
    bufs = make_buffers(state, device, poison)
    for m in state.metas:
        write_entry(bufs[m.buf_index], m, key_ids[m.fqn], fill, seed)
    return bufs
