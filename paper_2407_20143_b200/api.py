"""Python binding of the C ABI in include/bcp.h: same names, argument marshalling only.

Every step of the resharding path (decomposition, matching, lowering, the copies) runs
inside libbcp.so; this module converts Python metadata objects to C structures and torch
tensors to device pointers.
"""
from __future__ import annotations

import ctypes as C
import struct
from typing import List, Optional, Sequence, Tuple

from . import _lib as L


class BcpError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"bcp error {code}: {msg}")
        self.code = code


ERR_INVALID, ERR_MISMATCH, ERR_OVERLAP, ERR_UNCOVERED, ERR_BOUNDS, ERR_DST_ALIAS = -1, -2, -3, -4, -5, -6
ERR_CUDA, ERR_NOMEM, ERR_DEVICE_TIMEOUT, ERR_CAPACITY = -7, -8, -9, -10
TILE_GRAN_MASK, TILE_ZERO, TILE_SMALL, TILE_TMA, TILE_TMA2D, TILE_FOLLOW = 0x7, 0x8, 0x10, 0x20, 0x40, 0x80
TILE_CVT_SHIFT, TILE_CVT_MASK = 11, 3 << 11
CONVERT_NONE, CONVERT_F32_TO_BF16, CONVERT_BF16_TO_F32 = 0, 1, 2


def _check(rc: int) -> None:
    if rc != 0:
        raise BcpError(rc, L.lib().bcp_last_error().decode("utf-8", "replace"))


_META_FMT = struct.Struct("<Q4I%dq2q2I2Q" % (3 * L.BCP_MAX_NDIM))  # field for field bcp_shard_meta (little endian, no padding needed)
_PAD = [(0,) * k for k in range(L.BCP_MAX_NDIM + 1)]


def _metas_to_c_loop(metas: Sequence) -> Tuple[C.Array, list]:
    arr = (L.ShardMetaC * max(1, len(metas)))()
    keep = []
    for c, m in zip(arr, metas):
        name = m.fqn.encode()
        keep.append(name)
        c.fqn = name
        c.itemsize, c.dtype_tag, c.ndim, c.kind = m.itemsize, m.dtype_tag, len(m.global_shape), m.kind
        for k, (g, o, l) in enumerate(zip(m.global_shape, m.offsets, m.lengths)):
            c.global_shape[k], c.offsets[k], c.lengths[k] = g, o, l
        c.flat_begin, c.flat_end = m.flat_begin, m.flat_end
        c.buf_index, c.byte_offset, c.byte_length = m.buf_index, m.byte_offset, m.byte_length
    return arr, keep


def _metas_to_c(metas: Sequence) -> Tuple[C.Array, list]:
    """Objects with the attributes of workloads.meta.ShardMeta -> array of bcp_shard_meta (plus what
    must stay alive with it).  Records are packed whole, names go into one NUL-separated buffer;
    anything irregular (values a C field cannot hold, ragged shapes, NUL inside a name) goes
    through the field-by-field loop, which passes it on for the library to judge."""
    n = len(metas)
    if _META_FMT.size != C.sizeof(L.ShardMetaC) or n == 0:
        return _metas_to_c_loop(metas)
    try:
        names = [m.fqn.encode() for m in metas]
        blob = b"\0".join(names) + b"\0"
        if blob.count(b"\0") != n:
            return _metas_to_c_loop(metas)
        text = C.create_string_buffer(blob, len(blob))
        at = C.addressof(text)
        arr = (L.ShardMetaC * n)()
        raw = (C.c_char * (n * _META_FMT.size)).from_buffer(arr)
        pack, size, pad = _META_FMT.pack_into, _META_FMT.size, _PAD
        for i, m in enumerate(metas):
            g = m.global_shape
            k = L.BCP_MAX_NDIM - len(g)
            if len(m.offsets) != len(g) or len(m.lengths) != len(g):
                return _metas_to_c_loop(metas)
            pack(raw, i * size, at, m.itemsize, m.dtype_tag, len(g), m.kind, *g, *pad[k], *m.offsets, *pad[k], *m.lengths, *pad[k],
                 m.flat_begin, m.flat_end, m.buf_index, 0, m.byte_offset, m.byte_length)
            at += len(names[i]) + 1
        return arr, [text]
    except (struct.error, IndexError, TypeError, OverflowError):
        return _metas_to_c_loop(metas)


def _u64(xs: Sequence[int]) -> C.Array:
    return (C.c_uint64 * max(1, len(xs)))(*xs)


def _ptrs(tensors: Sequence) -> C.Array:
    return (C.c_void_p * max(1, len(tensors)))(*[t if isinstance(t, int) else t.data_ptr() for t in tensors])


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


class Plan:
    """Owner of a bcp_plan_t handle."""

    def __init__(self, handle: int, n_src_bufs: int, n_dst_bufs: int):
        self._h = C.c_void_p(handle)
        self.n_src_bufs, self.n_dst_bufs = n_src_bufs, n_dst_bufs

    @property
    def handle(self) -> C.c_void_p:
        if not self._h:
            raise BcpError(ERR_INVALID, "plan already destroyed")
        return self._h

    def stats(self) -> dict:
        st = L.PlanStatsC()
        _check(L.lib().bcp_plan_stats(self.handle, C.byref(st)))
        return {n: getattr(st, n) for n, _ in L.PlanStatsC._fields_}

    def used_sources(self) -> List[int]:
        """Indices (into the saved metas given to bcp_plan) of the entries the plan reads, ascending."""
        n = C.c_size_t()
        _check(L.lib().bcp_plan_used_sources(self.handle, None, 0, C.byref(n)))
        arr = (C.c_uint32 * max(1, n.value))()
        _check(L.lib().bcp_plan_used_sources(self.handle, arr, n.value, C.byref(n)))
        return list(arr[: n.value])

    def tiles(self) -> List[L.TileC]:
        n = C.c_size_t()
        _check(L.lib().bcp_plan_tiles(self.handle, None, 0, C.byref(n)))
        arr = (L.TileC * max(1, n.value))()
        _check(L.lib().bcp_plan_tiles(self.handle, arr, n.value, C.byref(n)))
        return list(arr[: n.value])

    def tiles_array(self):
        """The same records as one numpy structured array (fields as in bcp_tile), for long lists."""
        import numpy as np

        n = C.c_size_t()
        _check(L.lib().bcp_plan_tiles(self.handle, None, 0, C.byref(n)))
        arr = (L.TileC * max(1, n.value))()
        _check(L.lib().bcp_plan_tiles(self.handle, arr, n.value, C.byref(n)))
        dt = np.dtype([("src_off", "<u8"), ("dst_off", "<u8"), ("src_pitch", "<u8"), ("dst_pitch", "<u8"), ("row_bytes", "<u4"),
                       ("rows", "<u4"), ("src_buf", "<u4"), ("dst_buf", "<u4"), ("flags", "<u4"), ("reserved", "<u4", (3,))])
        assert dt.itemsize == C.sizeof(L.TileC)
        return np.frombuffer(arr, dtype=dt, count=n.value)

    def serialize(self) -> bytes:
        """Self-contained image of the plan (bcp_plan_serialize) for reuse in another process."""
        n = C.c_size_t()
        L.lib().bcp_plan_serialize(self.handle, None, 0, C.byref(n))
        buf = (C.c_uint8 * max(1, n.value))()
        _check(L.lib().bcp_plan_serialize(self.handle, buf, n.value, C.byref(n)))
        return bytes(buf[: n.value])

    @staticmethod
    def deserialize(image: bytes) -> "Plan":
        h = C.c_void_p()
        buf = (C.c_uint8 * max(1, len(image))).from_buffer_copy(image) if image else (C.c_uint8 * 1)()
        _check(L.lib().bcp_plan_deserialize(buf, len(image), C.byref(h)))
        p = Plan(h.value, 0, 0)
        return p

    def destroy(self) -> None:
        if self._h:
            h, self._h = self._h, C.c_void_p(None)
            _check(L.lib().bcp_plan_destroy(h))

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def bcp_version() -> int:
    return L.lib().bcp_version()


def bcp_decompose(lengths: Sequence[int], flat_begin: int, flat_end: int):
    """Regular boxes (offsets, lengths), relative to the local tensor, that tile a flat range."""
    nd = len(lengths)
    cap = max(1, 2 * nd)
    off = ((C.c_int64 * L.BCP_MAX_NDIM) * cap)()
    ln = ((C.c_int64 * L.BCP_MAX_NDIM) * cap)()
    n = C.c_size_t()
    la = (C.c_int64 * max(1, nd))(*lengths)
    _check(L.lib().bcp_decompose(la, nd, flat_begin, flat_end, off, ln, cap, C.byref(n)))
    return [(tuple(off[i][:nd]), tuple(ln[i][:nd])) for i in range(n.value)]


def bcp_dedup_assign(shard_bytes: Sequence[int], holders: Sequence[Sequence[int]], n_ranks: int,
                     initial_load: Optional[Sequence[int]] = None) -> Tuple[List[int], List[int]]:
    """Worst-fit owner of every replicated shard; returns (owners, final per-rank loads)."""
    n = len(shard_bytes)
    offs, flat = [0], []
    for h in holders:
        flat.extend(h)
        offs.append(len(flat))
    load = (C.c_uint64 * max(1, n_ranks))(*(initial_load if initial_load is not None else [0] * n_ranks))
    owner = (C.c_uint32 * max(1, n))()
    _check(L.lib().bcp_dedup_assign(_u64(shard_bytes), _u64(offs), (C.c_uint32 * max(1, len(flat)))(*flat), n, n_ranks,
                                    load, owner))
    return list(owner[:n]), list(load[:n_ranks])


def bcp_plan(src_metas: Sequence, src_buf_bytes: Sequence[int], dst_metas: Sequence, dst_buf_bytes: Sequence[int],
             **opts) -> Plan:
    """Match wanted against saved entries and build the work list (host only)."""
    sa, keep_s = _metas_to_c(src_metas)
    da, keep_d = _metas_to_c(dst_metas)
    o = None
    if opts:
        o = L.PlanOptsC()
        for k, v in opts.items():
            if not hasattr(o, k):
                raise BcpError(ERR_INVALID, f"unknown plan option {k}")
            setattr(o, k, v)
    h = C.c_void_p()
    _check(L.lib().bcp_plan(sa, len(src_metas), _u64(src_buf_bytes), len(src_buf_bytes), da, len(dst_metas),
                            _u64(dst_buf_bytes), len(dst_buf_bytes), C.byref(o) if o is not None else None,
                            C.byref(h)))
    del keep_s, keep_d
    return Plan(h.value, len(src_buf_bytes), len(dst_buf_bytes))


def bcp_reshard(plan: Plan, src_blobs: Sequence, dst_bufs: Sequence, stream=None) -> None:
    """Enqueue the copies of `plan` on `stream` (torch stream, raw handle, or None = current).
    src_blobs / dst_bufs: torch CUDA tensors or raw device addresses."""
    _check(L.lib().bcp_reshard(plan.handle, _ptrs(src_blobs), len(src_blobs), _ptrs(dst_bufs), len(dst_bufs),
                               _stream(stream)))


def bcp_reshard_host(plan: Plan, src_blobs: Sequence, dst_bufs: Sequence, stream=None) -> None:
    """Same with host tensors (pinned for full speed); returns when the targets are filled."""
    _check(L.lib().bcp_reshard_host(plan.handle, _ptrs(src_blobs), len(src_blobs), _ptrs(dst_bufs), len(dst_bufs),
                                    _stream(stream)))


def bcp_plan_device_status(plan: Plan, stream=None) -> None:
    _check(L.lib().bcp_plan_device_status(plan.handle, _stream(stream)))


def bcp_pack_layout(tensor_bytes: Sequence[int], align: int = 256) -> Tuple[List[int], int]:
    n = len(tensor_bytes)
    offs = (C.c_uint64 * max(1, n))()
    total = C.c_uint64()
    _check(L.lib().bcp_pack_layout(_u64(tensor_bytes), n, align, offs, C.byref(total)))
    return list(offs[:n]), total.value


def _pack_metas(metas: Sequence[Tuple[int, int]]) -> C.Array:
    arr = (L.PackMetaC * max(1, len(metas)))()
    for c, (o, n) in zip(arr, metas):
        c.byte_offset, c.byte_length = o, n
    return arr


def bcp_pack(tensors: Sequence, metas: Sequence[Tuple[int, int]], blob, blob_bytes: Optional[int] = None,
             stream=None) -> None:
    """tensors[i] -> blob[metas[i] = (byte_offset, byte_length)]; padding bytes become zero."""
    nb = blob_bytes if blob_bytes is not None else blob.numel() * blob.element_size()
    bp = blob if isinstance(blob, int) else blob.data_ptr()
    _check(L.lib().bcp_pack(_ptrs(tensors), _pack_metas(metas), len(tensors), bp, nb, _stream(stream)))


def bcp_ipc_export(tensor) -> bytes:
    """Handle (96 plain bytes) under which another process can map the device memory `tensor` starts at."""
    h = L.IpcHandleC()
    _check(L.lib().bcp_ipc_export(tensor if isinstance(tensor, int) else tensor.data_ptr(), C.byref(h)))
    return bytes(h)


def bcp_ipc_open(handle: bytes) -> int:
    """Address, in this process and on the current device, of memory another process exported."""
    h = L.IpcHandleC.from_buffer_copy(handle)
    p = C.c_void_p()
    _check(L.lib().bcp_ipc_open(C.byref(h), C.byref(p)))
    return p.value


def bcp_ipc_close(ptr: int) -> None:
    _check(L.lib().bcp_ipc_close(ptr))


def marshal_pack(tensors: Sequence, metas: Sequence[Tuple[int, int]]):
    """The C arrays of a pack call, for callers that repeat one pack many times (see bcp_pack_marshalled)."""
    return _ptrs(tensors), _pack_metas(metas), len(tensors)


def bcp_pack_marshalled(args, blob, blob_bytes: Optional[int] = None, stream=None) -> None:
    """bcp_pack with arrays prepared by marshal_pack (same call, no per-call marshalling)."""
    ptrs, metas, n = args
    nb = blob_bytes if blob_bytes is not None else blob.numel() * blob.element_size()
    bp = blob if isinstance(blob, int) else blob.data_ptr()
    _check(L.lib().bcp_pack(ptrs, metas, n, bp, nb, _stream(stream)))


def bcp_pack_static(tensors: Sequence, metas: Sequence[Tuple[int, int]], blob, blob_bytes: Optional[int] = None,
                    stream=None) -> None:
    """bcp_pack without any allocation: the work list lives in a fixed device array inside the
    library (at most 4096 tensors per call).  For hosts that own all device memory themselves or
    call from a place where allocating is not allowed.  Calls must not overlap on the GPU; make
    the first call on a device before any stream capture."""
    nb = blob_bytes if blob_bytes is not None else blob.numel() * blob.element_size()
    bp = blob if isinstance(blob, int) else blob.data_ptr()
    _check(L.lib().bcp_pack_static(_ptrs(tensors), _pack_metas(metas), len(tensors), bp, nb, _stream(stream)))


def bcp_unpack(blob, metas: Sequence[Tuple[int, int]], tensors: Sequence, blob_bytes: Optional[int] = None,
               stream=None) -> None:
    nb = blob_bytes if blob_bytes is not None else blob.numel() * blob.element_size()
    bp = blob if isinstance(blob, int) else blob.data_ptr()
    _check(L.lib().bcp_unpack(bp, nb, _pack_metas(metas), len(tensors), _ptrs(tensors), _stream(stream)))


def _export_entries(entries: Sequence[Tuple[str, str, Sequence[int]]]):
    arr = (L.ExportEntryC * max(1, len(entries)))()
    keep = []
    for c, (name, dtype, shape) in zip(arr, entries):
        nb, db = name.encode(), dtype.encode()
        keep += [nb, db]
        c.name, c.dtype, c.ndim = nb, db, len(shape)
        for k, x in enumerate(shape):
            c.shape[k] = x
    return arr, keep


def bcp_safetensors_layout(entries: Sequence[Tuple[str, str, Sequence[int]]]) -> Tuple[bytes, List[Tuple[int, int]], int]:
    """(header bytes, per-tensor (offset, length) inside the image, image size) for tensors given
    as (name, safetensors dtype string, shape)."""
    arr, keep = _export_entries(entries)
    n = len(entries)
    hb, fb = C.c_size_t(), C.c_uint64()
    metas = (L.PackMetaC * max(1, n))()
    L.lib().bcp_safetensors_layout(arr, n, None, 0, C.byref(hb), metas, C.byref(fb))
    buf = (C.c_uint8 * max(1, hb.value))()
    _check(L.lib().bcp_safetensors_layout(arr, n, buf, hb.value, C.byref(hb), metas, C.byref(fb)))
    del keep
    return bytes(buf[: hb.value]), [(m.byte_offset, m.byte_length) for m in metas[:n]], fb.value


def bcp_safetensors_export(entries: Sequence[Tuple[str, str, Sequence[int]]], tensors: Sequence, file, file_cap: Optional[int] = None,
                           stream=None) -> int:
    """Build a Safetensors image of `tensors` in the device buffer `file`; returns its size in bytes."""
    arr, keep = _export_entries(entries)
    cap = file_cap if file_cap is not None else file.numel() * file.element_size()
    fp = file if isinstance(file, int) else file.data_ptr()
    fb = C.c_uint64()
    _check(L.lib().bcp_safetensors_export(arr, _ptrs(tensors), len(entries), fp, cap, C.byref(fb), _stream(stream)))
    del keep
    return fb.value


class Stager:
    """Pinned ping-pong pool for asynchronous save / load staging (bcp_stager_* calls)."""

    def __init__(self, slot_bytes: int, n_slots: int = 2):
        h = C.c_void_p()
        _check(L.lib().bcp_stager_create(slot_bytes, n_slots, C.byref(h)))
        self._h, self.slot_bytes, self.n_slots = h, slot_bytes, n_slots

    def save(self, tensors: Sequence, metas: Sequence[Tuple[int, int]], blob_bytes: int, stream=None) -> int:
        slot = C.c_uint32()
        _check(L.lib().bcp_stager_save(self._h, _ptrs(tensors), _pack_metas(metas), len(tensors), blob_bytes,
                                       _stream(stream), C.byref(slot)))
        return slot.value

    def wait(self, slot: int) -> int:
        """Blocks until the slot's blob is in pinned host memory; returns its host address."""
        p = C.c_void_p()
        _check(L.lib().bcp_stager_wait(self._h, slot, C.byref(p)))
        return p.value

    def acquire(self) -> Tuple[int, int]:
        """(slot, host address of its pinned buffer) for the caller to fill before load()."""
        slot, p = C.c_uint32(), C.c_void_p()
        _check(L.lib().bcp_stager_acquire(self._h, C.byref(slot), C.byref(p)))
        return slot.value, p.value

    def load(self, slot: int, blob_bytes: int, metas: Sequence[Tuple[int, int]], tensors: Sequence, stream=None) -> None:
        _check(L.lib().bcp_stager_load(self._h, slot, blob_bytes, _pack_metas(metas), len(tensors), _ptrs(tensors),
                                       _stream(stream)))

    def release(self, slot: int) -> None:
        _check(L.lib().bcp_stager_release(self._h, slot))

    def host_view(self, address: int, nbytes: int):
        """numpy uint8 view of a pinned slot (no copy)."""
        import numpy as np

        return np.ctypeslib.as_array((C.c_uint8 * nbytes).from_address(address))

    def destroy(self) -> None:
        if self._h:
            h, self._h = self._h, C.c_void_p(None)
            _check(L.lib().bcp_stager_destroy(h))

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def bcp_pack_cache_clear() -> None:
    _check(L.lib().bcp_pack_cache_clear())
