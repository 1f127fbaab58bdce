"""ctypes view of libbcp.so: structures and prototypes of include/bcp.h, nothing else."""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

BCP_MAX_NDIM = 8


class ShardMetaC(C.Structure):
    _fields_ = [
        ("fqn", C.c_char_p),
        ("itemsize", C.c_uint32),
        ("dtype_tag", C.c_uint32),
        ("ndim", C.c_uint32),
        ("kind", C.c_uint32),
        ("global_shape", C.c_int64 * BCP_MAX_NDIM),
        ("offsets", C.c_int64 * BCP_MAX_NDIM),
        ("lengths", C.c_int64 * BCP_MAX_NDIM),
        ("flat_begin", C.c_int64),
        ("flat_end", C.c_int64),
        ("buf_index", C.c_uint32),
        ("reserved", C.c_uint32),
        ("byte_offset", C.c_uint64),
        ("byte_length", C.c_uint64),
    ]


class PlanOptsC(C.Structure):
    _fields_ = [
        ("tile_bytes", C.c_uint32),
        ("small_bytes", C.c_uint32),
        ("block_threads", C.c_uint32),
        ("ctas_per_sm", C.c_uint32),
        ("order", C.c_uint32),
        ("path_mask", C.c_uint32),
        ("cache_hints", C.c_uint32),
        ("tma_stage_bytes", C.c_uint32),
        ("tma_stages", C.c_uint32),
        ("tma_ctas_per_sm", C.c_uint32),
        ("unroll", C.c_uint32),
        ("worker", C.c_uint32),
        ("tma_min_row_bytes", C.c_uint32),
        ("allow_replicas", C.c_uint32),
        ("tma_wait_ms", C.c_uint32),
        ("fanout", C.c_uint32),
        ("test_stall", C.c_uint32),
        ("convert", C.c_uint32),
        ("convert_src_tag", C.c_uint32),
        ("convert_dst_tag", C.c_uint32),
        ("src_buf_first", C.c_uint32),
        ("src_buf_count", C.c_uint32),
    ]


class TileC(C.Structure):
    _fields_ = [
        ("src_off", C.c_uint64),
        ("dst_off", C.c_uint64),
        ("src_pitch", C.c_uint64),
        ("dst_pitch", C.c_uint64),
        ("row_bytes", C.c_uint32),
        ("rows", C.c_uint32),
        ("src_buf", C.c_uint32),
        ("dst_buf", C.c_uint32),
        ("flags", C.c_uint32),
        ("reserved", C.c_uint32 * 3),
    ]


class PlanStatsC(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "n_src_entries", "n_dst_entries", "n_fqns", "n_intersections", "n_items", "n_tiles", "n_small_tiles",
        "n_strided_tiles", "n_tma_tiles", "bytes_copied", "bytes_src_unique", "bytes_misaligned")] + [
        ("plan_ms", C.c_double), ("n_cvt_tiles", C.c_uint64), ("n_kernels", C.c_uint64)]


class IpcHandleC(C.Structure):
    _fields_ = [("handle", C.c_ubyte * 64), ("offset", C.c_uint64), ("bytes_after", C.c_uint64), ("device", C.c_int32),
                ("reserved", C.c_int32 * 3)]


class ExportEntryC(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dtype", C.c_char_p), ("ndim", C.c_uint32), ("reserved", C.c_uint32),
                ("shape", C.c_int64 * BCP_MAX_NDIM)]


class PackMetaC(C.Structure):
    _fields_ = [("byte_offset", C.c_uint64), ("byte_length", C.c_uint64)]


_VP = C.c_void_p
_PROTOS = {
    "bcp_version": (C.c_int, []),
    "bcp_last_error": (C.c_char_p, []),
    "bcp_decompose": (C.c_int, [C.POINTER(C.c_int64), C.c_uint32, C.c_int64, C.c_int64, _VP, _VP, C.c_size_t,
                                C.POINTER(C.c_size_t)]),
    "bcp_dedup_assign": (C.c_int, [C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.POINTER(C.c_uint32), C.c_size_t,
                                   C.c_size_t, C.POINTER(C.c_uint64), C.POINTER(C.c_uint32)]),
    "bcp_plan": (C.c_int, [C.POINTER(ShardMetaC), C.c_size_t, C.POINTER(C.c_uint64), C.c_size_t,
                           C.POINTER(ShardMetaC), C.c_size_t, C.POINTER(C.c_uint64), C.c_size_t,
                           C.POINTER(PlanOptsC), C.POINTER(_VP)]),
    "bcp_plan_stats": (C.c_int, [_VP, C.POINTER(PlanStatsC)]),
    "bcp_plan_serialize": (C.c_int, [_VP, _VP, C.c_size_t, C.POINTER(C.c_size_t)]),
    "bcp_plan_deserialize": (C.c_int, [_VP, C.c_size_t, C.POINTER(_VP)]),
    "bcp_plan_tiles": (C.c_int, [_VP, C.POINTER(TileC), C.c_size_t, C.POINTER(C.c_size_t)]),
    "bcp_plan_used_sources": (C.c_int, [_VP, C.POINTER(C.c_uint32), C.c_size_t, C.POINTER(C.c_size_t)]),
    "bcp_reshard": (C.c_int, [_VP, C.POINTER(_VP), C.c_size_t, C.POINTER(_VP), C.c_size_t, _VP]),
    "bcp_reshard_host": (C.c_int, [_VP, C.POINTER(_VP), C.c_size_t, C.POINTER(_VP), C.c_size_t, _VP]),
    "bcp_plan_device_status": (C.c_int, [_VP, _VP]),
    "bcp_plan_destroy": (C.c_int, [_VP]),
    "bcp_pack_layout": (C.c_int, [C.POINTER(C.c_uint64), C.c_size_t, C.c_uint64, C.POINTER(C.c_uint64),
                                  C.POINTER(C.c_uint64)]),
    "bcp_pack": (C.c_int, [C.POINTER(_VP), C.POINTER(PackMetaC), C.c_size_t, _VP, C.c_uint64, _VP]),
    "bcp_unpack": (C.c_int, [_VP, C.c_uint64, C.POINTER(PackMetaC), C.c_size_t, C.POINTER(_VP), _VP]),
    "bcp_pack_cache_clear": (C.c_int, []),
    "bcp_safetensors_layout": (C.c_int, [C.POINTER(ExportEntryC), C.c_size_t, _VP, C.c_size_t, C.POINTER(C.c_size_t),
                                         C.POINTER(PackMetaC), C.POINTER(C.c_uint64)]),
    "bcp_safetensors_export": (C.c_int, [C.POINTER(ExportEntryC), C.POINTER(_VP), C.c_size_t, _VP, C.c_uint64,
                                         C.POINTER(C.c_uint64), _VP]),
    "bcp_stager_create": (C.c_int, [C.c_uint64, C.c_uint32, C.POINTER(_VP)]),
    "bcp_stager_destroy": (C.c_int, [_VP]),
    "bcp_stager_save": (C.c_int, [_VP, C.POINTER(_VP), C.POINTER(PackMetaC), C.c_size_t, C.c_uint64, _VP,
                                  C.POINTER(C.c_uint32)]),
    "bcp_stager_wait": (C.c_int, [_VP, C.c_uint32, C.POINTER(_VP)]),
    "bcp_stager_acquire": (C.c_int, [_VP, C.POINTER(C.c_uint32), C.POINTER(_VP)]),
    "bcp_stager_load": (C.c_int, [_VP, C.c_uint32, C.c_uint64, C.POINTER(PackMetaC), C.c_size_t, C.POINTER(_VP), _VP]),
    "bcp_stager_release": (C.c_int, [_VP, C.c_uint32]),
    "bcp_ipc_export": (C.c_int, [_VP, C.POINTER(IpcHandleC)]),
    "bcp_ipc_open": (C.c_int, [C.POINTER(IpcHandleC), C.POINTER(_VP)]),
    "bcp_ipc_close": (C.c_int, [_VP]),
    "bcp_pack_static": (C.c_int, [C.POINTER(_VP), C.POINTER(PackMetaC), C.c_size_t, _VP, C.c_uint64, _VP]),
}

EXPORTS = tuple(_PROTOS)
_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Built on first use if the in-tree .so is missing or older than
    its sources; raises if it can be neither found nor built (there is no fallback path)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.is_stale():
            try:
                _build.build_library()
            except Exception as e:  # no compiler here: an existing library is still usable
                if not os.path.exists(path):
                    raise ImportError(f"libbcp.so is missing and could not be built: {e}") from e
        h = C.CDLL(path)
        for name, (res, args) in _PROTOS.items():
            f = getattr(h, name)
            f.restype, f.argtypes = res, args
        _lib = h
    return _lib
