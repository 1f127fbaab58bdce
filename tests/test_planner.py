"""Host logic of the library on CPU: decomposition, matching, lowering, work-list properties,
error codes, exported symbols.  The work list is executed by a numpy tile simulator written
here (the kernels are not involved) and compared with the oracle."""
import itertools
import os
import re

import numpy as np
import pytest

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import _lib, api
from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import CONFIGS, EXPECTED_TOTALS, convert_cases, scenario_cases
from workloads.meta import BOX, FLAT_SLICE, ShardMeta
from workloads.random_cases import big_random_case, random_case, random_convert_case

from helpers import np_bufs, read_irregular_example

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


# ---- C ABI surface -------------------------------------------------------------------------------
def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "bcp.h")).read()
    declared = set(re.findall(r"BCP_API\s+[\w\s\*]+?\b(bcp_\w+)\s*\(", text))
    assert declared == set(_lib.EXPORTS) and len(declared) >= 14
    lib = _lib.lib()
    for name in declared:
        assert getattr(lib, name) is not None
    assert bcp.bcp_version() >= 100


def test_struct_sizes_match_header():
    import ctypes as C

    assert C.sizeof(_lib.TileC) == 64
    assert C.sizeof(_lib.ShardMetaC) == 8 + 16 + 3 * 64 + 16 + 8 + 16
    assert C.sizeof(_lib.PlanOptsC) == 88
    assert C.sizeof(_lib.PlanStatsC) == 15 * 8


# ---- decomposition (Sec. 3.2) ----------------------------------------------------------------------
def test_decompose_paper_example():
    shape, recs = read_irregular_example()
    for _, a, b, boxes in recs:
        assert bcp.bcp_decompose(shape, a, b) == boxes


def _check_decomposition(shape, a, b):
    boxes = bcp.bcp_decompose(shape, a, b)
    n = len(shape)
    assert len(boxes) <= max(1, 2 * n - 1)
    idx = np.arange(int(np.prod(shape, dtype=np.int64))).reshape(shape)
    pos = a
    for off, ln in boxes:
        sub = idx[tuple(slice(o, o + l) for o, l in zip(off, ln))].ravel()
        # each box is a contiguous piece of the flattening and the boxes follow one another
        assert sub.size > 0 and np.array_equal(sub, np.arange(pos, pos + sub.size))
        pos += sub.size
    assert pos == max(a, b) if b > a else boxes == []


def test_decompose_brute_force_small_shapes():
    shapes = [s for nd in (1, 2, 3) for s in itertools.product(range(1, 5), repeat=nd)] + [(2, 1, 3, 2), (1, 1, 5), (3, 2, 2, 2)]
    for shape in shapes:
        n = int(np.prod(shape))
        for a in range(n + 1):
            for b in range(a, n + 1):
                _check_decomposition(shape, a, b)
    assert bcp.bcp_decompose((), 0, 1) == [((), ())]
    assert bcp.bcp_decompose((), 0, 0) == []


def test_decompose_large_and_errors():
    _check_decomposition((128, 97, 3), 1234, 30001)
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_decompose((3, 2), 2, 9)
    assert e.value.code == api.ERR_INVALID


# ---- tile simulator -----------------------------------------------------------------------------------
def run_tiles(tiles, src, dst_sizes, poison=0xA5):
    out = [np.full(n, poison, dtype=np.uint8) for n in dst_sizes]
    count = [np.zeros(n, dtype=np.uint8) for n in dst_sizes]
    for t in tiles:
        g = 1 << (t.flags & api.TILE_GRAN_MASK)
        assert t.dst_off % g == 0 and t.row_bytes % g == 0 and t.dst_pitch % g == 0
        kind = (t.flags & api.TILE_CVT_MASK) >> api.TILE_CVT_SHIFT
        if kind:  # converting unit: row_bytes counts target bytes, the source row holds the same elements
            assert not t.flags & (api.TILE_ZERO | api.TILE_SMALL | api.TILE_TMA2D | api.TILE_FOLLOW)
            s_isz, d_isz = (4, 2) if kind == api.CONVERT_F32_TO_BF16 else (2, 4)
            assert t.row_bytes % d_isz == 0 and t.dst_off % d_isz == 0 and t.src_off % s_isz == 0
            n = t.row_bytes // d_isz
            for r in range(t.rows):
                d0, s0 = t.dst_off + r * t.dst_pitch, t.src_off + r * t.src_pitch
                chunk = src[t.src_buf][s0:s0 + n * s_isz]
                assert chunk.size == n * s_isz
                if kind == api.CONVERT_F32_TO_BF16:  # the usual integer form of round-to-nearest-even
                    x = chunk.view(np.uint32).astype(np.uint64)
                    y = np.where((x & 0x7FFFFFFF) > 0x7F800000, 0x7FC0, (x + 0x7FFF + ((x >> 16) & 1)) >> 16).astype(np.uint16)
                else:
                    y = chunk.view(np.uint16).astype(np.uint32) << 16
                out[t.dst_buf][d0:d0 + t.row_bytes] = y.view(np.uint8)
                count[t.dst_buf][d0:d0 + t.row_bytes] += 1
            continue
        for r in range(t.rows):
            d0 = t.dst_off + r * t.dst_pitch
            if t.flags & api.TILE_ZERO:
                out[t.dst_buf][d0:d0 + t.row_bytes] = 0
            else:
                assert t.src_off % g == 0 and t.src_pitch % g == 0
                s0 = t.src_off + r * t.src_pitch
                chunk = src[t.src_buf][s0:s0 + t.row_bytes]
                assert chunk.size == t.row_bytes
                out[t.dst_buf][d0:d0 + t.row_bytes] = chunk
            count[t.dst_buf][d0:d0 + t.row_bytes] += 1
    return out, count


def check_case(case, fill="index", **opts):
    blobs = np_bufs(fills.fill_state(case.src, case.key_ids, fill, case.seed, "cpu", poison=0x5A))
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts, **case.plan_opts)
    tiles = plan.tiles()
    st = plan.stats()
    got, count = run_tiles(tiles, blobs, case.dst.buf_bytes)
    want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, convert=case.convert)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    # every named target byte is written exactly once, every other byte never
    named = [np.zeros(n, dtype=np.uint8) for n in case.dst.buf_bytes]
    for m in case.dst.metas:
        named[m.buf_index][m.byte_offset:m.byte_offset + m.byte_length] += 1
    for c, n in zip(count, named):
        assert np.array_equal(c, n)
    assert st["bytes_copied"] == case.dst.total_bytes
    tb = opts.get("tile_bytes", 65536)
    assert all(t.rows * t.row_bytes <= tb for t in tiles)
    assert st["n_tiles"] + st["n_small_tiles"] + st["n_cvt_tiles"] == len(tiles)
    rank = [2 if t.flags & api.TILE_CVT_MASK else 1 if t.flags & api.TILE_SMALL else 0 for t in tiles]
    assert rank == sorted(rank), "CTA-wide units come first, converting units last"
    plan.destroy()
    return st


@pytest.mark.parametrize("case", scenario_cases(), ids=lambda c: c.name)
def test_scenarios_match_oracle(case):
    check_case(case)


@pytest.mark.parametrize("fill", ["uniform", "index"])
def test_cfg1_matches_oracle(fill):
    st = check_case(CONFIGS["cfg1"](fill), fill)
    assert st["bytes_misaligned"] == 0 and st["bytes_src_unique"] == EXPECTED_TOTALS["cfg1"][0]
    assert (st["n_src_entries"], st["n_dst_entries"], st["n_intersections"]) == (234, 211, 423)


@pytest.mark.parametrize("seed", range(60))
def test_random_tiny_cases(seed):
    check_case(random_case(seed, dst_replicas=1 + seed % 2), tile_bytes=4096, small_bytes=64 if seed % 3 else 4096)


@pytest.mark.parametrize("seed", range(100, 112))
def test_random_cases_up_to_eight_dims(seed):
    """The maximum rank the ABI allows, with flat slices that need deep decompositions."""
    check_case(random_case(seed, n_tensors=3, max_ndim=8, max_dim=3, dst_replicas=1 + seed % 2), tile_bytes=4096)


@pytest.mark.parametrize("itemsize,seed", [(1, 1), (2, 2), (4, 3), (8, 4), (2, 5)])
def test_big_random_cases(itemsize, seed):
    st = check_case(big_random_case(seed, itemsize=itemsize), tile_bytes=8192, order=1 + seed % 2)
    assert st["bytes_misaligned"] > 0


@pytest.mark.parametrize("opts", [dict(tile_bytes=4096), dict(order=2), dict(tile_bytes=1 << 20, small_bytes=65536),
                                  dict(path_mask=7), dict(path_mask=7, tile_bytes=8192)])
def test_options_do_not_change_the_result(opts):
    check_case(scenario_cases()[3], **opts)
    check_case(CONFIGS["cfg1"]("index"), **opts)


def test_tensor_map_rectangles_are_whole_boxes():
    """Units flagged for 2-D tensor-map staging cover whole boxes of their rectangle."""
    case = CONFIGS["cfg1"]("index")
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=7)
    tiles = [t for t in plan.tiles() if t.flags & api.TILE_TMA2D]
    assert tiles, "cfg1 has row-parallel weights with rows of 256..1024 bytes"
    for t in tiles:
        box_rows = t.reserved[2]
        assert t.reserved[0] >= 1 and box_rows >= 1 and t.reserved[1] % box_rows == 0
        assert 16 <= t.row_bytes <= 2048 and box_rows * t.row_bytes <= 16384
        assert (t.src_off | t.dst_off | t.src_pitch | t.dst_pitch | t.row_bytes) % 16 == 0
    again = bcp.Plan.deserialize(plan.serialize())
    assert [_tile_tuple(t) for t in again.tiles()] == [_tile_tuple(t) for t in plan.tiles()]


def test_plans_partitioned_by_target_rank_cover_everything():
    """Several devices by construction: each device plans only the target ranks it hosts against
    the full saved metadata (the saved side may hold more than is wanted) and reads remote
    source blobs through whatever pointers it is given.  The per-device plans together must
    write exactly what the single plan writes."""
    case = scenario_cases()[3]
    blobs = np_bufs(fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu"))
    want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5)
    n_dev = 3
    got = [None] * len(case.dst.buf_bytes)
    total = 0
    for dev in range(n_dev):
        ranks = [r for r in range(len(case.dst.buf_bytes)) if r % n_dev == dev]
        local = {r: i for i, r in enumerate(ranks)}
        metas = []
        for m in case.dst.metas:
            if m.buf_index in local:
                metas.append(ShardMeta(m.fqn, m.itemsize, m.dtype_tag, m.global_shape, m.offsets, m.lengths,
                                       local[m.buf_index], m.byte_offset, m.kind, m.flat_begin, m.flat_end))
        sizes = [case.dst.buf_bytes[r] for r in ranks]
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, metas, sizes)
        out, _ = run_tiles(plan.tiles(), blobs, sizes)
        total += plan.stats()["bytes_copied"]
        for r, o in zip(ranks, out):
            got[r] = o
    assert total == case.dst.total_bytes
    for g, w in zip(got, want):
        assert np.array_equal(g, w)


# ---- replicated saved shards (a checkpoint written without de-duplication) ------------------------------
def _replicated_case():
    """The hybrid scenario with its saved side NOT de-duplicated: every holder stores its copy."""
    from workloads.configs import MIXED, small_gpt
    from workloads.layouts import Parallelism, ReshardCase, build_state

    g = small_gpt()
    src = build_state(g, Parallelism(tp=2, dp=2, pp=2, zero="zero1"), MIXED, dedup=False)
    dst = build_state(g, Parallelism(tp=1, dp=3, pp=4, zero="zero1"), MIXED, dedup=False)
    return ReshardCase("replicated-source", src, dst, "index", 5)


def test_replicas_are_an_error_unless_allowed():
    case = _replicated_case()
    assert _plan_err(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes) == api.ERR_OVERLAP
    blobs = np_bufs(fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu"))
    with pytest.raises(orc.OracleError):
        orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, allow_replicas=1)
    got, _ = run_tiles(plan.tiles(), blobs, case.dst.buf_bytes)
    want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, allow_replicas=True)
    assert all(np.array_equal(g, w) for g, w in zip(got, want))
    # consistent replicas: same result as the closed-form fill of the wanted side
    closed = np_bufs(fills.fill_state(case.dst, case.key_ids, "index", case.seed, "cpu", poison=0xA5))
    assert all(np.array_equal(g, w) for g, w in zip(got, closed))
    assert plan.stats()["bytes_src_unique"] < case.src.total_bytes


def test_first_replica_wins_and_partial_overlap_stays_an_error():
    a = _m(boff=0)
    b = _m(boff=64)  # same box, different bytes
    blob = np.concatenate([np.full(64, 1, np.uint8), np.full(64, 2, np.uint8)])
    plan = bcp.bcp_plan([a, b], [128], [_m()], [64], allow_replicas=1)
    got, _ = run_tiles(plan.tiles(), [blob], [64])
    want = orc.reshard([a, b], [blob], [_m()], [64], allow_replicas=True)
    assert np.array_equal(got[0], want[0]) and set(got[0]) == {1}
    plan = bcp.bcp_plan([b, a], [128], [_m()], [64], allow_replicas=1)  # input order decides, not byte order
    got, _ = run_tiles(plan.tiles(), [blob], [64])
    assert set(got[0]) == {2} and np.array_equal(got[0], orc.reshard([b, a], [blob], [_m()], [64], allow_replicas=True)[0])
    assert _plan_err([_m(ln=(3, 4)), _m(off=(2, 0), ln=(2, 4), boff=48)], [80], [_m()], [64], allow_replicas=1) == api.ERR_OVERLAP


def test_single_run_larger_than_4_gib_is_cut_without_overflow():
    n = 6 * (1 << 30) + 48
    m = ShardMeta("huge", 1, 3, (n,), (0,), (n,), 0, 16)
    plan = bcp.bcp_plan([m], [n + 16], [ShardMeta("huge", 1, 3, (n,), (0,), (n,), 0, 0)], [n])
    tiles = plan.tiles()
    assert sum(t.rows * t.row_bytes for t in tiles) == n and plan.stats()["bytes_copied"] == n
    order = sorted(tiles, key=lambda t: t.dst_off)
    assert order[0].dst_off == 0 and all(a.dst_off + a.row_bytes == b.dst_off for a, b in zip(order, order[1:]))
    assert all(t.src_off == t.dst_off + 16 for t in tiles) and order[-1].dst_off + order[-1].row_bytes == n


def test_replica_units_follow_their_head():
    """Units that read the same source bytes are grouped (read once, write many): followers sit
    right behind a head with identical source geometry, at most 7 per head."""
    case = scenario_cases()[2]  # dp4 -> dp8: every parameter shard is wanted by 8 data-parallel ranks
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3, tile_bytes=4096,
                        tma_min_row_bytes=64, fanout=1)
    tiles = plan.tiles()
    heads = [i for i, t in enumerate(tiles) if (t.flags >> 8) & 7]
    for i in heads:  # a head announces exactly the followers behind it
        k = (tiles[i].flags >> 8) & 7
        assert all(tiles[i + j].flags & api.TILE_FOLLOW for j in range(1, k + 1))
        assert i + k + 1 == len(tiles) or not (tiles[i + k + 1].flags & api.TILE_FOLLOW)
    n_follow, run = 0, 1
    for prev, t in zip(tiles, tiles[1:]):
        if t.flags & api.TILE_FOLLOW:
            n_follow += 1
            run += 1
            assert run <= 8 and t.flags & api.TILE_TMA and prev.flags & api.TILE_TMA
            assert (prev.src_buf, prev.src_off, prev.rows, prev.row_bytes, prev.src_pitch) == \
                   (t.src_buf, t.src_off, t.rows, t.row_bytes, t.src_pitch)
            assert (prev.dst_buf, prev.dst_off) != (t.dst_buf, t.dst_off)
        else:
            run = 1
    assert n_follow > 0 and not (tiles[0].flags & api.TILE_FOLLOW)
    assert not any(t.flags & api.TILE_FOLLOW for t in bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas,
                                                                  case.dst.buf_bytes, path_mask=3, order=2, fanout=1).tiles())
    assert not any(t.flags & api.TILE_FOLLOW for t in bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas,
                                                                  case.dst.buf_bytes, path_mask=3, fanout=2).tiles())
    again = bcp.Plan.deserialize(plan.serialize())
    assert [_tile_tuple(t) for t in again.tiles()] == [_tile_tuple(t) for t in tiles]


# ---- plan images (plan cache across processes, Sec. 4.1) ----------------------------------------------
def _tile_tuple(t):
    return (t.src_off, t.dst_off, t.src_pitch, t.dst_pitch, t.row_bytes, t.rows, t.src_buf, t.dst_buf, t.flags)


@pytest.mark.parametrize("case", [CONFIGS["cfg1"]("index"), scenario_cases()[3], big_random_case(5, itemsize=2)],
                         ids=lambda c: c.name)
def test_plan_image_round_trip(case):
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3, tile_bytes=16384)
    image = plan.serialize()
    again = bcp.Plan.deserialize(image)
    assert [_tile_tuple(t) for t in again.tiles()] == [_tile_tuple(t) for t in plan.tiles()]
    assert again.stats() == plan.stats()
    assert again.serialize() == image
    # the rebuilt work list still computes the oracle's result
    blobs = np_bufs(fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu"))
    got, _ = run_tiles(again.tiles(), blobs, case.dst.buf_bytes)
    want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5)
    assert all(np.array_equal(g, w) for g, w in zip(got, want))


def _image_without_clock(plan):
    """Plan image with the planning-time field and the checksum over it blanked."""
    import struct

    image = plan.serialize()
    at = image.find(struct.pack("<d", plan.stats()["plan_ms"]))
    assert 0 < at < 256
    return image[:at] + bytes(8) + image[at + 8:-8]


@pytest.mark.parametrize("opts", [dict(), dict(order=2, tile_bytes=16384), dict(path_mask=1)], ids=str)
def test_work_list_does_not_depend_on_the_number_of_planner_threads(opts, monkeypatch):
    case = CONFIGS["cfg3"]()  # 16 GB, a quarter of a million units: large enough for helper threads
    images = []
    for threads in ("1", "3", "8"):
        monkeypatch.setenv("BCP_PLAN_THREADS", threads)
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts)
        assert plan.stats()["n_tiles"] > 100_000
        images.append(_image_without_clock(plan))
        plan.destroy()
    assert images[0] == images[1] == images[2]


def test_matching_does_not_depend_on_the_number_of_planner_threads(monkeypatch):
    """Above 32k input entries tensors are expanded and matched by several threads; the plan, its
    statistics and the error that is reported (the earliest tensor's, as in serial order) stay the same."""
    import copy

    from workloads.configs import OPTIM_ONLY
    from workloads.layouts import Parallelism, llama_model, reshard_case

    m = llama_model("llama-3b-fsdp", L=28, H=3072, nq=24, nkv=8, F=8192, V=128256, fused=False, tied=True, fsdp_units=True)
    case = reshard_case("dp256-to-dp192", m, Parallelism(dp=256, zero="fsdp"), Parallelism(dp=192, zero="fsdp"), OPTIM_ONLY)
    assert len(case.src.metas) + len(case.dst.metas) > 32768
    twice = list(case.src.metas) + [copy.copy(case.src.metas[len(case.src.metas) // 2]), copy.copy(case.src.metas[len(case.src.metas) // 5])]
    images, errors = [], []
    for threads in ("1", "8", "3"):
        monkeypatch.setenv("BCP_PLAN_THREADS", threads)
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
        images.append(_image_without_clock(plan))
        plan.destroy()
        with pytest.raises(bcp.BcpError) as e:  # two tensors hold an element twice
            bcp.bcp_plan(twice, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
        assert e.value.code == api.ERR_OVERLAP
        errors.append(str(e.value))
    assert images[0] == images[1] == images[2]
    assert errors[0] == errors[1] == errors[2]


def test_plan_image_is_verified():
    case = scenario_cases()[0]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    image = bytearray(plan.serialize())
    for bad in (image[:-1], image[:40], b"", bytes(len(image))):
        with pytest.raises(bcp.BcpError):
            bcp.Plan.deserialize(bytes(bad))
    flipped = bytearray(image)
    flipped[len(flipped) // 2] ^= 0x40  # a corrupted unit: caught by the checksum
    with pytest.raises(bcp.BcpError) as e:
        bcp.Plan.deserialize(bytes(flipped))
    assert "checksum" in str(e.value)


def _reseal(image: bytearray) -> bytes:
    """Recompute the trailing FNV-1a checksum after editing an image (what a careless or hostile
    writer of plan files could do)."""
    h = 1469598103934665603
    for b in image[:-8]:
        h = ((h ^ b) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return bytes(image[:-8]) + h.to_bytes(8, "little")


def test_plan_image_units_are_checked_against_the_buffers():
    """A unit drives device copies, so a well-formed image with a wrong unit must be refused:
    plain and converting units are edited in place and the image is resealed."""
    import ctypes as C
    import struct

    case = convert_cases()[2]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, tile_bytes=4096, **case.plan_opts)
    tiles = plan.tiles()
    image = bytearray(plan.serialize())
    first = image.find(bytes(tiles[0]))  # the first unit record inside the image
    assert first > 0 and bcp.Plan.deserialize(_reseal(bytearray(image))).stats() == plan.stats()
    cvt = next(i for i, t in enumerate(tiles) if t.flags & api.TILE_CVT_MASK)
    F = {n: getattr(_lib.TileC, n).offset for n, _ in _lib.TileC._fields_}

    def edited(i, field, fn):
        out = bytearray(image)
        at = first + i * C.sizeof(_lib.TileC) + F[field]
        width = 8 if field.endswith("off") or field.endswith("pitch") else 4
        v = int.from_bytes(out[at:at + width], "little")
        out[at:at + width] = fn(v).to_bytes(width, "little")
        return _reseal(out)

    bad = [
        edited(cvt, "row_bytes", lambda v: v + (1 << 24)),        # runs past both buffers
        edited(cvt, "src_off", lambda v: v + 2),                   # binary32 source not 4-byte aligned
        edited(cvt, "dst_off", lambda v: v + 1),                   # bfloat16 target not 2-byte aligned
        edited(cvt, "flags", lambda v: v | api.TILE_SMALL),        # a converting unit has no other class
        edited(cvt, "flags", lambda v: v | api.TILE_CVT_MASK),     # unknown conversion kind
        edited(cvt, "flags", lambda v: v & ~api.TILE_CVT_MASK),    # plain unit in the converting class
        edited(cvt, "src_buf", lambda v: v + 1000),
        edited(0, "dst_off", lambda v: v + (1 << 40)),
    ]
    for im in bad:
        with pytest.raises(bcp.BcpError) as e:
            bcp.Plan.deserialize(im)
        assert "work unit" in str(e.value) or "inconsistent" in str(e.value)
    plan.destroy()


# ---- full-size configurations: planning is host-only, so their work lists are checked here ---------
@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_config_plans(name):
    case = CONFIGS[name]()
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    st = plan.stats()
    src_total, dst_total = EXPECTED_TOTALS[name]
    assert st["bytes_copied"] == dst_total and st["bytes_src_unique"] == src_total
    assert st["bytes_misaligned"] == 0, "every unit of the benchmark configs moves whole 16-byte vectors"
    tiles = plan.tiles()
    written = sum(t.rows * t.row_bytes for t in tiles)
    assert written == dst_total
    # in-bounds on both sides and 16-byte aligned
    sb, db = case.src.buf_bytes, case.dst.buf_bytes
    for t in tiles[:: max(1, len(tiles) // 5000)]:
        assert t.src_off + (t.rows - 1) * t.src_pitch + t.row_bytes <= sb[t.src_buf]
        assert t.dst_off + (t.rows - 1) * t.dst_pitch + t.row_bytes <= db[t.dst_buf]
        assert (t.src_off | t.dst_off | t.row_bytes | t.src_pitch | t.dst_pitch) % 16 == 0
    plan.destroy()


# ---- error behaviour (all detected on the host, before any launch) -----------------------------------
def _m(fqn="w", isz=4, tag=2, shape=(4, 4), off=(0, 0), ln=(4, 4), buf=0, boff=0, **kw):
    return ShardMeta(fqn, isz, tag, shape, off, ln, buf, boff, **kw)


def _plan_err(src, sb, dst, db, **opts):
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_plan(src, sb, dst, db, **opts)
    assert str(e.value)
    return e.value.code


def test_error_codes():
    full = [_m()]
    assert _plan_err([_m(isz=3)], [64], full, [64]) == api.ERR_INVALID
    assert _plan_err([_m(off=(1, 0))], [64], full, [64]) == api.ERR_INVALID  # box leaves the global shape
    assert _plan_err([_m(kind=FLAT_SLICE, flat_begin=3, flat_end=20)], [128], full, [64]) == api.ERR_INVALID
    assert _plan_err(full, [64], [_m(tag=9)], [64]) == api.ERR_MISMATCH
    assert _plan_err(full, [64], [_m(shape=(4, 5), ln=(4, 4))], [64]) == api.ERR_MISMATCH
    assert _plan_err([_m(ln=(3, 4)), _m(off=(2, 0), ln=(2, 4), boff=48)], [80], full, [64]) == api.ERR_OVERLAP
    assert _plan_err([_m(ln=(3, 4))], [64], full, [64]) == api.ERR_UNCOVERED
    assert _plan_err([], [], full, [64]) == api.ERR_UNCOVERED
    assert _plan_err(full, [63], full, [64]) == api.ERR_BOUNDS
    assert _plan_err(full, [64], [_m(buf=1)], [64]) == api.ERR_BOUNDS
    assert _plan_err(full, [64], [_m(), _m(boff=32)], [128]) == api.ERR_DST_ALIAS
    assert _plan_err(full, [64], full, [64], tile_bytes=1000) == api.ERR_INVALID
    assert _plan_err(full, [64], full, [64], block_threads=100) == api.ERR_INVALID
    # partial loads are fine: the saved side may hold more than is wanted
    p = bcp.bcp_plan(full, [64], [_m(off=(1, 1), ln=(2, 2))], [16])
    assert p.stats()["bytes_copied"] == 16
    # zero-volume and scalar entries
    p = bcp.bcp_plan([_m("s", 8, 4, (), (), ()), _m("e", shape=(4, 0), ln=(4, 0))], [8],
                     [_m("s", 8, 4, (), (), ()), _m("e", shape=(4, 0), off=(1, 0), ln=(2, 0), boff=8)], [8])
    assert p.stats()["bytes_copied"] == 8


def test_pack_layout_matches_closed_form():
    sizes = [1, 255, 256, 257, 4096, 3, 0, 1000]
    for align in (16, 256, 4096):
        assert bcp.bcp_pack_layout(sizes, align) == orc.pack_layout(sizes, align)
    with pytest.raises(bcp.BcpError):
        bcp.bcp_pack_layout(sizes, 24)


# ---- element conversion (an extension: the paper moves bytes only) -------------------------------
@pytest.mark.parametrize("case", convert_cases(), ids=lambda c: c.name)
@pytest.mark.parametrize("opts", [dict(), dict(tile_bytes=4096, order=2)], ids=str)
def test_converting_plans_match_oracle(case, opts):
    st = check_case(case, **opts)
    assert st["n_cvt_tiles"] > 0 and st["n_tma_tiles"] == 0
    # source bytes are counted in the saved type, target bytes in the wanted one
    assert st["bytes_copied"] == case.dst.total_bytes and st["bytes_src_unique"] == case.src.total_bytes


@pytest.mark.parametrize("seed", range(40))
def test_random_converting_cases(seed):
    """Converted and unchanged tensors in one plan, flat slices, odd offsets, replicas on the wanted side."""
    check_case(random_convert_case(seed, narrow=seed % 2 == 0, dst_replicas=1 + seed % 3 // 2), tile_bytes=4096)


@pytest.mark.parametrize("seed,narrow", [(1, True), (2, False)])
def test_big_random_converting_cases(seed, narrow):
    st = check_case(random_convert_case(seed, narrow=narrow, big=True, dst_replicas=2), tile_bytes=8192)
    assert st["n_cvt_tiles"] > 100 and st["n_tiles"] + st["n_small_tiles"] > 0


def test_converting_entries_must_be_element_aligned():
    """A plain copy may start at any byte; a conversion reads and writes whole elements."""
    f32, bf16 = 2, 1
    opts = dict(convert=api.CONVERT_F32_TO_BF16, convert_src_tag=f32, convert_dst_tag=bf16)
    assert _plan_err([_m("a", 4, f32, boff=2)], [96], [_m("a", 2, bf16)], [64], **opts) == api.ERR_INVALID
    assert _plan_err([_m("a", 4, f32)], [96], [_m("a", 2, bf16, boff=1)], [64], **opts) == api.ERR_INVALID
    bcp.bcp_plan([_m("a", 4, f32, boff=4)], [96], [_m("a", 2, bf16, boff=6)], [64], **opts).destroy()


def test_conversion_is_per_tensor_and_needs_both_tags():
    f32, bf16 = 2, 1
    src = [_m("a", 4, f32, boff=0), _m("b", 2, bf16, boff=64)]
    dst = [_m("a", 2, bf16, boff=0), _m("b", 2, bf16, boff=32)]
    # without the option a tensor that changes its type is a mismatch, as before
    assert _plan_err(src, [96], dst, [64]) == api.ERR_MISMATCH
    plan = bcp.bcp_plan(src, [96], dst, [64], convert=api.CONVERT_F32_TO_BF16, convert_src_tag=f32, convert_dst_tag=bf16)
    tiles = plan.tiles()
    assert sorted((t.flags & api.TILE_CVT_MASK) >> api.TILE_CVT_SHIFT for t in tiles) == [0, 1]  # "b" is copied, "a" converted
    plan.destroy()
    # the wrong direction, the wrong tags, or the wrong sizes are still mismatches
    assert _plan_err(src, [96], dst, [64], convert=api.CONVERT_BF16_TO_F32, convert_src_tag=f32, convert_dst_tag=bf16) == api.ERR_MISMATCH
    assert _plan_err(src, [96], dst, [64], convert=api.CONVERT_F32_TO_BF16, convert_src_tag=bf16, convert_dst_tag=f32) == api.ERR_MISMATCH
    assert _plan_err([_m("a", 8, f32)], [128], [_m("a", 2, bf16)], [32], convert=1, convert_src_tag=f32, convert_dst_tag=bf16) == api.ERR_MISMATCH
    # wanted entries of one tensor must agree among themselves
    two = [_m("a", 2, bf16, off=(0, 0), ln=(2, 4), boff=0), _m("a", 4, f32, off=(2, 0), ln=(2, 4), boff=32)]
    assert _plan_err(src[:1], [64], two, [64], convert=1, convert_src_tag=f32, convert_dst_tag=bf16) == api.ERR_MISMATCH
    # option checks
    assert _plan_err(src, [96], dst, [64], convert=3, convert_src_tag=f32, convert_dst_tag=bf16) == api.ERR_INVALID
    assert _plan_err(src, [96], dst, [64], convert=1, convert_src_tag=f32, convert_dst_tag=f32) == api.ERR_INVALID
    assert _plan_err(src, [96], dst, [64], convert_src_tag=f32) == api.ERR_INVALID


def test_converting_plan_image_round_trip():
    case = convert_cases()[2]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, tile_bytes=4096, **case.plan_opts)
    image = plan.serialize()
    again = bcp.Plan.deserialize(image)
    assert again.serialize() == image and again.stats()["n_cvt_tiles"] == plan.stats()["n_cvt_tiles"] > 0
    blobs = np_bufs(fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu"))
    got, _ = run_tiles(again.tiles(), blobs, case.dst.buf_bytes)
    want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, convert=case.convert)
    assert all(np.array_equal(g, w) for g, w in zip(got, want))


# ---- host threads --------------------------------------------------------------------------------
def test_planning_from_several_threads_at_once():
    """Different plans may be built and read from different threads at the same time; error
    texts are per thread.  (The binding releases the interpreter lock inside every call.)"""
    import threading

    cases = [random_case(s) for s in range(6)] + [big_random_case(2, itemsize=2), big_random_case(4, itemsize=4)]

    def image(case):
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, tile_bytes=4096)
        out = _image_without_clock(plan)
        plan.destroy()
        return out

    want = [image(c) for c in cases]
    failures = []

    def work(tid):
        try:
            for rep in range(12):
                k = (tid + rep) % len(cases)
                if image(cases[k]) != want[k]:
                    failures.append(f"thread {tid}: plan {k} differs")
                if tid % 2:  # this thread also fails on purpose; the message must be its own
                    name = f"t{tid}r{rep}"
                    try:
                        bcp.bcp_plan([_m(fqn=name, isz=3)], [64], [_m(fqn=name)], [64])
                        failures.append("no error raised")
                    except bcp.BcpError as e:
                        if e.code != api.ERR_INVALID or name not in str(e):
                            failures.append(f"thread {tid}: foreign error text {e}")
        except Exception as e:  # noqa: BLE001 - reported below
            failures.append(f"thread {tid}: {e!r}")

    threads = [threading.Thread(target=work, args=(t,)) for t in range(6)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not failures, failures[:3]


# ---- plans restricted to some source buffers (the two-plan form of the cross-rank exchange) -------
@pytest.mark.parametrize("path_mask", [1, 3])
def test_source_ranges_partition_the_work_list(path_mask):
    """Plans for disjoint source-buffer ranges that cover all buffers hold, between them, exactly
    the units of the unrestricted plan, each reads only its own range, and coverage is still
    checked against every saved entry."""
    for case in [c for c in scenario_cases() if c.name in ("hybrid", "llama-tp8-to-tp2", "dp150-to-dp75")] + [random_case(5, n_tensors=4)]:
        ns = len(case.src.buf_bytes)
        args = (case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
        opts = dict(case.plan_opts, path_mask=path_mask, tile_bytes=8192)
        whole = bcp.bcp_plan(*args, **opts)
        key = lambda t: (t.src_buf, t.src_off, t.dst_buf, t.dst_off, t.rows, t.row_bytes, t.src_pitch, t.dst_pitch)  # noqa: E731
        want = sorted(key(t) for t in whole.tiles())
        for cuts in ([0, ns], [0, 1, ns], [0, ns // 2, ns], [0, ns // 3, ns - 1, ns]):
            cuts = sorted(set(cuts))
            got, copied, uniq = [], 0, 0
            for lo, hi in zip(cuts[:-1], cuts[1:]):
                part = bcp.bcp_plan(*args, src_buf_first=lo, src_buf_count=hi - lo, **opts)
                ts = part.tiles()
                assert all(lo <= t.src_buf < hi for t in ts)
                got += [key(t) for t in ts]
                copied += part.stats()["bytes_copied"]
                uniq += part.stats()["bytes_src_unique"]
                part.destroy()
            assert sorted(got) == want, (case.name, cuts)
            assert copied == whole.stats()["bytes_copied"] and uniq == whole.stats()["bytes_src_unique"]
        whole.destroy()
    # a restricted plan still refuses a target that the saved entries as a whole do not cover
    case = [c for c in scenario_cases() if c.name == "hybrid"][0]
    fewer = [m for m in case.src.metas if m.buf_index != 0]
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_plan(fewer, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, src_buf_first=1, src_buf_count=1)
    assert e.value.code == api.ERR_UNCOVERED
    for first, count in ((1, 0), (0, len(case.src.buf_bytes) + 1), (len(case.src.buf_bytes), 1)):
        with pytest.raises(bcp.BcpError) as e:
            bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, src_buf_first=first, src_buf_count=count)
        assert e.value.code == api.ERR_INVALID


# ---- replicated saved shards, random layouts ---------------------------------------------------------
@pytest.mark.parametrize("seed", range(12))
def test_random_replicated_sources_first_in_input_order_is_read(seed):
    """Some saved shards are stored twice with different bytes, at random places of the input:
    the work list (numpy simulator) must read the first one, as the oracle does."""
    import copy

    rng = np.random.default_rng(2000 + seed)
    case = random_case(seed, n_tensors=4, dst_replicas=1 + seed % 2)
    metas, pos = list(case.src.metas), 0
    extra = []
    for m in case.src.metas:
        if m.byte_length and rng.random() < 0.5:
            k = copy.copy(m)
            k.buf_index, k.byte_offset = len(case.src.buf_bytes), pos
            pos += m.byte_length + int(rng.integers(0, 3)) * m.itemsize
            extra.append(k)
    for k in extra:
        metas.insert(int(rng.integers(0, len(metas) + 1)), k)
    sizes = list(case.src.buf_bytes) + [max(pos, 1)]
    blobs = [rng.integers(0, 256, size=n, dtype=np.uint8) for n in sizes]
    plan = bcp.bcp_plan(metas, sizes, case.dst.metas, case.dst.buf_bytes, allow_replicas=1, tile_bytes=4096)
    got, _ = run_tiles(plan.tiles(), blobs, case.dst.buf_bytes)
    want = orc.reshard(metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, allow_replicas=True)
    assert all(np.array_equal(g, w) for g, w in zip(got, want))
    plan.destroy()
    if extra:
        assert _plan_err(metas, sizes, case.dst.metas, case.dst.buf_bytes) == api.ERR_OVERLAP


def test_replicas_must_be_whole_shards():
    """One rank saved a tensor whole, another saved the same tensor as two flat slices: the element
    sets overlap only partly entry by entry, which is an error with and without allow_replicas
    (library and oracle alike): replicas are shards stored more than once, box for box."""
    whole = ShardMeta("x", 4, 2, (6, 4), (0, 0), (6, 4), 0, 0)
    lo = ShardMeta("x", 4, 2, (6, 4), (0, 0), (6, 4), 1, 0, kind=FLAT_SLICE, flat_begin=0, flat_end=10)
    hi = ShardMeta("x", 4, 2, (6, 4), (0, 0), (6, 4), 1, 40, kind=FLAT_SLICE, flat_begin=10, flat_end=24)
    want = [ShardMeta("x", 4, 2, (6, 4), (0, 0), (6, 4), 0, 0)]
    blobs = [np.arange(96, dtype=np.uint8), np.arange(96, dtype=np.uint8)[::-1].copy()]
    for allow in (0, 1):
        assert _plan_err([whole, lo, hi], [96, 96], want, [96], allow_replicas=allow) == api.ERR_OVERLAP
        with pytest.raises(orc.OracleError):
            orc.reshard([whole, lo, hi], blobs, want, [96], allow_replicas=bool(allow))
    # the same flat slices stored twice are replicas
    lo2, hi2 = ShardMeta(**{**lo.__dict__, "buf_index": 0}), ShardMeta(**{**hi.__dict__, "buf_index": 0})
    plan = bcp.bcp_plan([lo, hi, lo2, hi2], [96, 96], want, [96], allow_replicas=1)
    got, _ = run_tiles(plan.tiles(), blobs, [96])
    assert np.array_equal(got[0], orc.reshard([lo, hi, lo2, hi2], blobs, want, [96], allow_replicas=True)[0])
    assert np.array_equal(got[0], blobs[1])
    plan.destroy()


# ---- which saved entries a plan reads ------------------------------------------------------------------
def _element_mask(m):
    mask = np.zeros(tuple(m.global_shape), dtype=bool)
    box = tuple(slice(o, o + l) for o, l in zip(m.offsets, m.lengths))
    if m.kind == FLAT_SLICE:
        flat = mask[box].ravel()
        flat[m.flat_begin:m.flat_end] = True
        mask[box] = flat.reshape(mask[box].shape)
    else:
        mask[box] = True
    return mask


@pytest.mark.parametrize("seed", range(20))
def test_used_sources_are_the_saved_entries_that_share_an_element_with_a_wanted_one(seed):
    case = random_case(300 + seed, n_tensors=5, dst_replicas=1 + seed % 2)
    wanted = {}
    for d in case.dst.metas:
        wanted[d.fqn] = wanted.get(d.fqn, False) | _element_mask(d)
    expect = [i for i, s in enumerate(case.src.metas) if s.fqn in wanted and bool((_element_mask(s) & wanted[s.fqn]).any())]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    assert plan.used_sources() == expect
    plan.destroy()
    # a plan for part of the targets reads fewer entries; a plan restricted to some source buffers only entries in them
    half = [d for d in case.dst.metas if d.buf_index == 0]
    if half:
        sub = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, half, case.dst.buf_bytes)
        assert set(sub.used_sources()) <= set(expect)
        sub.destroy()
    only0 = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, src_buf_first=0, src_buf_count=1)
    assert only0.used_sources() == [i for i in expect if case.src.metas[i].buf_index == 0]
    image = only0.serialize()
    only0.destroy()
    again = bcp.Plan.deserialize(image)
    with pytest.raises(bcp.BcpError):
        again.used_sources()
    again.destroy()
