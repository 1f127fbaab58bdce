"""Pins for the CPU oracle: what the paper and plain mathematics fix, never the oracle itself."""
import numpy as np
import pytest

from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import CONFIGS, MIXED, OPTIM_ONLY, PARAMS_ONLY, scenario_cases, small_gpt, small_llama
from workloads.layouts import Parallelism, build_state, reshard_case
from workloads.meta import BOX, FLAT_SLICE, ShardMeta, ShardedState
from workloads.random_cases import random_case

from helpers import brute_force_reshard, np_bufs, read_irregular_example


def filled(case, state, fill=None):
    return np_bufs(fills.fill_state(state, case.key_ids, fill or case.fill, case.seed, "cpu"))


# ---- the paper's worked example (Sec. 3.2, irregular tensor B of shape (3, 2)) -------------
def test_paper_irregular_example():
    shape, recs = read_irregular_example()
    n = int(np.prod(shape))
    full = np.arange(100, 100 + n, dtype=np.uint32)
    # saved side: the two irregular shards, one per rank, each in its own blob
    src = [ShardMeta("B", 4, 2, shape, (0,) * len(shape), shape, r, 0, FLAT_SLICE, a, b) for r, a, b, _ in recs]
    blobs = [full[a:b].copy().view(np.uint8) for _, a, b, _ in recs]
    # wanted side: for every rank the regular boxes the paper's decomposition names, in order
    dst, pos = [], 0
    for r, a, b, boxes in recs:
        for off, ln in boxes:
            m = ShardMeta("B", 4, 2, shape, off, ln, 0, pos)
            dst.append(m)
            pos += m.byte_length
    out = orc.reshard(src, blobs, dst, [pos])[0].view(np.uint32)
    # the boxes of rank r, concatenated in order, are exactly rank r's flat shard
    assert np.array_equal(out, full)
    # and each box holds the elements of the row-major (3, 2) tensor at its coordinates
    T = full.reshape(shape)
    for m in dst:
        sl = tuple(slice(o, o + l) for o, l in zip(m.offsets, m.lengths))
        assert np.array_equal(out[m.byte_offset // 4:m.byte_offset // 4 + m.numel], T[sl].ravel())


# ---- invariants of the representation ---------------------------------------------------------
SMALL = [c for c in scenario_cases()]


@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_identity_reshard(case):
    """Unchanged parallelism returns bit-identical shards (Sec. 6.4: bit-wise resume)."""
    blobs = filled(case, case.src, "uniform")
    out = orc.reshard(case.src.metas, blobs, case.src.metas, case.src.buf_bytes)
    for a, b in zip(out, blobs):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("case", SMALL[:6], ids=lambda c: c.name)
def test_round_trip(case):
    """A -> B -> A gives back A's blobs.  B is the de-duplicated form of the target layout."""
    blobs = filled(case, case.src, "uniform")
    mid = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes)
    # keep one replica of every wanted shard as the saved side of the way back
    seen, uniq = set(), []
    for m in case.dst.metas:
        k = (m.fqn, m.offsets, m.lengths, m.kind, m.flat_begin, m.flat_end)
        if k not in seen:
            seen.add(k)
            uniq.append(m)
    back = orc.reshard(uniq, mid, case.src.metas, case.src.buf_bytes)
    for a, b in zip(back, blobs):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_exact_cover(case):
    """Saved shards tile every global tensor exactly once; wanted shards k times (k replicas)."""
    for fqn, es in orc.group_by_fqn(case.src.metas).items():
        shape, isz = orc.check_family(es)
        _, cover = orc.assemble(shape, isz, es, [np.zeros(e.numel, dtype=orc._UINT[isz]) for e in es])
        assert cover.min() == 1 and cover.max() == 1, fqn
    for fqn, es in orc.group_by_fqn(case.dst.metas).items():
        shape, isz = orc.check_family(es)
        _, cover = orc.assemble(shape, isz, es, [np.zeros(e.numel, dtype=orc._UINT[isz]) for e in es])
        assert cover.min() == cover.max() >= 1, fqn
        assert sum(e.numel for e in es) == int(cover.max()) * int(np.prod(shape, dtype=np.int64))


def test_path_independence():
    """A -> C equals A -> B -> C."""
    g = small_gpt()
    A = build_state(g, Parallelism(tp=2, dp=2, pp=2, zero="zero1"), MIXED, dedup=True)
    B = build_state(g, Parallelism(tp=4, dp=3, pp=1, zero="zero1"), MIXED, dedup=True)
    C = build_state(g, Parallelism(tp=1, dp=5, pp=4, zero="zero1"), MIXED, dedup=False)
    case = reshard_case("x", g, Parallelism(tp=2, dp=2, pp=2, zero="zero1"), Parallelism(), MIXED)
    a = np_bufs(fills.fill_state(A, case.key_ids, "uniform", 3, "cpu"))
    direct = orc.reshard(A.metas, a, C.metas, C.buf_bytes)
    b = orc.reshard(A.metas, a, B.metas, B.buf_bytes)
    via = orc.reshard(B.metas, b, C.metas, C.buf_bytes)
    for x, y in zip(direct, via):
        assert np.array_equal(x, y)


# ---- closed form: the index-pattern fill needs no oracle to predict the target bytes ---------
@pytest.mark.parametrize("case", [CONFIGS["cfg1"]("index")] + SMALL, ids=lambda c: c.name)
def test_index_fill_closed_form(case):
    blobs = filled(case, case.src, "index")
    out = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes)
    want = filled(case, case.dst, "index")
    for a, b in zip(out, want):
        assert np.array_equal(a, b)


def test_cfg1_uniform_matches_generative_fill():
    case = CONFIGS["cfg1"]("uniform")
    blobs = filled(case, case.src)
    out = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes)
    want = filled(case, case.dst)
    for a, b in zip(out, want):
        assert np.array_equal(a, b)


# ---- textbook reductions -------------------------------------------------------------------------
@pytest.mark.parametrize("dim,src_tp,dst_tp", [(0, 4, 2), (1, 2, 8), (0, 8, 1), (1, 1, 4)])
def test_pure_tp_change_is_concatenate_then_split(dim, src_tp, dst_tp):
    rng = np.random.default_rng(5)
    shape = (48, 32)
    full = rng.integers(0, 2 ** 16, size=shape, dtype=np.uint16)

    def side(tp):
        metas, blobs = [], []
        for r, piece in enumerate(np.split(full, tp, axis=dim)):
            off = tuple((r * shape[d] // tp) if d == dim else 0 for d in range(2))
            metas.append(ShardMeta("w", 2, 1, shape, off, piece.shape, r, 0))
            blobs.append(np.ascontiguousarray(piece).reshape(-1).view(np.uint8))
        return metas, blobs

    sm, sb = side(src_tp)
    dm, db = side(dst_tp)
    # library routine: np.concatenate(shards, axis) then np.split -> db by construction
    assert np.array_equal(np.concatenate([b.view(np.uint16).reshape(m.lengths) for m, b in zip(sm, sb)], axis=dim), full)
    out = orc.reshard(sm, sb, dm, [b.size for b in db])
    for a, b in zip(out, db):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("src_dp,dst_dp", [(4, 3), (3, 8), (75, 150), (8, 6)])
def test_pure_zero_dp_change_is_ravel_concat_then_even_split(src_dp, dst_dp):
    rng = np.random.default_rng(9)
    shapes = [(7, 5), (11,), (3, 4, 5), (6, 6)]
    tensors = [rng.integers(0, 2 ** 32, size=s, dtype=np.uint32) for s in shapes]
    flat = np.concatenate([t.ravel() for t in tensors])

    def side(dp):
        S = -(-flat.size // dp)
        metas, blobs = [], []
        for r in range(dp):
            lo, hi = r * S, min((r + 1) * S, flat.size)
            blobs.append(flat[lo:max(lo, hi)].copy().view(np.uint8))
            pos = 0
            for i, t in enumerate(tensors):
                a, b = max(lo, pos), min(hi, pos + t.size)
                if b > a:
                    metas.append(ShardMeta(f"t{i}", 4, 2, t.shape, (0,) * t.ndim, t.shape, r, (a - lo) * 4,
                                           FLAT_SLICE, a - pos, b - pos))
                pos += t.size
        return metas, blobs

    sm, sb = side(src_dp)
    dm, db = side(dst_dp)
    out = orc.reshard(sm, sb, dm, [b.size for b in db])
    for a, b in zip(out, db):
        assert np.array_equal(a, b)


# ---- brute force on tiny inputs ---------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(40))
def test_brute_force_tiny(seed):
    case = random_case(seed, dst_replicas=1 + seed % 2)
    blobs = filled(case, case.src, "index")
    want = brute_force_reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, 0xA5)
    got = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, 0xA5)
    for a, b in zip(got, want):
        assert np.array_equal(a, b)


# ---- degenerate cases -----------------------------------------------------------------------------
def test_scalar_and_empty_entries():
    s = [ShardMeta("s", 8, 4, (), (), (), 0, 8), ShardMeta("e", 4, 2, (4, 0), (0, 0), (4, 0), 0, 0)]
    d = [ShardMeta("s", 8, 4, (), (), (), 0, 0), ShardMeta("e", 4, 2, (4, 0), (1, 0), (2, 0), 0, 8)]
    blob = np.arange(16, dtype=np.uint8)
    out = orc.reshard(s, [blob], d, [8])
    assert np.array_equal(out[0], blob[8:16])


def test_uncovered_and_overlap_are_errors():
    s = [ShardMeta("w", 4, 2, (4,), (0,), (2,), 0, 0)]
    d = [ShardMeta("w", 4, 2, (4,), (1,), (2,), 0, 0)]
    with pytest.raises(orc.OracleError):
        orc.reshard(s, [np.zeros(8, np.uint8)], d, [8])
    s2 = [ShardMeta("w", 4, 2, (4,), (0,), (3,), 0, 0), ShardMeta("w", 4, 2, (4,), (2,), (2,), 0, 12)]
    with pytest.raises(orc.OracleError):
        orc.reshard(s2, [np.zeros(20, np.uint8)], d, [8])
    s3 = [ShardMeta("w", 4, 2, (4,), (0,), (4,), 0, 0), ShardMeta("w", 2, 1, (4,), (0,), (0,), 0, 0)]
    with pytest.raises(orc.OracleError):
        orc.reshard(s3, [np.zeros(16, np.uint8)], d, [8])


# ---- pack / unpack -----------------------------------------------------------------------------------
def test_pack_is_join_with_zero_padding():
    rng = np.random.default_rng(1)
    sizes = [1, 255, 256, 257, 4096, 3, 0, 1000]
    ts = [rng.integers(1, 256, size=n, dtype=np.uint8) for n in sizes]
    for align in (16, 256, 4096):
        blob, table = orc.pack(ts, align)
        ref = b"".join(t.tobytes() + b"\0" * (-len(t) % align) for t in ts)
        # an empty tensor adds nothing; the join above pads it with zero bytes of length 0
        assert blob.tobytes() == ref
        offs, total = orc.pack_layout(sizes, align)
        assert offs == [o for o, _ in table] and total == len(ref)
        assert all(o % align == 0 for o in offs)
        assert offs == list(np.cumsum([0] + [-(-n // align) * align for n in sizes[:-1]]))
        back = orc.unpack(blob, table)
        assert all(np.array_equal(a, b) for a, b in zip(back, ts))


# ---- element conversion (extension; the paper moves bytes only) ----------------------------------
def _conversion_examples():
    import os

    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "f32_to_bf16_examples.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    return [(int(r[0], 16), int(r[1], 16)) for r in rows]


def test_conversion_hand_worked_examples():
    ex = _conversion_examples()
    assert len(ex) >= 20
    got = orc.f32_to_bf16(np.array([a for a, _ in ex], dtype=np.uint32))
    assert [int(g) for g in got] == [b for _, b in ex]
    # widening appends sixteen zero bits
    assert [int(x) for x in orc.bf16_to_f32(np.array([0x3F80, 0xC049, 0x0001, 0x7FC0, 0xFFFF], dtype=np.uint16))] == [
        0x3F800000, 0xC0490000, 0x00010000, 0x7FC00000, 0xFFFF0000]


def _patterns():
    rng = np.random.default_rng(11)
    sweep = np.arange(0, 1 << 32, 16381, dtype=np.uint64).astype(np.uint32)  # every exponent, both signs
    ties = (np.arange(0, 1 << 16, dtype=np.uint64) << 16 | 0x8000).astype(np.uint32)  # every halfway point
    return np.concatenate([rng.integers(0, 1 << 32, 400_000, dtype=np.uint64).astype(np.uint32), sweep, ties, ties - 1, ties + 1])


def test_conversion_agrees_with_the_library_cast():
    """torch's own binary32 -> bfloat16 cast on everything but NaN (NaN encodings are not fixed by IEEE 754)."""
    import torch

    bits = _patterns()
    bits = bits[(bits & 0x7FFFFFFF) <= 0x7F800000]
    lib = torch.from_numpy(bits.view(np.float32).copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.f32_to_bf16(bits), lib)
    back = torch.from_numpy(lib.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy().view(np.uint32)
    assert np.array_equal(orc.bf16_to_f32(lib), back)


def test_conversion_error_bound_fixed_points_and_order():
    bits = _patterns()
    finite = bits[(bits & 0x7FFFFFFF) < 0x7F800000]
    out = orc.f32_to_bf16(finite)
    x = finite.view(np.float32).astype(np.float64)
    with np.errstate(over="ignore"):
        y = orc.bf16_to_f32(out).view(np.float32).astype(np.float64)
    # half a unit in the last place of the result: 2^-8 relative for normal numbers, 2^-134 absolute below
    ok = np.isfinite(y)
    assert np.all(np.abs(y[ok] - x[ok]) <= np.maximum(np.abs(x[ok]) * 2.0 ** -8, 2.0 ** -134))
    assert np.all(np.abs(x[~ok]) >= (2.0 - 2.0 ** -8) * 2.0 ** 127)  # only values past the last halfway point overflow
    assert np.all((y == 0) | (np.sign(y) == np.sign(x)))
    # every bfloat16 is a fixed point (all 65,536 patterns but the NaNs)
    h = np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)
    h = h[(h & 0x7FFF) <= 0x7F80]
    assert np.array_equal(orc.f32_to_bf16(orc.bf16_to_f32(h)), h)
    # rounding never reverses the order of two values
    pos = np.sort(finite[finite < 0x7F800000])
    assert np.all(np.diff(orc.f32_to_bf16(pos).astype(np.int64)) >= 0)
    # NaNs: one canonical pattern
    assert set(orc.f32_to_bf16(np.array([0x7F800001, 0x7FFFFFFF, 0xFFC00000, 0xFF800001], dtype=np.uint32)).tolist()) == {0x7FC0}


def test_conversion_commutes_with_resharding():
    """Converting reshard == plain reshard of the saved type into the wanted layout, then the library cast,
    element by element (no NaN in this fill)."""
    import torch
    from workloads.configs import convert_cases
    from workloads.meta import DTYPE_BF16, DTYPE_F32

    for case in convert_cases():
        blobs = filled(case, case.src, "uniform")
        got = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, convert=case.convert)
        narrow = case.convert[0] == orc.F32_TO_BF16
        # the same wanted boxes in the saved type, packed back to back
        same, pos = [], 0
        for m in case.dst.metas:
            k = ShardMeta(m.fqn, 4 if narrow else 2, DTYPE_F32 if narrow else DTYPE_BF16, m.global_shape, m.offsets, m.lengths,
                          0, pos, m.kind, m.flat_begin, m.flat_end)
            same.append(k)
            pos += k.byte_length
        plain = orc.reshard(case.src.metas, blobs, same, [pos])[0]
        for m, k in zip(case.dst.metas, same):
            raw = plain[k.byte_offset:k.byte_offset + k.byte_length]
            if narrow:
                want = torch.from_numpy(raw.view(np.float32).copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint8)
            else:
                want = torch.from_numpy(raw.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy().view(np.uint8)
            assert np.array_equal(got[m.buf_index][m.byte_offset:m.byte_offset + m.byte_length], want), (case.name, m.fqn)


# ---- replicated saved shards: the first entry in input order wins --------------------------------
def _with_replicas(case, rng):
    """Every saved entry of `case`, plus copies of about half of them in a new blob holding OTHER
    bytes, inserted at random places of the entry list (so that who comes first varies)."""
    import copy

    metas = list(case.src.metas)
    extra, pos = [], 0
    for m in case.src.metas:
        if m.byte_length and rng.random() < 0.5:
            k = copy.copy(m)
            k.buf_index, k.byte_offset = len(case.src.buf_bytes), pos
            pos += m.byte_length + int(rng.integers(0, 3)) * m.itemsize
            extra.append(k)
    for k in extra:
        metas.insert(int(rng.integers(0, len(metas) + 1)), k)
    return metas, list(case.src.buf_bytes) + [max(pos, 1)], len(extra)


@pytest.mark.parametrize("seed", range(24))
def test_first_replica_wins_against_brute_force(seed):
    """Random tiny problems whose saved side stores some shards twice with different bytes: the
    oracle's first-wins rule (assign last to first) against the element-by-element mapper that
    takes the first saved entry, in input order, holding each wanted element."""
    rng = np.random.default_rng(1000 + seed)
    case = random_case(seed, n_tensors=3, max_dim=5, dst_replicas=1 + seed % 2)
    metas, sizes, n_extra = _with_replicas(case, rng)
    blobs = [rng.integers(0, 256, size=n, dtype=np.uint8) for n in sizes]
    want = brute_force_reshard(metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, first_wins=True)
    got = orc.reshard(metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, allow_replicas=True)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    if n_extra:  # without the permission the same input is an error
        with pytest.raises(orc.OracleError):
            orc.reshard(metas, blobs, case.dst.metas, case.dst.buf_bytes)


def test_partly_overlapping_saved_shards_are_an_error_even_with_replicas_allowed():
    from workloads.meta import ShardMeta

    whole = ShardMeta("x", 1, 3, (4, 4), (0, 0), (4, 4), 0, 0)
    a = ShardMeta("x", 1, 3, (4, 4), (0, 0), (3, 4), 0, 0)
    b = ShardMeta("x", 1, 3, (4, 4), (2, 0), (2, 4), 0, 16)   # shares row 2 with a
    blob = np.arange(32, dtype=np.uint8)
    for allow in (False, True):
        with pytest.raises(orc.OracleError):
            orc.reshard([a, b], [blob], [whole], [16], allow_replicas=allow)
    # a flat slice and a box that share some but not all of their elements
    f = ShardMeta("x", 1, 3, (4, 4), (0, 0), (4, 4), 0, 0, kind=1, flat_begin=2, flat_end=10)
    with pytest.raises(orc.OracleError):
        orc.reshard([f, a], [blob], [ShardMeta("x", 1, 3, (4, 4), (0, 2), (1, 2), 0, 0)], [2], allow_replicas=True)
