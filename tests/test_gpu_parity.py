"""Parity of the CUDA path against the CPU oracle, through the C ABI, on a real GPU.

Small cases are compared byte by byte over whole buffers (with guard bands and a poison fill
around and between the named bytes).  The five full-size configurations run in the launch
configuration the benchmark times; every target byte is checked against the closed-form
index-pattern fill (a property that needs no oracle) and a sample of FQNs is pushed through
the oracle element by element.
"""
import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import api
from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import CONFIGS, STRESS, convert_cases, scenario_cases
from workloads.meta import ShardMeta
from workloads.random_cases import big_random_case, many_tiny_case, random_case

pytestmark = pytest.mark.gpu
GUARD = 4096
POISON = 0xA5


def guarded(sizes, device, poison=POISON):
    """Buffers with a poisoned guard band on both sides; returns (views, backing tensors)."""
    backs = [torch.full((n + 2 * GUARD,), poison, dtype=torch.uint8, device=device) for n in sizes]
    return [b[GUARD:GUARD + n] for b, n in zip(backs, sizes)], backs


def guards_intact(backs, sizes, poison=POISON):
    return all(bool((b[:GUARD] == poison).all()) and bool((b[GUARD + n:] == poison).all()) for b, n in zip(backs, sizes))


def run_and_compare(case, device, fill="index", runs=1, stream=None, **opts):
    src = fills.fill_state(case.src, case.key_ids, fill, case.seed, device, poison=0x5A)
    want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON,
                       convert=case.convert)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts, **case.plan_opts)
    for _ in range(runs):
        dst, backs = guarded(case.dst.buf_bytes, device)
        bcp.bcp_reshard(plan, src, dst, stream=stream)
        (stream or torch.cuda.current_stream()).synchronize()
        bcp.bcp_plan_device_status(plan)
        for i, (d, w) in enumerate(zip(dst, want)):
            got = d.cpu().numpy()
            if not np.array_equal(got, w):
                bad = np.flatnonzero(got != w)
                pytest.fail(f"{case.name}: buffer {i} differs at {bad.size} bytes, first at {bad[0]} "
                            f"(got {got[bad[0]]}, want {w[bad[0]]})")
        assert guards_intact(backs, case.dst.buf_bytes), "write outside the target buffer"
    st = plan.stats()
    plan.destroy()
    return st


# ---- small cases, whole buffers ------------------------------------------------------------------
@pytest.mark.parametrize("fill", ["uniform", "index"])
def test_cfg1(cuda_device, fill):
    st = run_and_compare(CONFIGS["cfg1"](fill), cuda_device, fill, runs=3)
    assert st["bytes_copied"] == 37_498_880


@pytest.mark.parametrize("case", scenario_cases(), ids=lambda c: c.name)
def test_scenarios(cuda_device, case):
    run_and_compare(case, cuda_device)


@pytest.mark.parametrize("seed", range(24))
def test_random_tiny(cuda_device, seed):
    run_and_compare(random_case(seed, dst_replicas=1 + seed % 2), cuda_device, tile_bytes=4096,
                    small_bytes=64 if seed % 3 else 4096)


@pytest.mark.parametrize("path_mask", [1, 3])
@pytest.mark.parametrize("itemsize,seed", [(1, 1), (2, 2), (4, 3), (8, 4), (2, 5), (4, 6)])
def test_big_random_misaligned(cuda_device, itemsize, seed, path_mask):
    """Odd shapes and byte offsets: every access width from 1 to 16 bytes, ragged heads and tails,
    through the register kernel and through the shifted-run staging of the TMA kernel."""
    st = run_and_compare(big_random_case(seed, itemsize=itemsize), cuda_device, tile_bytes=8192 if seed % 2 else 65536,
                         path_mask=path_mask, tma_stage_bytes=4096 if seed % 3 == 0 else 32768)
    assert st["bytes_misaligned"] > 0
    assert (st["n_tma_tiles"] > 0) == (path_mask == 3)


@pytest.mark.parametrize("opts", [dict(block_threads=256, ctas_per_sm=4), dict(block_threads=1024, ctas_per_sm=1),
                                  dict(tile_bytes=4096), dict(tile_bytes=1 << 20, small_bytes=1 << 16),
                                  dict(cache_hints=2), dict(order=2), dict(unroll=8), dict(path_mask=1, worker=2),
                                  dict(path_mask=1, worker=2, unroll=8, ctas_per_sm=4, tile_bytes=16384),
                                  dict(path_mask=3), dict(path_mask=3, tma_stage_bytes=4096, tma_stages=2, tile_bytes=32768),
                                  dict(path_mask=3, tma_stage_bytes=32768, tma_stages=6, tma_ctas_per_sm=1),
                                  dict(path_mask=7), dict(path_mask=7, tile_bytes=8192, tma_stage_bytes=4096),
                                  dict(path_mask=7, fanout=2), dict(path_mask=3, fanout=1, tile_bytes=4096, tma_stage_bytes=2048, tma_stages=2)])
def test_launch_options(cuda_device, opts):
    run_and_compare(CONFIGS["cfg1"]("index"), cuda_device, **opts)
    run_and_compare(big_random_case(11, itemsize=2), cuda_device, **opts)


def _dim1_split_case(shape, isz, src_parts, dst_parts):
    from workloads.layouts import ReshardCase
    from workloads.meta import ShardedState

    def side(parts):
        metas, sizes = [], []
        for r in range(parts):
            b, e = shape[1] * r // parts, shape[1] * (r + 1) // parts
            metas.append(ShardMeta("w", isz, isz, shape, (0, b), (shape[0], e - b), r, 256))
            sizes.append(256 + shape[0] * (e - b) * isz + 256)
        return ShardedState(metas, sizes)

    return ReshardCase(f"dim1-{src_parts}-to-{dst_parts}", side(src_parts), side(dst_parts), "index", 1)


@pytest.mark.parametrize("opts", [dict(path_mask=3), dict(path_mask=3, tma_stage_bytes=4096, tma_stages=3),
                                  dict(path_mask=3, tma_stage_bytes=2048, tma_stages=8, tma_ctas_per_sm=6, tile_bytes=16384),
                                  dict(path_mask=1, unroll=8), dict(path_mask=7), dict(path_mask=7, tma_stage_bytes=16384, tile_bytes=32768)])
def test_wide_strided_rows(cuda_device, opts):
    """Strided rectangles with rows of 4-12 KiB (longer than a small TMA stage) and of 512 B."""
    run_and_compare(_dim1_split_case((96, 6144), 4, 2, 3), cuda_device, runs=2, **opts)
    run_and_compare(_dim1_split_case((1000, 1024), 2, 4, 1), cuda_device, **opts)
    run_and_compare(_dim1_split_case((333, 4096), 2, 1, 8), cuda_device, **opts)
    run_and_compare(_dim1_split_case((5003, 256), 2, 2, 4), cuda_device, runs=2, **opts)   # 128-byte rows, ragged last box
    run_and_compare(_dim1_split_case((777, 1032), 4, 3, 1), cuda_device, **opts)           # rows of 1376 bytes


@pytest.mark.parametrize("case", scenario_cases()[:4] + scenario_cases()[8:10], ids=lambda c: c.name)
def test_scenarios_tma_path(cuda_device, case):
    run_and_compare(case, cuda_device, path_mask=3, tile_bytes=16384, tma_stage_bytes=4096)
    run_and_compare(case, cuda_device, path_mask=7, tile_bytes=8192, tma_min_row_bytes=64, fanout=1)


def test_plans_with_different_ring_sizes_interleave(cuda_device):
    """The TMA kernel's shared-memory ring is sized per plan; executions of plans with large and
    small rings may alternate in any order."""
    case = scenario_cases()[3]
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device)
    want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    big = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3,
                       tma_stage_bytes=32768, tma_stages=6, tile_bytes=16384)
    small = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3,
                         tma_stage_bytes=2048, tma_stages=2, tile_bytes=16384)
    for plan in (big, small, big, small, big):
        dst, backs = guarded(case.dst.buf_bytes, cuda_device)
        bcp.bcp_reshard(plan, src, dst)
        torch.cuda.synchronize()
        assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)) and guards_intact(backs, case.dst.buf_bytes)


def test_bounded_wait_runs_out_and_is_reported(cuda_device):
    """Failure detection without a fault: a test hook arms one stage of one CTA for bytes that
    never arrive; that CTA's bounded wait gives up after 20 ms, the kernel ends, the status call
    reports BCP_ERR_DEVICE_TIMEOUT, and the context and the library stay usable."""
    from paper_2407_20143_b200 import api

    case = _dim1_split_case((4096, 8192), 2, 1, 1)  # 64 MB, all aligned runs
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device)
    want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    stalled = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3,
                           test_stall=1, tma_wait_ms=20)
    dst, _ = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(stalled, src, dst)
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_plan_device_status(stalled)
    assert e.value.code == api.ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()  # no sticky error: the kernel returned normally
    got = dst[0].cpu().numpy()
    missing = int((got != want[0]).sum())
    assert 0 < missing <= 2 * 65536 + 32768, "only the unit the stalled CTA held may be incomplete"
    bcp.bcp_plan_device_status(stalled)  # the status word was cleared by the report
    # an ordinary plan on the same device right afterwards is exact
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3)
    dst2, backs = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(plan, src, dst2)
    torch.cuda.synchronize()
    bcp.bcp_plan_device_status(plan)
    assert np.array_equal(dst2[0].cpu().numpy(), want[0]) and guards_intact(backs, case.dst.buf_bytes)


def test_bounded_wait_of_the_staged_converting_kernel(cuda_device):
    """The same for the staged converting kernel: one over-armed stage, a 20 ms wait that runs out, the status
    word, and an exact converting plan on the same device right afterwards."""
    case = convert_cases()[1]
    host = fills.fill_state(case.src, case.key_ids, "uniform", case.seed, "cpu")
    want = orc.reshard(case.src.metas, [h.numpy() for h in host], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON, convert=case.convert)
    src = [h.to(cuda_device) for h in host]
    opts = dict(case.plan_opts, path_mask=3, tma_min_row_bytes=16)
    stalled = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, test_stall=1, tma_wait_ms=20, **opts)
    assert any(t.flags & api.TILE_TMA and t.flags & api.TILE_CVT_MASK for t in stalled.tiles())
    dst, _ = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(stalled, src, dst)
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_plan_device_status(stalled)
    assert e.value.code == api.ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()  # no sticky error: the kernel returned normally
    assert any(not np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)), "the stalled CTA's unit stays incomplete"
    bcp.bcp_plan_device_status(stalled)
    stalled.destroy()
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts)
    dst2, backs = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(plan, src, dst2)
    torch.cuda.synchronize()
    bcp.bcp_plan_device_status(plan)
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst2, want)) and guards_intact(backs, case.dst.buf_bytes)
    plan.destroy()


def test_side_stream_and_plan_reuse(cuda_device):
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        run_and_compare(scenario_cases()[3], cuda_device, runs=4, stream=s)


@pytest.mark.parametrize("seed", range(100, 106))
def test_random_up_to_eight_dims(cuda_device, seed):
    run_and_compare(random_case(seed, n_tensors=3, max_ndim=8, max_dim=3, dst_replicas=1 + seed % 2), cuda_device,
                    tile_bytes=4096)


def test_hundred_thousand_tiny_tensors(cuda_device):
    case = many_tiny_case(100_000)
    g = torch.Generator(device="cpu").manual_seed(11)
    host = [torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g) for n in case.src.buf_bytes]
    want = orc.reshard(case.src.metas, [h.numpy() for h in host], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    st = plan.stats()
    assert st["n_fqns"] == 100_000 and st["n_small_tiles"] > 50_000 and st["plan_ms"] < 5000
    dst, backs = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(plan, [h.to(cuda_device) for h in host], dst)
    torch.cuda.synchronize()
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)) and guards_intact(backs, case.dst.buf_bytes)


def test_replicated_saved_side(cuda_device):
    """A checkpoint written without de-duplication: replicas allowed, the first one is read."""
    from workloads.configs import MIXED, small_gpt
    from workloads.layouts import Parallelism, ReshardCase, build_state

    g = small_gpt()
    case = ReshardCase("replicated-source", build_state(g, Parallelism(tp=2, dp=2, pp=2, zero="zero1"), MIXED, dedup=False),
                       build_state(g, Parallelism(tp=1, dp=3, pp=4, zero="zero1"), MIXED, dedup=False), "index", 5)
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device)
    want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON,
                       allow_replicas=True)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, allow_replicas=1)
    dst, backs = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(plan, src, dst)
    torch.cuda.synchronize()
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)) and guards_intact(backs, case.dst.buf_bytes)


def test_deserialized_plan_executes(cuda_device):
    """A plan image written by one plan object runs identically when rebuilt (plan cache)."""
    case = CONFIGS["cfg1"]("index")
    first = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3)
    plan = bcp.Plan.deserialize(first.serialize())
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device)
    dst, backs = guarded(case.dst.buf_bytes, cuda_device)
    bcp.bcp_reshard(plan, src, dst)
    torch.cuda.synchronize()
    want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)) and guards_intact(backs, case.dst.buf_bytes)


def test_degenerate_entries(cuda_device):
    src_m = [ShardMeta("s", 8, 4, (), (), (), 0, 16), ShardMeta("e", 4, 2, (4, 0), (0, 0), (4, 0), 0, 0),
             ShardMeta("one", 1, 3, (1,), (0,), (1,), 0, 31)]
    dst_m = [ShardMeta("s", 8, 4, (), (), (), 0, 0), ShardMeta("e", 4, 2, (4, 0), (1, 0), (2, 0), 0, 8),
             ShardMeta("one", 1, 3, (1,), (0,), (1,), 1, 5)]
    src = [torch.arange(32, dtype=torch.uint8, device=cuda_device)]
    plan = bcp.bcp_plan(src_m, [32], dst_m, [16, 16])
    dst, backs = guarded([16, 16], cuda_device)
    bcp.bcp_reshard(plan, src, dst)
    torch.cuda.synchronize()
    want = orc.reshard(src_m, [src[0].cpu().numpy()], dst_m, [16, 16], fill_byte=POISON)
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)) and guards_intact(backs, [16, 16])
    # a plan with no work at all is legal and launches nothing
    empty = bcp.bcp_plan([], [], [], [])
    bcp.bcp_reshard(empty, [], [])


def test_execution_errors(cuda_device):
    case = scenario_cases()[0]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    src = fills.make_buffers(case.src, cuda_device)
    dst = fills.make_buffers(case.dst, cuda_device)
    with pytest.raises(bcp.BcpError):
        bcp.bcp_reshard(plan, src[:-1], dst)
    with pytest.raises(bcp.BcpError):
        bcp.bcp_reshard(plan, src, [d.data_ptr() + 4 for d in dst])  # misaligned base
    bcp.bcp_reshard(plan, src, dst)  # the plan is still usable
    torch.cuda.synchronize()


def test_reshard_host(cuda_device):
    case = CONFIGS["cfg1"]("uniform")
    src = [s.pin_memory() for s in fills.fill_state(case.src, case.key_ids, "uniform", 0, "cpu")]
    dst = [torch.full((n,), POISON, dtype=torch.uint8).pin_memory() for n in case.dst.buf_bytes]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    for _ in range(2):
        bcp.bcp_reshard_host(plan, src, dst)
        want = orc.reshard(case.src.metas, [s.numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=0)
        assert all(np.array_equal(d.numpy(), w) for d, w in zip(dst, want))


@pytest.mark.parametrize("name", ["dp150-to-dp75", "hybrid", "llama-tp8-to-tp2"])
def test_reshard_host_scenarios(cuda_device, name):
    """Host-buffer path on layouts with many buffers (600 saved ranks, two of them empty), replicas
    and strided pieces; pageable host memory works too, pinned is only faster."""
    case = [c for c in scenario_cases() if c.name == name][0]
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu")
    dst = [torch.full((n,), POISON, dtype=torch.uint8) for n in case.dst.buf_bytes]
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    bcp.bcp_reshard_host(plan, [s.data_ptr() if s.numel() else 0 for s in src], [d.data_ptr() if d.numel() else 0 for d in dst])
    want = orc.reshard(case.src.metas, [s.numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=0)
    assert all(np.array_equal(d.numpy(), w) for d, w in zip(dst, want))
    # the same plan still serves device buffers afterwards
    dsrc = [s.to(cuda_device) for s in src]
    ddst = [torch.zeros(n, dtype=torch.uint8, device=cuda_device) for n in case.dst.buf_bytes]
    bcp.bcp_reshard(plan, [s.data_ptr() if s.numel() else 0 for s in dsrc], [d.data_ptr() if d.numel() else 0 for d in ddst])
    torch.cuda.synchronize()
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(ddst, want))


# ---- pack / unpack ---------------------------------------------------------------------------------
def _pack_check(device, sizes, align, offsets=None, misalign=0):
    g = torch.Generator(device="cpu").manual_seed(len(sizes) * 7919 + align + misalign)
    host = [torch.randint(1, 256, (n,), dtype=torch.uint8, generator=g) for n in sizes]
    if misalign:  # tensors that start at odd addresses inside a larger allocation
        backing = [torch.zeros(n + 64, dtype=torch.uint8, device=device) for n in sizes]
        dev = [b[(misalign * (i + 1)) % 61:][:n] for i, (b, n) in enumerate(zip(backing, sizes))]
        for d, h in zip(dev, host):
            d.copy_(h)
    else:
        dev = [h.to(device) for h in host]
    offs, total = bcp.bcp_pack_layout(sizes, align)
    want, table = orc.pack([h.numpy() for h in host], align)
    assert total == want.size and offs == [o for o, _ in table]
    metas = list(zip(offs, sizes))
    blob_back = torch.full((total + 2 * GUARD + 16,), POISON, dtype=torch.uint8, device=device)
    blob = blob_back[GUARD + misalign % 16:][:total]
    for _ in range(2):
        bcp.bcp_pack(dev, metas, blob)
        torch.cuda.synchronize()
        assert np.array_equal(blob.cpu().numpy(), want)
    assert bool((blob_back[:GUARD + misalign % 16] == POISON).all()) and bool((blob_back[GUARD + misalign % 16 + total:] == POISON).all())
    out = [torch.full((n,), POISON, dtype=torch.uint8, device=device) for n in sizes]
    bcp.bcp_unpack(blob, metas, out)
    torch.cuda.synchronize()
    for o, h, w in zip(out, host, orc.unpack(want, table)):
        assert np.array_equal(o.cpu().numpy(), w) and np.array_equal(w, h.numpy())


def test_pack_unpack_small(cuda_device):
    _pack_check(cuda_device, [1, 255, 256, 257, 4096, 3, 0, 1000, 70_001, 16, 300_000], 256)
    _pack_check(cuda_device, [5_000_000, 17, 1 << 20, 999_999], 4096)
    _pack_check(cuda_device, [], 256)
    _pack_check(cuda_device, [7, 9, 100_003, 65536], 16, misalign=3)
    bcp.bcp_pack_cache_clear()


def test_pack_rejects_bad_tables(cuda_device):
    t = [torch.zeros(100, dtype=torch.uint8, device=cuda_device) for _ in range(2)]
    blob = torch.zeros(512, dtype=torch.uint8, device=cuda_device)
    with pytest.raises(bcp.BcpError):
        bcp.bcp_pack(t, [(0, 100), (50, 100)], blob)  # overlap
    with pytest.raises(bcp.BcpError):
        bcp.bcp_pack(t, [(0, 100), (450, 100)], blob)  # past the end


def test_reshard_then_pack_small_moe(cuda_device):
    """EP8 -> EP4 on a small MoE, then every target rank's tensors packed into one blob."""
    case = [c for c in scenario_cases() if c.name == "moe-ep8-to-ep4"][0]
    src = fills.fill_state(case.src, case.key_ids, "uniform", case.seed, cuda_device)
    dst = fills.make_buffers(case.dst, cuda_device, POISON)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    bcp.bcp_reshard(plan, src, dst)
    want_dst = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, POISON)
    for r in range(len(dst)):
        ms = [m for m in case.dst.metas if m.buf_index == r]
        sizes = [m.byte_length for m in ms]
        offs, total = bcp.bcp_pack_layout(sizes, 256)
        blob = torch.full((total,), POISON, dtype=torch.uint8, device=cuda_device)
        bcp.bcp_pack([dst[r].data_ptr() + m.byte_offset for m in ms], list(zip(offs, sizes)), blob)
        torch.cuda.synchronize()
        want_blob, _ = orc.pack([want_dst[r][m.byte_offset:m.byte_offset + m.byte_length] for m in ms], 256)
        assert np.array_equal(blob.cpu().numpy(), want_blob)


# ---- the five configurations at full size -------------------------------------------------------------
def _sample_fqns(case, k):
    names = sorted({m.fqn for m in case.dst.metas})
    # one name of every tensor kind first (the last two dotted components), then evenly spaced ones
    kinds, picked = set(), []
    for n in names:
        kind = ".".join(n.split(".")[-2:])
        if kind not in kinds:
            kinds.add(kind)
            picked.append(n)
    step = max(1, len(names) // k)
    picked += names[::step]
    return list(dict.fromkeys(picked))


def _free_gb():
    import gc

    gc.collect()
    torch.cuda.empty_cache()  # memory cached by earlier tests counts as free
    free, _ = torch.cuda.mem_get_info()
    return free / 1e9


@pytest.mark.parametrize("name,max_fqn_bytes", [("cfg2", 450e6), ("cfg3", 1.2e9), ("cfg4", 0.5e9), ("cfg5", 300e6),
                                                ("cfg4odd", 0.5e9), ("narrow", 0.6e9), ("oddgpt", 0.6e9), ("evalmerge", 1.2e9)])
def test_full_size_config(cuda_device, name, max_fqn_bytes):
    case = (CONFIGS.get(name) or STRESS[name])()
    need = (sum(case.src.buf_bytes) + sum(case.dst.buf_bytes)) / 1e9 + 8
    assert _free_gb() > need, f"{name} needs {need:.0f} GB of device memory"
    keys = case.key_ids
    # closed form of the expected target bytes: the index pattern for plain copies; for a narrowing
    # conversion the value fills, whose bfloat16 form is the rounded binary32 form of the same pool
    fill = "normal" if case.convert else "index"
    src = fills.fill_state(case.src, keys, fill, case.seed, cuda_device, poison=0x5A)
    dst = fills.make_buffers(case.dst, cuda_device, POISON)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **case.plan_opts)  # bench defaults
    bcp.bcp_reshard(plan, src, dst)
    torch.cuda.synchronize()
    bcp.bcp_plan_device_status(plan)
    # (1) property at full size: every named target byte equals the closed-form fill of its
    #     global index; every other byte kept the poison
    named = 0
    for m in case.dst.metas:
        n = m.numel
        for lo in range(0, n, 1 << 26):
            hi = min(n, lo + (1 << 26))
            want = fills.entry_bytes(m, keys[m.fqn], fill, case.seed, cuda_device, lo, hi)
            b = m.byte_offset + lo * m.itemsize
            got = dst[m.buf_index][b:b + (hi - lo) * m.itemsize]
            if not torch.equal(got, want):
                bad = int((got != want).nonzero()[0])
                pytest.fail(f"{name} {m.fqn}: target rank {m.buf_index} differs at byte {b + bad}")
        named += m.byte_length
    assert named == case.dst.total_bytes
    # padding between entries kept the poison
    for r, d in enumerate(dst):
        end = 0
        for m in sorted((m for m in case.dst.metas if m.buf_index == r), key=lambda m: m.byte_offset):
            if m.byte_offset > end:
                assert bool((d[end:m.byte_offset] == POISON).all()), f"{name}: padding of rank {r} overwritten"
            end = max(end, m.byte_offset + m.byte_length)
        assert bool((d[end:] == POISON).all())
    # (2) oracle, element by element, on a sample of FQNs
    by_src, by_dst = orc.group_by_fqn(case.src.metas), orc.group_by_fqn(case.dst.metas)
    checked = 0
    for fqn in _sample_fqns(case, 10):
        ss, ds = by_src[fqn], by_dst[fqn]
        if sum(s.byte_length for s in ss) > max_fqn_bytes:
            continue
        payloads = [src[s.buf_index][s.byte_offset:s.byte_offset + s.byte_length].cpu().numpy().view(orc._UINT[s.itemsize]) for s in ss]
        for d, w in zip(ds, orc.reshard_fqn(ss, payloads, ds, convert=case.convert)):
            got = dst[d.buf_index][d.byte_offset:d.byte_offset + d.byte_length].cpu().numpy()
            assert np.array_equal(got, w), f"{name} {fqn}: oracle mismatch on target rank {d.buf_index}"
            checked += d.byte_length
    assert checked > 0
    plan.destroy()
    if name == "cfg5":
        _pack_full_rank(case, dst, cuda_device)


def _pack_full_rank(case, dst, device):
    """cfg5: pack one target rank's 1,766 tensors (15.7 GB) into a blob with an offset table."""
    r = len(dst) - 1
    ms = [m for m in case.dst.metas if m.buf_index == r]
    sizes = [m.byte_length for m in ms]
    offs, total = bcp.bcp_pack_layout(sizes, 256)
    assert (offs, total) == orc.pack_layout(sizes, 256)
    blob = torch.full((total,), POISON, dtype=torch.uint8, device=device)
    ptrs = [dst[r].data_ptr() + m.byte_offset for m in ms]
    bcp.bcp_pack(ptrs, list(zip(offs, sizes)), blob)
    torch.cuda.synchronize()
    end = 0
    for m, o in zip(ms, offs):
        assert not bool(blob[end:o].any()), "padding must be zero"
        assert torch.equal(blob[o:o + m.byte_length], dst[r][m.byte_offset:m.byte_offset + m.byte_length])
        end = o + m.byte_length
    assert not bool(blob[end:].any())
    # oracle on the first 64 tensors as one blob ...
    k = 64
    want, _ = orc.pack([dst[r][m.byte_offset:m.byte_offset + m.byte_length].cpu().numpy() for m in ms[:k]], 256)
    assert np.array_equal(blob[:offs[k]].cpu().numpy()[:want.size], want)
    # ... and on a spread sample (first, last, largest, 64 evenly spaced), one tensor at a time: the blob from the
    # tensor's offset in the oracle's table to the next offset is the oracle's pack of that tensor alone
    table, table_total = orc.pack_layout(sizes, 256)
    ends = list(table[1:]) + [table_total]
    largest = max(range(len(ms)), key=lambda i: sizes[i])
    for i in sorted({0, len(ms) - 1, largest, *range(0, len(ms), max(1, len(ms) // 64))}):
        m = ms[i]
        want, _ = orc.pack([dst[r][m.byte_offset:m.byte_offset + m.byte_length].cpu().numpy()], 256)
        assert want.size == ends[i] - table[i]
        assert np.array_equal(blob[table[i]:ends[i]].cpu().numpy(), want), f"packed tensor {i} differs from the oracle"
    out = torch.full((ms[0].byte_length + ms[1].byte_length,), POISON, dtype=torch.uint8, device=device)
    bcp.bcp_unpack(blob, list(zip(offs[:2], sizes[:2])), [out.data_ptr(), out.data_ptr() + sizes[0]], blob_bytes=total)
    torch.cuda.synchronize()
    assert torch.equal(out[:sizes[0]], blob[offs[0]:offs[0] + sizes[0]]) and torch.equal(out[sizes[0]:], blob[offs[1]:offs[1] + sizes[1]])
    bcp.bcp_pack_cache_clear()


# ---- CUDA graphs ---------------------------------------------------------------------------------
@pytest.mark.parametrize("name,opts", [("cfg1", dict()), ("cfg1", dict(path_mask=7, tma_min_row_bytes=512)),
                                       ("big_random", dict(path_mask=3, tile_bytes=8192))], ids=str)
def test_reshard_replays_from_a_cuda_graph(cuda_device, name, opts):
    """A plan that has run once on some buffers is pure kernel launches on those buffers, so a
    stream capture records it and a replay reshards whatever the buffers hold by then."""
    case = CONFIGS["cfg1"]("index") if name == "cfg1" else big_random_case(3, itemsize=2)
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device, poison=0x5A)
    dst, backs = guarded(case.dst.buf_bytes, cuda_device)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts)
    bcp.bcp_reshard(plan, src, dst)  # binds the plan to the device and uploads its tables
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        bcp.bcp_reshard(plan, src, dst)  # the binding launches on torch's current stream: the capturing one
    for seed in (case.seed + 1, case.seed + 2):
        fresh = fills.fill_state(case.src, case.key_ids, "uniform", seed, cuda_device, poison=0x5A)
        for s, f in zip(src, fresh):
            s.copy_(f)
        for b in backs:
            b.fill_(POISON)
        want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
        graph.replay()
        torch.cuda.synchronize()
        bcp.bcp_plan_device_status(plan)
        assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want))
        assert guards_intact(backs, case.dst.buf_bytes)
    del graph
    plan.destroy()


# ---- host threads --------------------------------------------------------------------------------
def test_plans_run_from_several_threads_on_their_own_streams(cuda_device):
    """Different plans are independent: three host threads, each with its own plan, buffers and
    stream, execute at the same time (their kernels share the GPU; none waits for another)."""
    import threading

    torch.cuda.init()
    cases = [big_random_case(1, itemsize=2), CONFIGS["cfg1"]("index"), big_random_case(6, itemsize=4)]
    opts = [dict(path_mask=3, tile_bytes=8192), dict(), dict(path_mask=1, tile_bytes=16384)]
    jobs = []
    for case, o in zip(cases, opts):
        src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device, poison=0x5A)
        want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
        jobs.append((case, o, src, want))
    torch.cuda.synchronize()
    failures = []

    def work(case, o, src, want):
        try:
            torch.cuda.set_device(cuda_device)
            stream = torch.cuda.Stream(device=cuda_device)
            plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **o)
            for _ in range(8):
                with torch.cuda.stream(stream):
                    dst, backs = guarded(case.dst.buf_bytes, cuda_device)
                bcp.bcp_reshard(plan, src, dst, stream=stream)
                stream.synchronize()
                bcp.bcp_plan_device_status(plan, stream=stream)
                if not all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst, want)):
                    failures.append(case.name + ": wrong bytes")
                if not guards_intact(backs, case.dst.buf_bytes):
                    failures.append(case.name + ": guard band overwritten")
            plan.destroy()
        except Exception as e:  # noqa: BLE001 - reported below
            failures.append(f"{case.name}: {e!r}")

    threads = [threading.Thread(target=work, args=j) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not failures, failures[:3]


# ---- element conversion (extension) --------------------------------------------------------------
# kernel: path_mask 1 keeps every converting unit on the register kernel; path_mask 3 sends every source row of
# at least tma_min_row_bytes through the staged kernel (16: nearly all of them, 512: a mix of both kernels)
CVT_PATHS = {"register": {"path_mask": 1}, "staged": {"path_mask": 3, "tma_min_row_bytes": 16}, "mixed": {"path_mask": 3, "tma_min_row_bytes": 512}}


@pytest.mark.parametrize("path", list(CVT_PATHS))
@pytest.mark.parametrize("fill", ["index", "uniform"])
@pytest.mark.parametrize("case", convert_cases(), ids=lambda c: c.name)
def test_converting_reshard(cuda_device, case, fill, path):
    st = run_and_compare(case, cuda_device, fill, runs=2, tile_bytes=4096 if fill == "index" else 65536, **CVT_PATHS[path])
    assert st["n_cvt_tiles"] > 0


@pytest.mark.parametrize("path", ["register", "staged"])
def test_converting_reshard_every_bit_pattern_and_alignment(cuda_device, path):
    """All 2^32 binary32 patterns are too many; all 2^16 upper halves times the lower halves around
    the halfway point are not (every exponent, every tie, NaNs, infinities), and rows that start
    at every element phase exercise the leading / body / tail split of the kernel."""
    hi = np.arange(1 << 16, dtype=np.uint64) << 16
    lows = np.array([0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF], dtype=np.uint64)
    bits = (hi[:, None] | lows[None, :]).reshape(-1).astype(np.uint32)  # 393,216 values
    n = bits.size
    rows, cols = 96, n // 96
    src_meta = [ShardMeta("x", 4, 2, (rows, cols), (0, 0), (rows, cols), 0, 0)]
    # wanted: column blocks of odd widths, so that row starts fall on every phase of 16 bytes
    cuts = [0, 1, 4, 9, 16, 23, 1000, 1003, cols]
    dst_meta, pos = [], 0
    for a, b in zip(cuts, cuts[1:]):
        m = ShardMeta("x", 2, 1, (rows, cols), (0, a), (rows, b - a), 0, pos)
        dst_meta.append(m)
        pos += m.byte_length + (2 if (b - a) % 2 else 6)  # odd gaps: targets start at odd element offsets too
    blob = torch.from_numpy(bits.view(np.uint8).copy()).to(cuda_device)
    want = orc.reshard(src_meta, [bits.view(np.uint8)], dst_meta, [pos], fill_byte=POISON, convert=(1, 2, 1))[0]
    plan = bcp.bcp_plan(src_meta, [n * 4], dst_meta, [pos], convert=1, convert_src_tag=2, convert_dst_tag=1, tile_bytes=8192,
                        **CVT_PATHS[path])
    staged = sum(1 for t in plan.tiles() if t.flags & api.TILE_TMA)
    assert (staged > 0) == (path == "staged")
    dst, backs = guarded([pos], cuda_device)
    bcp.bcp_reshard(plan, [blob], dst)
    torch.cuda.synchronize()
    bcp.bcp_plan_device_status(plan)
    assert np.array_equal(dst[0].cpu().numpy(), want) and guards_intact(backs, [pos])
    plan.destroy()
    # and back: every bfloat16 pattern widened
    h = np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)
    src_meta = [ShardMeta("h", 2, 1, (1 << 16,), (0,), (1 << 16,), 0, 0)]
    dst_meta = [ShardMeta("h", 4, 2, (1 << 16,), (a,), (b - a,), 0, 4 * a + 4) for a, b in ((0, 3), (3, 40001), (40001, 1 << 16))]
    total = 4 * (1 << 16) + 4
    want = orc.reshard(src_meta, [h.view(np.uint8)], dst_meta, [total], fill_byte=POISON, convert=(2, 1, 2))[0]
    plan = bcp.bcp_plan(src_meta, [h.nbytes], dst_meta, [total], convert=2, convert_src_tag=1, convert_dst_tag=2, **CVT_PATHS[path])
    dst, backs = guarded([total], cuda_device)
    bcp.bcp_reshard(plan, [torch.from_numpy(h.view(np.uint8).copy()).to(cuda_device)], dst)
    torch.cuda.synchronize()
    assert np.array_equal(dst[0].cpu().numpy(), want) and guards_intact(backs, [total])
    plan.destroy()


def test_converting_reshard_from_host_buffers(cuda_device):
    case = convert_cases()[1]
    src = [s.cpu() for s in fills.fill_state(case.src, case.key_ids, "uniform", case.seed, "cpu")]
    want = orc.reshard(case.src.metas, [s.numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=0, convert=case.convert)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **case.plan_opts)
    for pinned in (False, True):
        a = [s.pin_memory() if pinned else s for s in src]
        dst = [torch.full((n,), POISON, dtype=torch.uint8, pin_memory=pinned) for n in case.dst.buf_bytes]
        bcp.bcp_reshard_host(plan, a, dst)
        assert all(np.array_equal(d.numpy(), w) for d, w in zip(dst, want))
    plan.destroy()


# ---- one plan, two streams -----------------------------------------------------------------------
def test_same_layout_on_two_streams_is_ordered(cuda_device):
    """Packs of one layout share a cached work list (pointer table, ticket counters); issued on two
    streams back to back, the second must wait for the first instead of racing it.  Same for a plan
    the caller executes on two streams."""
    n, parts = 96 << 20, 6
    sizes = [n // parts] * parts
    offs, total = bcp.bcp_pack_layout(sizes, 256)
    metas = list(zip(offs, sizes))
    s1, s2 = torch.cuda.Stream(device=cuda_device), torch.cuda.Stream(device=cuda_device)
    a = [torch.full((m,), 1 + i, dtype=torch.uint8, device=cuda_device) for i, m in enumerate(sizes)]
    b = [torch.full((m,), 101 + i, dtype=torch.uint8, device=cuda_device) for i, m in enumerate(sizes)]
    blob_a = torch.full((total,), POISON, dtype=torch.uint8, device=cuda_device)
    blob_b = torch.full((total,), POISON, dtype=torch.uint8, device=cuda_device)
    torch.cuda.synchronize()
    for _ in range(3):
        bcp.bcp_pack(a, metas, blob_a, stream=s1)
        bcp.bcp_pack(b, metas, blob_b, stream=s2)  # no host synchronisation in between
    torch.cuda.synchronize()
    for i, (o, m) in enumerate(metas):
        assert bool((blob_a[o:o + m] == 1 + i).all()) and bool((blob_b[o:o + m] == 101 + i).all())
    # a plan executed alternately on two streams, with different buffers
    case = big_random_case(2, itemsize=4)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, path_mask=3, tile_bytes=8192)
    src1 = fills.fill_state(case.src, case.key_ids, "index", 1, cuda_device)
    src2 = fills.fill_state(case.src, case.key_ids, "index", 2, cuda_device)
    want1 = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src1], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    want2 = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src2], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    dst1 = [torch.full((m,), POISON, dtype=torch.uint8, device=cuda_device) for m in case.dst.buf_bytes]
    dst2 = [torch.full((m,), POISON, dtype=torch.uint8, device=cuda_device) for m in case.dst.buf_bytes]
    torch.cuda.synchronize()
    for _ in range(4):
        bcp.bcp_reshard(plan, src1, dst1, stream=s1)
        bcp.bcp_reshard(plan, src2, dst2, stream=s2)
    torch.cuda.synchronize()
    bcp.bcp_plan_device_status(plan)
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst1, want1))
    assert all(np.array_equal(d.cpu().numpy(), w) for d, w in zip(dst2, want2))
    plan.destroy()


# ---- tracing -------------------------------------------------------------------------------------
def test_trace_spans_time_stream_work(cuda_device, tmp_path):
    from paper_2407_20143_b200.trace import Trace

    case = CONFIGS["cfg1"]("index")
    src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device)
    dst = fills.make_buffers(case.dst, cuda_device, POISON)
    plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes)
    st = plan.stats()
    moved = st["bytes_src_unique"] + st["bytes_copied"]
    tr = Trace(rank=3)
    for step in range(4):
        with tr.span("reshard", nbytes=moved, step=step):
            bcp.bcp_reshard(plan, src, dst)
    with tr.span("idle"):
        pass
    rows = tr.rows()
    assert [r["name"] for r in rows] == ["reshard"] * 4 + ["idle"] and all(r["rank"] == 3 for r in rows)
    assert [r["step"] for r in rows[:4]] == [0, 1, 2, 3]
    assert all(0.001 < r["ms"] < 50 and r["gbps"] > 1 for r in rows[:4]) and rows[4]["gbps"] is None
    tot = tr.totals()
    assert tot["reshard"]["calls"] == 4 and tot["reshard"]["bytes"] == 4 * moved
    tr.dump(str(tmp_path / "trace.jsonl"))
    assert len(open(tmp_path / "trace.jsonl").read().splitlines()) == 5
    plan.destroy()
