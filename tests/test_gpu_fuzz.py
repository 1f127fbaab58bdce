"""Differential fuzz on the GPU: seeded random problems x seeded random launch options, every
target byte against the CPU oracle (a campaign of 4,400 such cases ran clean when this was
written; the suite keeps a short, fixed slice of it)."""
import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import scenario_cases
from workloads.random_cases import big_random_case, random_case, random_convert_case

pytestmark = pytest.mark.gpu


def _draw(rng, it, scen):
    seed = int(rng.integers(0, 1 << 30))
    if it % 4 == 0:
        case = random_case(seed, n_tensors=int(rng.integers(1, 6)), max_ndim=int(rng.integers(1, 9)), max_dim=int(rng.integers(2, 9)),
                           gap_mod=int(rng.integers(0, 9)), dst_replicas=int(rng.integers(1, 4)))
    elif it % 4 in (1, 2):
        case = big_random_case(seed, itemsize=int(rng.choice([1, 2, 4, 8])), gap_mod=int(rng.choice([0, 1, 4, 7, 8])))
    else:
        case = scen[int(rng.integers(0, len(scen)))]
    opts = dict(path_mask=int(rng.choice([0, 1, 3, 7])), tile_bytes=int(rng.choice([0, 4096, 8192, 16384, 65536, 262144])),
                fanout=int(rng.choice([1, 2])), order=int(rng.choice([0, 1, 2])),
                tma_stage_bytes=int(rng.choice([1024, 2048, 4096, 16384, 32768])), tma_stages=int(rng.choice([2, 3, 4, 6])),
                tma_ctas_per_sm=int(rng.choice([1, 2, 4])), tma_min_row_bytes=int(rng.choice([16, 64, 512, 2048])),
                worker=int(rng.choice([1, 2])), unroll=int(rng.choice([4, 8])), block_threads=int(rng.choice([256, 512, 1024])),
                small_bytes=int(rng.choice([64, 1024, 4096])))
    opts["small_bytes"] = min(opts["small_bytes"], opts["tile_bytes"])
    return case, opts


@pytest.mark.parametrize("stream_seed", [1, 2, 3])
def test_random_problems_and_options(cuda_device, stream_seed):
    rng = np.random.default_rng(stream_seed)
    scen = scenario_cases()
    for it in range(40):
        case, opts = _draw(rng, it, scen)
        src = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device, poison=0x5A)
        want = orc.reshard(case.src.metas, [s.cpu().numpy() for s in src], case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5)
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts)
        backs = [torch.full((m + 8192,), 0xA5, dtype=torch.uint8, device=cuda_device) for m in case.dst.buf_bytes]
        dst = [b[4096:4096 + m] for b, m in zip(backs, case.dst.buf_bytes)]
        for _ in range(2):
            bcp.bcp_reshard(plan, src, dst)
        torch.cuda.synchronize()
        bcp.bcp_plan_device_status(plan)
        for d, w in zip(dst, want):
            assert np.array_equal(d.cpu().numpy(), w), (case.name, opts)
        for b, m in zip(backs, case.dst.buf_bytes):
            assert bool((b[:4096] == 0xA5).all()) and bool((b[4096 + m:] == 0xA5).all()), (case.name, opts)
        plan.destroy()


@pytest.mark.parametrize("stream_seed", [11, 12])
def test_random_converting_problems_and_options(cuda_device, stream_seed):
    """The same for plans that convert some tensors (binary32 <-> bfloat16) and copy the others;
    sources are random bytes, so every bit pattern (NaN, infinities, subnormals) takes part."""
    rng = np.random.default_rng(stream_seed)
    for it in range(30):
        seed = int(rng.integers(0, 1 << 30))
        case = random_convert_case(seed, narrow=bool(it % 2), big=it % 3 == 0, dst_replicas=int(rng.integers(1, 3)))
        opts = dict(path_mask=int(rng.choice([0, 1, 3, 7])), tile_bytes=int(rng.choice([4096, 8192, 65536])), order=int(rng.choice([0, 1, 2])),
                    tma_min_row_bytes=int(rng.choice([16, 512])), worker=int(rng.choice([1, 2])), small_bytes=int(rng.choice([64, 4096])))
        g = torch.Generator(device="cpu").manual_seed(seed)
        host = [torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g) for n in case.src.buf_bytes]
        want = orc.reshard(case.src.metas, [h.numpy() for h in host], case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5,
                           convert=case.convert)
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, **opts, **case.plan_opts)
        assert plan.stats()["n_cvt_tiles"] > 0
        src = [h.to(cuda_device) for h in host]
        backs = [torch.full((m + 8192,), 0xA5, dtype=torch.uint8, device=cuda_device) for m in case.dst.buf_bytes]
        dst = [b[4096:4096 + m] for b, m in zip(backs, case.dst.buf_bytes)]
        for _ in range(2):
            bcp.bcp_reshard(plan, src, dst)
        torch.cuda.synchronize()
        bcp.bcp_plan_device_status(plan)
        for d, w in zip(dst, want):
            assert np.array_equal(d.cpu().numpy(), w), (case.name, opts)
        for b, m in zip(backs, case.dst.buf_bytes):
            assert bool((b[:4096] == 0xA5).all()) and bool((b[4096 + m:] == 0xA5).all()), (case.name, opts)
        plan.destroy()


@pytest.mark.parametrize("stream_seed", [21, 22])
def test_random_pack_layouts(cuda_device, stream_seed):
    """Random save-blob layouts through bcp_pack, bcp_pack_static and bcp_unpack against the
    oracle: many tensors under 4 KiB at odd addresses, a few large ones, alignments 16..4096,
    tensor counts up to the fixed-scratch limit (cases beyond its work-unit limit must be
    refused, never wrong)."""
    from paper_2407_20143_b200 import api

    rng = np.random.default_rng(stream_seed)
    for it in range(12):
        n = int(rng.choice([1, 7, 300, 2000, 4096]))
        kind = it % 3
        if kind == 0:
            sizes = rng.integers(0, 400, size=n)
        elif kind == 1:
            sizes = rng.integers(1, 5000, size=n)
        else:
            sizes = np.where(rng.random(n) < 0.02, rng.integers(60_000, 3_000_000, size=n), rng.integers(1, 300, size=n))
        sizes = [int(x) for x in sizes]
        align = int(rng.choice([16, 64, 256, 4096]))
        starts, pos = [], 0
        for s in sizes:
            pos = (pos + 15) // 16 * 16 + int(rng.integers(0, 16)) * int(rng.integers(0, 2))
            starts.append(pos)
            pos += s
        host = rng.integers(0, 256, size=pos + 16, dtype=np.uint8)
        back = torch.from_numpy(host).to(cuda_device)
        tensors = [back[a:a + s] for a, s in zip(starts, sizes)]
        ref, table = orc.pack([host[a:a + s] for a, s in zip(starts, sizes)], align)
        offs, total = bcp.bcp_pack_layout(sizes, align)
        assert total == ref.size and [int(o) for o, _ in table] == [int(o) for o in offs]
        metas = list(zip(offs, sizes))
        blob = torch.full((total,), 0xA5, dtype=torch.uint8, device=cuda_device)
        bcp.bcp_pack(tensors, metas, blob)
        torch.cuda.synchronize()
        assert np.array_equal(blob.cpu().numpy(), ref), ("pack", it, n, align)
        blob2 = torch.full((total,), 0x5A, dtype=torch.uint8, device=cuda_device)
        try:
            bcp.bcp_pack_static(tensors, metas, blob2)
            torch.cuda.synchronize()
            assert np.array_equal(blob2.cpu().numpy(), ref), ("static pack", it, n, align)
        except bcp.BcpError as e:
            assert e.code == api.ERR_CAPACITY, e
            torch.cuda.synchronize()
            assert bool((blob2 == 0x5A).all()), "a refused call must not write"
        out_back = torch.full((pos + 16,), 0x33, dtype=torch.uint8, device=cuda_device)
        outs = [out_back[a:a + s] for a, s in zip(starts, sizes)]
        bcp.bcp_unpack(blob, metas, outs)
        torch.cuda.synchronize()
        got = out_back.cpu().numpy()
        expect = np.full(pos + 16, 0x33, dtype=np.uint8)
        for a, s in zip(starts, sizes):
            expect[a:a + s] = host[a:a + s]
        assert np.array_equal(got, expect), ("unpack", it, n, align)
    bcp.bcp_pack_cache_clear()
