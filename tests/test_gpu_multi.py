"""Cross-rank resharding on one GPU: the ranks of a 2- and 3-rank job are emulated one after the
other in one process (pack of all ranks, then the segment swap an all-to-all would do, then every
rank's reshard), so every device step of the exchange runs through the library; only the
collective itself is replaced by tensor copies.  No kernel waits for another."""
import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import multi
from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import convert_cases, scenario_cases
from workloads.random_cases import big_random_case

pytestmark = pytest.mark.gpu
POISON = 0xA5

CASES = [c for c in scenario_cases() if c.name in ("hybrid", "dp150-to-dp75", "llama-tp8-to-tp2")] + [big_random_case(4, itemsize=2), convert_cases()[1]]


@pytest.mark.parametrize("world", [1, 2, 3])
@pytest.mark.parametrize("case", CASES, ids=lambda c: c.name)
def test_emulated_ranks_exchange_and_reshard(cuda_device, case, world):
    ns, nd = len(case.src.buf_bytes), len(case.dst.buf_bytes)
    src_owner = [b % world for b in range(ns)]
    dst_owner = [(b * world) // nd for b in range(nd)]  # contiguous blocks of target buffers
    opts = case.plan_opts
    blobs = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device, poison=0x5A)
    want = orc.reshard(case.src.metas, [b.cpu().numpy() for b in blobs], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON,
                       convert=case.convert)
    needs = [multi.needed_entries(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, dst_owner, r, **opts)
             for r in range(world)]
    xs = [multi.build_exchange(case.src.metas, case.src.buf_bytes, src_owner, case.dst.metas, case.dst.buf_bytes, dst_owner, r, world,
                               needs, **opts) for r in range(world)]
    # sender side of every rank
    sends = []
    for x in xs:
        buf = torch.full((max(1, sum(x.send_bytes)),), 0xEE, dtype=torch.uint8, device=cuda_device)
        multi.pack_sends(x, case.src.metas, [blobs[b] for b in x.local_src], buf)
        sends.append(buf)
    torch.cuda.synchronize()
    for r, x in enumerate(xs):
        assert x.recv_bytes == [xs[s].send_bytes[r] for s in range(world)]

        def swap(recv, send, recv_splits, send_splits, r=r):  # what all_to_all_single does, from the emulated peers' buffers
            at = 0
            for s in range(world):
                off = sum(xs[s].send_bytes[:r])
                recv[at:at + recv_splits[s]].copy_(sends[s][off:off + recv_splits[s]])
                at += recv_splits[s]

        dst = [torch.full((n,), POISON, dtype=torch.uint8, device=cuda_device) for n in x.dst_buf_bytes]
        for rep in range(2):  # the second step reuses the exchange's buffers, stream and marshalled pack
            if rep:
                for d in dst:
                    d.fill_(POISON)
            multi.run_exchange(x, case.src.metas, [blobs[b] for b in x.local_src], dst, all_to_all=swap)
            torch.cuda.synchronize()
            for p in (x.plan_local, x.plan_remote):
                if p is not None:
                    bcp.bcp_plan_device_status(p)
            for d, b in zip(dst, x.local_dst):
                assert np.array_equal(d.cpu().numpy(), want[b]), (case.name, world, r, b, rep)
        ms = x.stage_ms()
        assert set(ms) == {"pack", "all_to_all", "reshard_remote", "reshard_local", "step"} and ms["step"] > 0
        assert (x.plan_remote is None) == (world == 1 or sum(x.recv_bytes) == 0)
    # every target buffer has exactly one owner
    assert sorted(b for x in xs for b in x.local_dst) == list(range(nd))
    if world > 1:  # bytes that crossed ranks: at most what the targets read, and none for a rank's own blobs
        assert all(x.send_bytes[x.rank] == 0 for x in xs) and sum(sum(x.send_bytes) for x in xs) > 0
    for x in xs:
        x.destroy()


@pytest.mark.parametrize("world", [2, 3])
def test_zero_copy_variant_reads_peer_blobs_in_place(cuda_device, world):
    """Without any exchange: every emulated rank plans only its own target buffers against the
    global saved metadata and hands bcp_reshard the addresses of ALL saved blobs (on several GPUs
    the other ranks' blobs would be peer-mapped; here they simply live on the same device).  The
    kernels fetch their tiles straight from wherever a blob lies, so the ranks' plans together
    write every target buffer and nothing is packed or received."""
    case = [c for c in scenario_cases() if c.name == "hybrid"][0]
    nd = len(case.dst.buf_bytes)
    dst_owner = [(b * world) // nd for b in range(nd)]
    blobs = fills.fill_state(case.src, case.key_ids, "index", case.seed, cuda_device, poison=0x5A)
    want = orc.reshard(case.src.metas, [b.cpu().numpy() for b in blobs], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
    written = 0
    for r in range(world):
        mine, metas, sizes = multi._local_targets(case.dst.metas, case.dst.buf_bytes, dst_owner, r)
        plan = bcp.bcp_plan(case.src.metas, case.src.buf_bytes, metas, sizes, path_mask=7, tma_min_row_bytes=16)
        dst = [torch.full((n,), POISON, dtype=torch.uint8, device=cuda_device) for n in sizes]
        bcp.bcp_reshard(plan, blobs, dst)
        torch.cuda.synchronize()
        bcp.bcp_plan_device_status(plan)
        for d, b in zip(dst, mine):
            assert np.array_equal(d.cpu().numpy(), want[b]), (world, r, b)
        written += plan.stats()["bytes_copied"]
        plan.destroy()
    assert written == case.dst.total_bytes


def test_two_processes_zero_copy_and_exchange(cuda_device):
    """Two rank processes on the one GPU (independent launches, host-side barriers): peers' blobs
    mapped through bcp_ipc_* and read in place, then the pack -> all-to-all -> two-plan exchange with
    a real collective carrying the segments; every rank's targets against the oracle."""
    import os
    import subprocess
    import sys

    torch.cuda.empty_cache()  # what this process has cached is not available to the two ranks
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    worker = os.path.join(root, "tests", "two_process_worker.py")
    port = 29700 + os.getpid() % 200
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK="0", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, worker], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=240))
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
    assert all(p.returncode == 0 for p in procs), [o[1][-1500:] for o in outs]
    assert all("two-process ok" in o[0] for o in outs)
