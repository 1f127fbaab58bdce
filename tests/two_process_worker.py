"""One rank of the two-process cross-rank tests (started by tests/test_gpu_multi.py, never collected by
pytest).  Both ranks use the SAME GPU: their kernels are independent launches that never wait for one
another, and the ranks synchronise on the host (gloo barriers), so sharing the device is safe; what the
test exercises is everything that differs from the one-process emulation: real process boundaries,
blobs mapped through IPC handles, a real collective for the segments (gloo over host copies here; NCCL
needs one GPU per rank)."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import numpy as np
import torch
import torch.distributed as tdist

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import dist, multi
from oracle import reshard_oracle as orc
from workloads import fills
from workloads.configs import scenario_cases

POISON = 0xA5


def main():
    assert dist.init("gloo")
    rank, _, ws = dist.world()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    for case in [c for c in scenario_cases() if c.name in ("hybrid", "llama-tp8-to-tp2")]:
        ns, nd = len(case.src.buf_bytes), len(case.dst.buf_bytes)
        src_owner = [b % ws for b in range(ns)]
        dst_owner = [(b * ws) // nd for b in range(nd)]
        host = fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu", poison=0x5A)
        want = orc.reshard(case.src.metas, [h.numpy() for h in host], case.dst.metas, case.dst.buf_bytes, fill_byte=POISON)
        mine = [b for b in range(ns) if src_owner[b] == rank]
        blobs = [host[b].to(dev) for b in mine]  # only this rank's blobs ever reach its memory
        torch.cuda.synchronize()

        # (1) no exchange: peers' blobs mapped through IPC handles, read in place by the copy kernels
        zc = multi.plan_zero_copy(case.src.metas, case.src.buf_bytes, src_owner, case.dst.metas, case.dst.buf_bytes, dst_owner, blobs,
                                  path_mask=7, tma_min_row_bytes=16)
        assert len(zc.opened) > 0, "a rank of this layout reads blobs of the other rank"
        dst = [torch.full((n,), POISON, dtype=torch.uint8, device=dev) for n in zc.dst_buf_bytes]
        dist.barrier()  # every owner's blobs are complete
        for _ in range(2):
            zc.run(dst)
        torch.cuda.synchronize()
        bcp.bcp_plan_device_status(zc.plan)
        for d, b in zip(dst, zc.local_dst):
            assert np.array_equal(d.cpu().numpy(), want[b]), ("zero-copy", case.name, rank, b)
        dist.barrier()  # nobody reads any more: blobs may go
        try:
            bcp.api.bcp_ipc_close(blobs[0].data_ptr())  # an address that no bcp_ipc_open returned
            raise AssertionError("closing a pointer that was never opened must fail")
        except bcp.BcpError as e:
            assert e.code == bcp.api.ERR_INVALID
        zc.close()

        # (2) the exchange: pack on the GPU, segments through a real collective, two plans
        x = multi.plan_exchange(case.src.metas, case.src.buf_bytes, src_owner, case.dst.metas, case.dst.buf_bytes, dst_owner)

        def a2a(recv, send, recv_splits, send_splits):
            torch.cuda.current_stream().synchronize()
            r = torch.zeros(max(1, sum(recv_splits)), dtype=torch.uint8)
            tdist.all_to_all_single(r[: sum(recv_splits)], send[: sum(send_splits)].cpu(), list(recv_splits), list(send_splits))
            recv[: sum(recv_splits)].copy_(r[: sum(recv_splits)])

        dst = [torch.full((n,), POISON, dtype=torch.uint8, device=dev) for n in x.dst_buf_bytes]
        for _ in range(2):
            multi.run_exchange(x, case.src.metas, blobs, dst, all_to_all=a2a)
        torch.cuda.synchronize()
        assert sum(x.send_bytes) > 0 and sum(x.recv_bytes) > 0 and x.plan_local is not None and x.plan_remote is not None
        for d, b in zip(dst, x.local_dst):
            assert np.array_equal(d.cpu().numpy(), want[b]), ("exchange", case.name, rank, b)
        x.destroy()
        dist.barrier()
    print("two-process ok", rank, flush=True)
    dist.shutdown()


if __name__ == "__main__":
    main()
