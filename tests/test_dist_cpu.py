"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, max-over-ranks timing."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2407_20143_b200 import dist
    assert dist.init("gloo")
    rank, _, ws = dist.world()
    dist.barrier()
    agg = dist.aggregate_throughput(units_local=100.0 * (rank + 1), ms_local=10.0 * (rank + 1))
    dist.barrier()
    if rank == 0:
        print(json.dumps(agg))
    dist.shutdown()
""") % ROOT


def test_two_rank_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29600 + os.getpid() % 300
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json

    agg = json.loads(outs[0][0].strip().splitlines()[-1])
    # slowest rank took 20 ms, both ranks together processed 300 units
    assert agg["ms"] == 20.0 and agg["units"] == 300.0 and abs(agg["per_second"] - 15000.0) < 1e-6


def test_single_process_is_a_no_op():
    from paper_2407_20143_b200 import dist

    env_ws = os.environ.pop("WORLD_SIZE", None)
    try:
        assert dist.init() is False
        assert dist.max_over_ranks(3.5) == 3.5
        assert dist.aggregate_throughput(10.0, 5.0)["per_second"] == 2000.0
    finally:
        if env_ws is not None:
            os.environ["WORLD_SIZE"] = env_ws


# ---- cross-rank resharding: the exchange schedule on two gloo ranks ------------------------------
EXCHANGE_WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    sys.path.insert(0, os.path.join(%r, "tests"))
    import numpy as np, torch, torch.distributed as tdist
    from paper_2407_20143_b200 import dist, multi
    from oracle import reshard_oracle as orc
    from workloads import fills
    from workloads.configs import scenario_cases, convert_cases
    from test_planner import run_tiles
    assert dist.init("gloo")
    rank, _, ws = dist.world()
    for case in [c for c in scenario_cases() if c.name in ("hybrid", "llama-tp8-to-tp2", "dp4-to-dp8")] + convert_cases()[:1]:
        opts = case.plan_opts
        src_owner = [b %% ws for b in range(len(case.src.buf_bytes))]            # saved blobs round-robin over the ranks
        nd = len(case.dst.buf_bytes)
        dst_owner = [((b // 2) if nd >= 4 else b) %% ws for b in range(nd)]      # target buffers in pairs (singly when there are two)
        x = multi.plan_exchange(case.src.metas, case.src.buf_bytes, src_owner, case.dst.metas, case.dst.buf_bytes, dst_owner, **opts)
        blobs = [t.numpy() for t in fills.fill_state(case.src, case.key_ids, "index", case.seed, "cpu")]
        # stand-in for the device pack: the schedule's entries at the schedule's offsets
        send = np.zeros(max(1, sum(x.send_bytes)), dtype=np.uint8)
        base = 0
        for q in range(ws):
            for i, o in zip(x.send_entries[q], x.send_offsets[q]):
                m = case.src.metas[i]
                assert src_owner[m.buf_index] == rank and q != rank
                send[base + o:base + o + m.byte_length] = blobs[m.buf_index][m.byte_offset:m.byte_offset + m.byte_length]
            base += x.send_bytes[q]
        recv = torch.zeros(max(1, sum(x.recv_bytes)), dtype=torch.uint8)
        tdist.all_to_all_single(recv[:sum(x.recv_bytes)], torch.from_numpy(send)[:sum(x.send_bytes)], list(x.recv_bytes), list(x.send_bytes))
        srcs, at = [blobs[b] for b in x.local_src], 0
        for s in range(ws):
            if x.recv_bytes[s]:
                srcs.append(recv[at:at + x.recv_bytes[s]].numpy())
                at += x.recv_bytes[s]
        assert [len(s) for s in srcs] == x.src_buf_bytes
        # the rank's work comes as two plans over the same buffer lists: pieces read from its own blobs and
        # pieces read from received segments; between them every target byte is written exactly once
        n_local = len(x.local_src)
        units = []
        for plan, lo, hi in ((x.plan_local, 0, n_local), (x.plan_remote, n_local, len(srcs))):
            assert plan is not None
            ts = plan.tiles()
            assert ts and all(lo <= t.src_buf < hi for t in ts), case.name
            units += ts
        got, count = run_tiles(units, srcs, x.dst_buf_bytes)
        named = [np.zeros(n, dtype=bool) for n in x.dst_buf_bytes]
        for m in case.dst.metas:
            if dst_owner[m.buf_index] == rank:
                named[x.local_dst.index(m.buf_index)][m.byte_offset:m.byte_offset + m.byte_length] = True
        for c, nm in zip(count, named):
            assert np.array_equal(c, nm.astype(c.dtype)), (case.name, rank)
        want = orc.reshard(case.src.metas, blobs, case.dst.metas, case.dst.buf_bytes, fill_byte=0xA5, convert=case.convert)
        assert len(x.local_dst) > 0 and sum(x.recv_bytes) > 0 and sum(x.send_bytes) > 0, case.name
        for g, b in zip(got, x.local_dst):
            assert np.array_equal(g, want[b]), (case.name, rank, b)
        # nothing is sent that the receiver does not read, and nothing twice
        assert all(len(set(e)) == len(e) for e in x.send_entries)
        x.destroy()
    dist.barrier()
    print("exchange ok", rank)
    dist.shutdown()
""") % (ROOT, ROOT)


def test_two_rank_exchange_schedule(tmp_path):
    """Every rank plans its targets against the global metadata, the needed saved entries travel in
    one all-to-all with the schedule's split sizes, and the final per-rank plan, run by the numpy
    unit simulator on the bytes as they arrived, equals the oracle on that rank's targets."""
    script = tmp_path / "exchange_worker.py"
    script.write_text(EXCHANGE_WORKER)
    port = 29900 + os.getpid() % 90
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("exchange ok" in o[0] for o in outs)


def test_exchange_schedule_properties_without_a_process_group():
    """Host logic of the exchange on emulated ranks: what one rank sends is what the other expects,
    only needed entries travel, a rank's own blobs are never sent, and with one rank nothing moves."""
    from paper_2407_20143_b200 import multi
    from workloads.configs import scenario_cases

    case = [c for c in scenario_cases() if c.name == "hybrid"][0]
    ns, nd = len(case.src.buf_bytes), len(case.dst.buf_bytes)
    for world in (1, 2, 4):
        src_owner = [b % world for b in range(ns)]
        dst_owner = [(b * world) // nd for b in range(nd)]
        needs = [multi.needed_entries(case.src.metas, case.src.buf_bytes, case.dst.metas, case.dst.buf_bytes, dst_owner, r)
                 for r in range(world)]
        xs = [multi.build_exchange(case.src.metas, case.src.buf_bytes, src_owner, case.dst.metas, case.dst.buf_bytes, dst_owner,
                                   r, world, needs) for r in range(world)]
        for r, x in enumerate(xs):
            assert x.recv_bytes == [xs[s].send_bytes[r] for s in range(world)]
            assert x.send_bytes[r] == 0 and x.send_entries[r] == []
            for q in range(world):
                assert set(x.send_entries[q]) <= set(needs[q])
                assert all(src_owner[case.src.metas[i].buf_index] == r for i in x.send_entries[q])
                assert x.send_bytes[q] % multi.SEGMENT_ALIGN == 0
            # the two final plans together write exactly this rank's target bytes
            mine = sum(m.byte_length for m in case.dst.metas if dst_owner[m.buf_index] == r)
            assert sum(p.stats()["bytes_copied"] for p in (x.plan_local, x.plan_remote) if p is not None) == mine
            assert (x.plan_remote is None) == (sum(x.recv_bytes) == 0)
        # every needed entry is either local or sent by its owner, once
        for q in range(world):
            got = sorted(i for x in xs for i in x.send_entries[q]) + [i for i in needs[q] if src_owner[case.src.metas[i].buf_index] == q]
            assert sorted(got) == sorted(needs[q])
        if world == 1:
            assert xs[0].send_bytes == [0] and xs[0].recv_bytes == [0] and xs[0].local_dst == list(range(nd))
        for x in xs:
            x.destroy()
