"""Resharding across several GPUs: saved blobs and target buffers are spread over the ranks of
a process group (one process per GPU), and every rank materialises its own target buffers.

The paper's load pipeline has exactly one exchange step: every saved shard is read by one
rank and the pieces other ranks need travel in an all-to-all (Sec. 4.1, "Eliminating redundant
loading", and the load pipeline of Sec. 4.2).  Here the saved blobs already sit in the HBM of
their owners, so the same step becomes:

  1. every rank plans its own targets against the GLOBAL saved metadata (host only) and reads
     off the plan which saved entries it touches;
  2. the lists of needed entries are gathered, so every owner knows what to send to whom;
  3. every owner packs, per receiver, the needed entries of its blobs into one send buffer
     (`bcp_pack`, on the GPU), and one `all_to_all_single` moves the segments (NCCL over NVLink);
  4. every rank re-plans its targets against the entries as they now lie in its memory (its
     own blobs plus one received segment per peer), as two plans: the pieces read from its own
     blobs, which are copied on a side stream while the segments travel, and the pieces read
     from received segments, copied once they have arrived (`bcp_reshard`, twice).

Steps 1, 2 and 4's planning are metadata work; all bytes move in library kernels and in the
collective.  Everything here is argument marshalling around the C ABI and `torch.distributed`.
"""
from __future__ import annotations

import copy
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

from . import api

SEGMENT_ALIGN = 256  # entries inside a send segment, and segments inside the buffers


@dataclass
class Exchange:
    """What one rank sends, receives and finally executes.

    The rank's final work is split in two plans over the same buffer lists (sources = own blobs,
    then one received segment per sender with recv_bytes > 0): `plan_local` holds the pieces read
    from the rank's own blobs, `plan_remote` the pieces read from received segments.  Between them
    they write every target byte exactly once, so the local one can run while the segments are
    still travelling."""

    rank: int
    world: int
    local_src: List[int]                 # global indices of the saved blobs this rank owns, in local order
    local_dst: List[int]                 # global indices of the target buffers this rank fills, in local order
    send_entries: List[List[int]]        # per receiver: indices into the global saved metas, in pack order
    send_offsets: List[List[int]]        # per receiver: byte offset of every such entry inside the segment
    send_bytes: List[int]                # per receiver: segment size (multiple of SEGMENT_ALIGN; 0 for none / self)
    recv_bytes: List[int]                # per sender
    plan_local: Optional[api.Plan] = None
    plan_remote: Optional[api.Plan] = None   # None when nothing is received
    src_buf_bytes: List[int] = field(default_factory=list)
    dst_buf_bytes: List[int] = field(default_factory=list)
    # device side, created once by bind(): nothing is allocated per step
    send_buf: object = None
    recv_buf: object = None
    side: object = None                  # stream of the local plan
    events: Dict[str, object] = field(default_factory=dict)
    pack_args: object = None             # marshalled arguments of the sender-side pack

    def bind(self, device) -> None:
        """Send / receive buffers, the side stream and the stage events, once per exchange."""
        import torch

        if self.send_buf is not None:
            return
        with torch.cuda.device(device):
            self.send_buf = torch.empty(max(1, sum(self.send_bytes)), dtype=torch.uint8, device=device)
            self.recv_buf = torch.empty(max(1, sum(self.recv_bytes)), dtype=torch.uint8, device=device)
            self.side = torch.cuda.Stream(device=device)
            for k in ("begin", "packed", "arrived", "remote_done", "local_begin", "local_done", "end"):
                self.events[k] = torch.cuda.Event(enable_timing=True)

    def sources(self, local_blobs: Sequence) -> List:
        """Source list of both plans: own blobs, then the received segments (views of recv_buf)."""
        srcs, at = list(local_blobs), 0
        for s in range(self.world):
            if self.recv_bytes[s]:
                srcs.append(self.recv_buf[at:at + self.recv_bytes[s]])
                at += self.recv_bytes[s]
        return srcs

    def stage_ms(self) -> Dict[str, float]:
        """Device times of the last step's stages (call after synchronising)."""
        e = self.events
        out = {"pack": e["begin"].elapsed_time(e["packed"]), "all_to_all": e["packed"].elapsed_time(e["arrived"]),
               "reshard_remote": e["arrived"].elapsed_time(e["remote_done"]),
               "reshard_local": e["local_begin"].elapsed_time(e["local_done"]), "step": e["begin"].elapsed_time(e["end"])}
        return out

    def destroy(self) -> None:
        for name in ("plan_local", "plan_remote"):
            p = getattr(self, name)
            if p is not None:
                p.destroy()
                setattr(self, name, None)
        self.send_buf = self.recv_buf = None


def _local_targets(dst_metas: Sequence, dst_buf_bytes: Sequence[int], dst_owner: Sequence[int], rank: int):
    """This rank's target entries with buffer indices renumbered densely."""
    mine = [b for b, o in enumerate(dst_owner) if o == rank]
    local = {b: i for i, b in enumerate(mine)}
    metas = []
    for m in dst_metas:
        if m.buf_index in local:
            k = copy.copy(m)
            k.buf_index = local[m.buf_index]
            metas.append(k)
    return mine, metas, [dst_buf_bytes[b] for b in mine]


def needed_entries(src_metas: Sequence, src_buf_bytes: Sequence[int], dst_metas: Sequence, dst_buf_bytes: Sequence[int],
                   dst_owner: Sequence[int], rank: int, **opts) -> List[int]:
    """Indices of the saved entries whose bytes this rank's targets read: the planner does the
    matching and reports them (bcp_plan_used_sources)."""
    _, mine, mine_bytes = _local_targets(dst_metas, dst_buf_bytes, dst_owner, rank)
    probe = api.bcp_plan(src_metas, src_buf_bytes, mine, mine_bytes, **opts)
    try:
        return probe.used_sources()
    finally:
        probe.destroy()


def build_exchange(src_metas: Sequence, src_buf_bytes: Sequence[int], src_owner: Sequence[int], dst_metas: Sequence,
                   dst_buf_bytes: Sequence[int], dst_owner: Sequence[int], rank: int, world: int,
                   all_needs: Sequence[Sequence[int]], **opts) -> Exchange:
    """all_needs[r] = needed_entries(...) of rank r, for every rank (gathered by the caller)."""
    owner_of = lambda i: src_owner[src_metas[i].buf_index]  # noqa: E731
    send_entries, send_offsets, send_bytes = [], [], []
    for q in range(world):
        ents = [i for i in all_needs[q] if owner_of(i) == rank] if q != rank else []
        offs, total = api.bcp_pack_layout([src_metas[i].byte_length for i in ents], SEGMENT_ALIGN) if ents else ([], 0)
        send_entries.append(ents)
        send_offsets.append(offs)
        send_bytes.append(total)
    # what arrives, and where every needed entry will lie in this rank's memory
    local_src = [b for b, o in enumerate(src_owner) if o == rank]
    local_id = {b: i for i, b in enumerate(local_src)}
    metas, sizes = [], [src_buf_bytes[b] for b in local_src]
    recv_bytes = [0] * world
    by_sender: Dict[int, List[int]] = {}
    for i in all_needs[rank]:
        by_sender.setdefault(owner_of(i), []).append(i)
    for s in range(world):
        ents = by_sender.get(s, [])
        if s == rank:
            for i in ents:
                k = copy.copy(src_metas[i])
                k.buf_index = local_id[k.buf_index]
                metas.append(k)
            continue
        if not ents:
            continue
        offs, total = api.bcp_pack_layout([src_metas[i].byte_length for i in ents], SEGMENT_ALIGN)
        recv_bytes[s] = total
        for i, o in zip(ents, offs):
            k = copy.copy(src_metas[i])
            k.buf_index, k.byte_offset = len(sizes), o
            metas.append(k)
        sizes.append(total)
    local_dst, mine, mine_bytes = _local_targets(dst_metas, dst_buf_bytes, dst_owner, rank)
    n_local = len(local_src)
    if len(sizes) == n_local:   # nothing is received: one plan does everything
        plan_local, plan_remote = api.bcp_plan(metas, sizes, mine, mine_bytes, **opts), None
    elif n_local == 0:          # the rank owns no blob: everything it reads arrives
        plan_local, plan_remote = None, api.bcp_plan(metas, sizes, mine, mine_bytes, **opts)
    else:
        plan_local = api.bcp_plan(metas, sizes, mine, mine_bytes, src_buf_first=0, src_buf_count=n_local, **opts)
        plan_remote = api.bcp_plan(metas, sizes, mine, mine_bytes, src_buf_first=n_local, src_buf_count=len(sizes) - n_local, **opts)
    return Exchange(rank, world, local_src, local_dst, send_entries, send_offsets, send_bytes, recv_bytes, plan_local, plan_remote,
                    sizes, mine_bytes)


def plan_exchange(src_metas: Sequence, src_buf_bytes: Sequence[int], src_owner: Sequence[int], dst_metas: Sequence,
                  dst_buf_bytes: Sequence[int], dst_owner: Sequence[int], **opts) -> Exchange:
    """Collective: every rank of the default process group calls this with the same metadata."""
    import torch.distributed as dist

    rank, world = (dist.get_rank(), dist.get_world_size()) if dist.is_initialized() else (0, 1)
    mine = needed_entries(src_metas, src_buf_bytes, dst_metas, dst_buf_bytes, dst_owner, rank, **opts)
    all_needs: List = [None] * world
    if world > 1:
        dist.all_gather_object(all_needs, mine)
    else:
        all_needs[0] = mine
    return build_exchange(src_metas, src_buf_bytes, src_owner, dst_metas, dst_buf_bytes, dst_owner, rank, world, all_needs, **opts)


def pack_sends(x: Exchange, src_metas: Sequence, local_blobs: Sequence, send_buf, stream=None) -> None:
    """Step 3, sender side: the needed entries of this rank's blobs, one segment per receiver,
    into `send_buf` (device, sum(send_bytes) bytes) with one multi-tensor pack.  The marshalled
    argument arrays are kept for as long as the blobs stay where they are."""
    key = tuple(b.data_ptr() for b in local_blobs)
    if x.pack_args is None or x.pack_args[0] != key:
        local_id = {b: i for i, b in enumerate(x.local_src)}
        ptrs, metas, base = [], [], 0
        for q in range(x.world):
            for i, o in zip(x.send_entries[q], x.send_offsets[q]):
                m = src_metas[i]
                ptrs.append(key[local_id[m.buf_index]] + m.byte_offset)
                metas.append((base + o, m.byte_length))
            base += x.send_bytes[q]
        x.pack_args = (key, api.marshal_pack(ptrs, metas), base)
    _, args, total = x.pack_args
    if total:
        api.bcp_pack_marshalled(args, send_buf, total, stream=stream)


def run_exchange(x: Exchange, src_metas: Sequence, local_blobs: Sequence, dst_bufs: Sequence, stream=None,
                 all_to_all: Optional[Callable] = None) -> None:
    """Steps 3 and 4 on the current device, asynchronous on `stream` (default: the current one).

    Main stream: pack the outgoing segments -> all-to-all -> copy the pieces that arrived.
    Side stream: once the pack has left the SMs, copy the pieces whose sources are this rank's own
    blobs; it runs while the segments travel (the paper overlaps the transfer between GPUs with the
    rest of the load pipeline, Sec. 4.1 / 4.2).  The main stream then waits for the side stream, so
    that work queued on `stream` afterwards sees complete targets.  The pack goes first on purpose:
    the copy kernels are persistent and fill every SM, so whatever is launched behind one waits for it.
    `all_to_all(recv, send, recv_splits, send_splits)` defaults to `torch.distributed.all_to_all_single`
    on `stream`.  Buffers, side stream and events live in the Exchange (x.bind); x.stage_ms() gives the
    device time of every stage after a synchronise."""
    import torch

    dev = local_blobs[0].device if local_blobs else dst_bufs[0].device
    x.bind(dev)
    main = torch.cuda.current_stream(dev) if stream is None else stream
    e = x.events
    srcs = x.sources(local_blobs)
    with torch.cuda.stream(main):
        e["begin"].record(main)
        pack_sends(x, src_metas, local_blobs, x.send_buf, main)
        e["packed"].record(main)
        if x.world > 1:
            if all_to_all is None:
                import torch.distributed as dist

                dist.all_to_all_single(x.recv_buf[: sum(x.recv_bytes)], x.send_buf[: sum(x.send_bytes)], list(x.recv_bytes),
                                       list(x.send_bytes))
            else:
                all_to_all(x.recv_buf, x.send_buf, list(x.recv_bytes), list(x.send_bytes))
        e["arrived"].record(main)
        # the local pieces, behind the pack and beside the transfer
        x.side.wait_event(e["packed"])
        e["local_begin"].record(x.side)
        if x.plan_local is not None:
            api.bcp_reshard(x.plan_local, srcs, dst_bufs, stream=x.side)
        e["local_done"].record(x.side)
        if x.plan_remote is not None:
            api.bcp_reshard(x.plan_remote, srcs, dst_bufs, stream=main)
        e["remote_done"].record(main)
        main.wait_event(e["local_done"])
        e["end"].record(main)


# ----------------------------------------------------------------------------- without an exchange
@dataclass
class ZeroCopy:
    """Cross-GPU resharding with no exchange step: this rank's plan for its own target buffers against
    the global saved metadata, and the addresses of ALL saved blobs (own pointers, peers' blobs mapped
    through bcp_ipc_open).  bcp_reshard then reads every tile where it lies."""

    rank: int
    world: int
    local_dst: List[int]
    dst_buf_bytes: List[int]
    plan: Optional[api.Plan]
    src_ptrs: List[int]                  # one address per saved blob, in global order
    opened: List[int] = field(default_factory=list)
    keep: List[object] = field(default_factory=list)   # own blobs, kept alive while peers may read them

    def run(self, dst_bufs: Sequence, stream=None) -> None:
        """Asynchronous on `stream`.  The caller orders it against the owners' writes of their blobs
        (a barrier between the processes before the first run and before anybody frees a blob)."""
        api.bcp_reshard(self.plan, self.src_ptrs, dst_bufs, stream=stream)

    def close(self) -> None:
        for p in self.opened:
            api.bcp_ipc_close(p)
        self.opened = []
        if self.plan is not None:
            self.plan.destroy()
            self.plan = None
        self.keep = []


def plan_zero_copy(src_metas: Sequence, src_buf_bytes: Sequence[int], src_owner: Sequence[int], dst_metas: Sequence,
                   dst_buf_bytes: Sequence[int], dst_owner: Sequence[int], local_blobs: Sequence, **opts) -> ZeroCopy:
    """Collective: every rank of the default process group calls this with the same metadata and its
    own blobs (device tensors, in the order of its entries in src_owner).  Handles of all blobs are
    gathered, every rank maps the blobs of the others, and plans its own targets against everything.
    Only the blobs a rank's plan reads are mapped."""
    import torch.distributed as dist

    rank, world = (dist.get_rank(), dist.get_world_size()) if dist.is_initialized() else (0, 1)
    mine = [b for b, o in enumerate(src_owner) if o == rank]
    assert len(mine) == len(local_blobs), "one device tensor per saved blob this rank owns"
    handles = {b: api.bcp_ipc_export(t) for b, t in zip(mine, local_blobs)} if world > 1 else {}
    everybody: List = [None] * world
    if world > 1:
        dist.all_gather_object(everybody, handles)
    local_dst, metas, sizes = _local_targets(dst_metas, dst_buf_bytes, dst_owner, rank)
    plan = api.bcp_plan(src_metas, src_buf_bytes, metas, sizes, **opts)
    wanted = {src_metas[i].buf_index for i in plan.used_sources()}
    own = dict(zip(mine, local_blobs))
    ptrs, opened = [], []
    try:
        for b in range(len(src_buf_bytes)):
            if b in own:
                ptrs.append(own[b].data_ptr())
            elif b in wanted:
                p = api.bcp_ipc_open(everybody[src_owner[b]][b])
                opened.append(p)
                ptrs.append(p)
            elif mine:
                ptrs.append(own[mine[0]].data_ptr())  # never read by this plan: any valid address will do
            else:  # a rank without blobs of its own has no address to spare: map the blob after all
                p = api.bcp_ipc_open(everybody[src_owner[b]][b])
                opened.append(p)
                ptrs.append(p)
    except Exception:
        for p in opened:
            api.bcp_ipc_close(p)
        plan.destroy()
        raise
    return ZeroCopy(rank, world, local_dst, sizes, plan, ptrs, opened, list(local_blobs))
