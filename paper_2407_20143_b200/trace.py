"""Per-operation timing of the device path, after the paper's monitoring (Sec. 5.3, "Monitoring
and Analysis": every checkpointing operation reports its duration and the bytes it moved,
tagged with rank and step, so that slow ranks and stages show up in a timeline).

A `Trace` brackets stream work with CUDA events, so a span costs two event records and no
synchronisation; durations are read when the rows are asked for.

    tr = Trace(rank=0)
    with tr.span("reshard", nbytes=plan_bytes, step=3):
        bcp.bcp_reshard(plan, src, dst)
    rows = tr.rows()        # [{"name": "reshard", "rank": 0, "step": 3, "ms": ..., "bytes": ..., "gbps": ...}]
"""
from __future__ import annotations

import json
from contextlib import contextmanager
from typing import List, Optional


class Trace:
    def __init__(self, rank: int = 0):
        self.rank = rank
        self._spans: list = []

    @contextmanager
    def span(self, name: str, nbytes: int = 0, step: Optional[int] = None, stream=None):
        """Times everything enqueued on `stream` (default: the current stream) inside the block."""
        import torch

        s = stream if stream is not None else torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        try:
            yield
        finally:
            e1.record(s)
            self._spans.append((name, int(nbytes), step, e0, e1))

    def rows(self) -> List[dict]:
        """Waits for the recorded spans and returns one row per span, in recording order."""
        out = []
        for name, nbytes, step, e0, e1 in self._spans:
            e1.synchronize()
            ms = e0.elapsed_time(e1)
            out.append({"name": name, "rank": self.rank, "step": step, "ms": ms, "bytes": nbytes,
                        "gbps": nbytes / (ms * 1e-3) / 1e9 if ms > 0 and nbytes else None})
        return out

    def totals(self) -> dict:
        """Per operation name: calls, total ms, total bytes (the aggregation behind a heat map)."""
        agg: dict = {}
        for r in self.rows():
            a = agg.setdefault(r["name"], {"calls": 0, "ms": 0.0, "bytes": 0})
            a["calls"] += 1
            a["ms"] += r["ms"]
            a["bytes"] += r["bytes"]
        return agg

    def dump(self, path: str) -> None:
        with open(path, "w") as f:
            for r in self.rows():
                f.write(json.dumps(r) + "\n")

    def clear(self) -> None:
        self._spans = []
