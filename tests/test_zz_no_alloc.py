"""bcp_pack_static: the pack entry point for callers that cannot allocate device memory
(their own pool owns it all, or they call from a place where allocating is forbidden).

It keeps its work list in a fixed device array inside the library, so this test checks what
that design could get wrong: the result must equal bcp_pack's byte for byte, on two calls in a
row with different layouts (the second call sees the first call's leftovers in the array), and
requests beyond the fixed capacity must be refused with a clear error and nothing written.
Collected last on purpose (file name), so a run that stops at the first failure has already
run everything else.
"""
import pytest
import torch

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import api

pytestmark = pytest.mark.gpu


def _make(device, sizes, seed, misalign=0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    tensors = []
    for i, n in enumerate(sizes):
        back = torch.randint(1, 256, (n + 32,), dtype=torch.uint8, generator=g).to(device)
        off = (misalign * (i + 1)) % 16 if misalign else 0
        tensors.append(back[off:off + n])
    offs, total = bcp.bcp_pack_layout(sizes, 256)
    return tensors, list(zip(offs, sizes)), total


def _both(device, sizes, seed, misalign=0):
    tensors, metas, total = _make(device, sizes, seed, misalign)
    want = torch.full((total,), 0xA5, dtype=torch.uint8, device=device)
    bcp.bcp_pack(tensors, metas, want)
    got_back = torch.full((total + 8192,), 0x5A, dtype=torch.uint8, device=device)
    got = got_back[4096:4096 + total]
    bcp.bcp_pack_static(tensors, metas, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want), "static-scratch pack differs from bcp_pack"
    assert bool((got_back[:4096] == 0x5A).all()) and bool((got_back[4096 + total:] == 0x5A).all())
    return tensors, metas, want


def test_two_calls_in_a_row_match_bcp_pack(cuda_device):
    # first call: many tensors, small and large, some starting at odd addresses
    big = [3_000_000, 17, 70_001, 4096, 1, 255, 257, 1 << 20, 999_999, 0, 65536] + [1000 + 13 * i for i in range(300)]
    _both(cuda_device, big, seed=1, misalign=3)
    # second call, directly after: fewer and different tensors; stale units of the first call must not run
    small = [5, 100_003, 12_345, 64]
    tensors, metas, want = _both(cuda_device, small, seed=2)
    # and once more into the same blob on a side stream (ordered after the first by a sync)
    s = torch.cuda.Stream()
    again = torch.zeros_like(want)
    with torch.cuda.stream(s):
        bcp.bcp_pack_static(tensors, metas, again, stream=s)
    s.synchronize()
    assert torch.equal(again, want)
    bcp.bcp_pack_cache_clear()


def test_large_blob_grows_the_unit_size(cuda_device):
    # 1.2 GB in two tensors: more than 12288 units of 64 KiB, so the unit size has to double
    _both(cuda_device, [700_000_000, 500_000_000], seed=3)
    bcp.bcp_pack_cache_clear()


def test_capacity_is_enforced(cuda_device):
    n = 4097
    t = torch.zeros(16, dtype=torch.uint8, device=cuda_device)
    offs, total = bcp.bcp_pack_layout([16] * n, 16)
    blob = torch.full((total,), 7, dtype=torch.uint8, device=cuda_device)
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_pack_static([t] * n, list(zip(offs, [16] * n)), blob)
    assert e.value.code == api.ERR_CAPACITY and "4096" in str(e.value)
    torch.cuda.synchronize()
    assert bool((blob == 7).all()), "a refused call must not write"
    with pytest.raises(bcp.BcpError):
        bcp.bcp_pack_static([t, t], [(0, 16), (8, 16)], blob)  # overlapping table
