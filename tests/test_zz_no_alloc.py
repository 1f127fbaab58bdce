"""bcp_pack_static: the pack entry point for callers that cannot allocate device memory
(their own pool owns it all, or they call from a place where allocating is forbidden).

It keeps its work list in a fixed device array inside the library, so this test checks what
that design could get wrong: the result must equal bcp_pack's and the CPU oracle's byte for
byte, on two calls in a row with different layouts (the second call sees the first call's
leftovers in the array), with work lists that fill the fixed array to its last slot, and
requests beyond either fixed capacity must be refused with a clear error and nothing written.
Collected last on purpose (file name), so a run that stops at the first failure has already
run everything else.
"""
import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from oracle import reshard_oracle as orc
from paper_2407_20143_b200 import api

pytestmark = pytest.mark.gpu


def _make(device, sizes, seed, misalign=0, align=256):
    # all tensors are slices of one host-generated backing buffer (one upload, no device-side fill)
    rng = np.random.default_rng(seed)
    starts, pos = [], 0
    for i, n in enumerate(sizes):
        pos = (pos + 15) // 16 * 16 + ((misalign * (i + 1)) % 16 if misalign else 0)
        starts.append(pos)
        pos += n
    host = rng.integers(1, 256, size=pos + 16, dtype=np.uint8)
    back = torch.from_numpy(host).to(device)
    tensors = [back[a:a + n] for a, n in zip(starts, sizes)]
    offs, total = bcp.bcp_pack_layout(sizes, align)
    return tensors, list(zip(offs, sizes)), total, [host[a:a + n] for a, n in zip(starts, sizes)]


def _both(device, sizes, seed, misalign=0, align=256, oracle=True):
    tensors, metas, total, host = _make(device, sizes, seed, misalign, align)
    want = torch.full((total,), 0xA5, dtype=torch.uint8, device=device)
    bcp.bcp_pack(tensors, metas, want)
    got_back = torch.full((total + 8192,), 0x5A, dtype=torch.uint8, device=device)
    got = got_back[4096:4096 + total]
    bcp.bcp_pack_static(tensors, metas, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want), "static-scratch pack differs from bcp_pack"
    assert bool((got_back[:4096] == 0x5A).all()) and bool((got_back[4096 + total:] == 0x5A).all())
    if oracle:
        ref, table = orc.pack(host, align)
        assert [int(o) for o, _ in table] == [int(o) for o, _ in metas]
        assert np.array_equal(got.cpu().numpy(), ref), "static-scratch pack differs from the CPU oracle"
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
    _both(cuda_device, [700_000_000, 500_000_000], seed=3, oracle=False)
    bcp.bcp_pack_cache_clear()


def test_many_warp_sized_units(cuda_device):
    # A 100-byte tensor at 256-byte alignment is four units under 4 KiB (16-byte body and ragged
    # tail of the tensor, ragged head and body of the padding): 2,000 of them make 8,000 warp
    # units, 3,072 fill the fixed work list to its last slot (12,288), with odd addresses more
    # units per tensor but fewer tensors.  All inside the documented limits, so all must be exact.
    _both(cuda_device, [100] * 2000, seed=4)
    _both(cuda_device, [100] * 3072, seed=5)
    _both(cuda_device, [100 + (i % 7) for i in range(1500)], seed=6, misalign=5)
    # mixed: CTA-wide units in front of thousands of warp units, twice in a row
    mixed = [1 << 20, 300_000] + [100] * 2500 + [70_000] * 40
    _both(cuda_device, mixed, seed=7)
    _both(cuda_device, mixed[::-1], seed=8, misalign=3)
    bcp.bcp_pack_cache_clear()


def test_padding_only_and_trailing_padding(cuda_device):
    # no tensors at all: the whole blob is padding and comes back as zeros
    blob = torch.full((5000,), 9, dtype=torch.uint8, device=cuda_device)
    bcp.bcp_pack_static([], [], blob)
    torch.cuda.synchronize()
    assert bool((blob == 0).all())
    # a blob that ends in a long stretch of padding after its last tensor
    t = torch.arange(1, 200, dtype=torch.uint8, device=cuda_device)
    blob = torch.full((100_000,), 9, dtype=torch.uint8, device=cuda_device)
    bcp.bcp_pack_static([t], [(48, t.numel())], blob)
    torch.cuda.synchronize()
    got = blob.cpu().numpy()
    assert not got[:48].any() and np.array_equal(got[48:48 + 199], t.cpu().numpy()) and not got[48 + 199:].any()


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
    # the work-unit limit: 3,073 tensors of 100 bytes need 12,292 units, all far below the
    # smallest unit size, so growing the unit size cannot help
    n = 3073
    t = torch.zeros(100, dtype=torch.uint8, device=cuda_device)
    offs, total = bcp.bcp_pack_layout([100] * n, 256)
    blob = torch.full((total,), 7, dtype=torch.uint8, device=cuda_device)
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_pack_static([t] * n, list(zip(offs, [100] * n)), blob)
    assert e.value.code == api.ERR_CAPACITY and "12288" in str(e.value)
    torch.cuda.synchronize()
    assert bool((blob == 7).all()), "a refused call must not write"


def test_a_capturing_stream_is_refused(cuda_device):
    t = torch.ones(64, dtype=torch.uint8, device=cuda_device)
    blob = torch.zeros(256, dtype=torch.uint8, device=cuda_device)
    bcp.bcp_pack_static([t], [(0, 64)], blob)  # first call on the device, outside any capture
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        g.capture_begin()
        try:
            with pytest.raises(bcp.BcpError) as e:
                bcp.bcp_pack_static([t], [(0, 64)], blob, stream=s)
            assert e.value.code == api.ERR_INVALID
        finally:
            g.capture_end()
