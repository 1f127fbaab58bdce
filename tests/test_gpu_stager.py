"""Asynchronous save / load staging through the pinned ping-pong pool (GPU)."""
import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import api
from oracle import reshard_oracle as orc

pytestmark = pytest.mark.gpu


def _tensors(device, sizes, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    host = [torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g) for n in sizes]
    return host, [h.to(device) for h in host]


def test_save_two_in_flight_then_load_back(cuda_device):
    sizes_a = [3_000_000, 17, 70_001, 4096, 1, 1 << 20]
    sizes_b = [999_999, 5, 2_500_000]
    host_a, dev_a = _tensors(cuda_device, sizes_a, 1)
    host_b, dev_b = _tensors(cuda_device, sizes_b, 2)
    offs_a, total_a = bcp.bcp_pack_layout(sizes_a, 256)
    offs_b, total_b = bcp.bcp_pack_layout(sizes_b, 256)
    want_a, _ = orc.pack([h.numpy() for h in host_a], 256)
    want_b, _ = orc.pack([h.numpy() for h in host_b], 256)
    st = bcp.Stager(max(total_a, total_b), 2)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        slot_a = st.save(dev_a, list(zip(offs_a, sizes_a)), total_a, stream=s)
        # the tensors may be overwritten as soon as the stream has passed the pack
        for d in dev_a:
            d.zero_()
        slot_b = st.save(dev_b, list(zip(offs_b, sizes_b)), total_b, stream=s)
    assert slot_a != slot_b
    with pytest.raises(bcp.BcpError) as e:  # both slots busy
        st.save(dev_b, list(zip(offs_b, sizes_b)), total_b, stream=s)
    assert e.value.code == api.ERR_CAPACITY
    got_a = st.host_view(st.wait(slot_a), total_a).copy()
    got_b = st.host_view(st.wait(slot_b), total_b).copy()
    assert np.array_equal(got_a, want_a) and np.array_equal(got_b, want_b)
    st.release(slot_a)
    st.release(slot_b)
    # load: fill a pinned slot with the oracle's blob and unpack it on the device
    slot, addr = st.acquire()
    st.host_view(addr, total_b)[:] = want_b
    out = [torch.full((n,), 0xA5, dtype=torch.uint8, device=cuda_device) for n in sizes_b]
    st.load(slot, total_b, list(zip(offs_b, sizes_b)), out)
    torch.cuda.synchronize()
    for o, h in zip(out, host_b):
        assert torch.equal(o.cpu(), h)
    st.release(slot)
    # a slot that carried a load is reused for a save
    host_c, dev_c = _tensors(cuda_device, sizes_a, 3)
    for _ in range(3):
        k = st.save(dev_c, list(zip(offs_a, sizes_a)), total_a)
        got = st.host_view(st.wait(k), total_a).copy()
        st.release(k)
        assert np.array_equal(got, orc.pack([h.numpy() for h in host_c], 256)[0])
    with pytest.raises(bcp.BcpError):
        st.save(dev_c, list(zip(offs_a, sizes_a)), st.slot_bytes + 256)
    with pytest.raises(bcp.BcpError):
        st.release(0)  # not in use
    st.destroy()
    bcp.bcp_pack_cache_clear()


def test_bad_arguments(cuda_device):
    with pytest.raises(bcp.BcpError):
        bcp.Stager(100, 2)  # not a multiple of 256
    with pytest.raises(bcp.BcpError):
        bcp.Stager(4096, 0)
