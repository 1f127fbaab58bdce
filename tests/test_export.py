"""Safetensors export: the header/layout is pinned on CPU by the real `safetensors` reader; the
device-side image is checked on the GPU."""
import json
import struct

import numpy as np
import pytest
import torch

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import api
from oracle import reshard_oracle as orc

safetensors_torch = pytest.importorskip("safetensors.torch")

ST = {torch.bfloat16: "BF16", torch.float32: "F32", torch.float16: "F16", torch.uint8: "U8", torch.int64: "I64",
      torch.int32: "I32", torch.float64: "F64", torch.bool: "BOOL", torch.int8: "I8", torch.int16: "I16"}


def _tensors(seed=0):
    g = torch.Generator().manual_seed(seed)
    return {
        "model.embed.weight": torch.randn(37, 24, generator=g).to(torch.bfloat16),
        "model.layers.0.attn.q.weight": torch.randn(16, 24, generator=g),
        "scalar": torch.tensor(3.5, dtype=torch.float64),
        "odd \"name\" \\ with\ttab": torch.randint(0, 255, (7,), generator=g, dtype=torch.uint8),
        "empty": torch.zeros((0, 5), dtype=torch.float16),
        "steps": torch.arange(11, dtype=torch.int64),
        "mask": torch.tensor([True, False, True]),
        "half.bf16.odd": torch.randn(3, generator=g).to(torch.bfloat16),
        "ids": torch.arange(9, dtype=torch.int32).reshape(3, 3),
    }


def _entries(ts):
    return [(k, ST[v.dtype], tuple(v.shape)) for k, v in ts.items()]


def _bytes(t):
    """uint8 view of a tensor's bytes (0-d and empty tensors included)."""
    return t.contiguous().reshape(-1).view(torch.uint8) if t.numel() else torch.zeros(0, dtype=torch.uint8)


def _raw(t):
    return _bytes(t).numpy()


def test_layout_is_read_by_the_safetensors_library():
    ts = _tensors()
    header, metas, total = bcp.bcp_safetensors_layout(_entries(ts))
    n = struct.unpack("<Q", header[:8])[0]
    assert len(header) == 8 + n and len(header) % 8 == 0
    meta = json.loads(header[8:].decode())
    pos = len(header)
    for (name, t), (off, length) in zip(ts.items(), metas):  # back to back, in order, offsets relative to the buffer
        assert meta[name]["data_offsets"] == [off - len(header), off - len(header) + length]
        assert off == pos and length == t.numel() * t.element_size() and meta[name]["shape"] == list(t.shape)
        pos += length
    assert pos == total
    # assemble the image on the host with the oracle's pack (no padding) and hand it to the real reader
    blob, table = orc.pack([_raw(t) for t in ts.values()], align=1)
    image = header + blob.tobytes()
    assert len(image) == total and [o + len(header) for o, _ in table] == [o for o, _ in metas]
    back = safetensors_torch.load(image)
    assert set(back) == set(ts)
    for k, t in ts.items():
        assert back[k].dtype == t.dtype and back[k].shape == t.shape
        assert torch.equal(_bytes(back[k]), _bytes(t))


def test_layout_errors():
    for bad in ([("a", "F33", (1,))], [("a", "F32", (1,)), ("a", "F32", (2,))], [("__metadata__", "F32", (1,))],
                [("", "F32", (1,))], [("a", "F32", (-1,))]):
        with pytest.raises(bcp.BcpError) as e:
            bcp.bcp_safetensors_layout(bad)
        assert e.value.code == api.ERR_INVALID
    header, metas, total = bcp.bcp_safetensors_layout([])
    assert metas == [] and total == len(header) and safetensors_torch.load(header) == {}


@pytest.mark.gpu
def test_device_export_round_trips_through_the_library(cuda_device):
    ts = _tensors(1)
    big = torch.randn(1 << 20, 33, generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)  # 69 MB, odd row length
    ts["big.weight"] = big
    dev = {k: v.to(cuda_device) for k, v in ts.items()}
    _, _, total = bcp.bcp_safetensors_layout(_entries(ts))
    file = torch.full((total + 64,), 0xA5, dtype=torch.uint8, device=cuda_device)
    for _ in range(2):
        n = bcp.bcp_safetensors_export(_entries(ts), [dev[k].data_ptr() if dev[k].numel() else 0 for k in ts], file)
        torch.cuda.synchronize()
        assert n == total and bool((file[total:] == 0xA5).all())
        back = safetensors_torch.load(file[:total].cpu().numpy().tobytes())
        for k, t in ts.items():
            assert back[k].dtype == t.dtype and back[k].shape == t.shape
            assert torch.equal(_bytes(back[k]), _bytes(t)), k
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_safetensors_export(_entries(ts), [dev[k].data_ptr() if dev[k].numel() else 0 for k in ts], file, file_cap=total - 1)
    assert e.value.code == api.ERR_CAPACITY
    bcp.bcp_pack_cache_clear()
