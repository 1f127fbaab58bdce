"""Input generators: closed-form byte totals, layout sanity, fill closed forms."""
import numpy as np
import pytest
import torch

from workloads import fills
from workloads.configs import CONFIGS, EXPECTED_TOTALS, scenario_cases
from workloads.layouts import Parallelism, build_state, gpt_model
from workloads.configs import MIXED
from workloads.meta import FLAT_SLICE, ShardMeta


@pytest.mark.parametrize("name", list(CONFIGS))
def test_config_byte_totals(name):
    c = CONFIGS[name]()
    assert (c.src.total_bytes, c.dst.total_bytes) == EXPECTED_TOTALS[name]
    for st in (c.src, c.dst):
        ends = {}
        for m in st.metas:
            assert m.byte_offset + m.byte_length <= st.buf_bytes[m.buf_index]
            ends.setdefault(m.buf_index, []).append((m.byte_offset, m.byte_offset + m.byte_length))
        for iv in ends.values():
            iv.sort()
            assert all(a[1] <= b[0] for a, b in zip(iv, iv[1:])), "entries overlap inside a buffer"


def test_cfg_shapes_are_the_named_models():
    assert CONFIGS["cfg1"]().src.total_bytes == 1_874_944 * 14
    assert CONFIGS["cfg2"]().src.total_bytes == 1_315_819_520 * 14
    assert CONFIGS["cfg3"]().src.total_bytes == 8_030_261_248 * 2
    assert CONFIGS["cfg4"]().src.total_bytes == 3_212_749_824 * 12
    assert CONFIGS["cfg5"]().src.total_bytes == 9_263_187_968 * 6


def test_zero1_slice_lengths():
    # per-rank flat slice of a model-parallel rank's local tensors: ceil(N / DP)
    m = gpt_model("gpt-tiny", L=2, H=256, F=1024, V=1024, P=128)
    st = build_state(m, Parallelism(tp=2, dp=2, zero="zero1"), MIXED, dedup=False)
    per = {}
    for e in st.metas:
        if e.fqn.startswith("optim.master."):
            per[e.buf_index] = per.get(e.buf_index, 0) + e.numel
    assert set(per.values()) == {477_824}


def test_worst_fit_balances_saved_bytes():
    c = CONFIGS["cfg2"]()
    assert max(c.src.buf_bytes) < 1.15 * (sum(c.src.buf_bytes) / len(c.src.buf_bytes))


def test_index_fill_closed_form():
    # a box entry and a flat entry of a (5, 7) tensor
    box = ShardMeta("w", 4, 2, (5, 7), (1, 2), (3, 4))
    flat = ShardMeta("w", 4, 2, (5, 7), (1, 2), (3, 4), kind=FLAT_SLICE, flat_begin=3, flat_end=9)
    g = np.arange(35).reshape(5, 7)[1:4, 2:6]
    s = fills.salt(3)
    got = fills.entry_bytes(box, 3, "index", 0, "cpu").numpy().view(np.uint32)
    assert np.array_equal(got, (g.ravel() + s).astype(np.uint32))
    got = fills.entry_bytes(flat, 3, "index", 0, "cpu").numpy().view(np.uint32)
    assert np.array_equal(got, (g.ravel()[3:9] + s).astype(np.uint32))
    b2 = ShardMeta("w", 2, 1, (5, 7), (1, 2), (3, 4))
    got = fills.entry_bytes(b2, 3, "index", 0, "cpu").numpy().view(np.uint16)
    assert np.array_equal(got, ((g.ravel() + s) % 65521).astype(np.uint16))


def test_pool_fill_statistics_and_bf16_rounding():
    m4 = ShardMeta("w", 4, 2, (1 << 16,), (0,), (1 << 16,))
    u = fills.entry_bytes(m4, 0, "uniform", 7, "cpu").numpy().view(np.float32)
    assert -1.0 <= u.min() and u.max() < 1.0 and abs(float(u.mean())) < 0.02
    n = fills.entry_bytes(m4, 0, "normal", 7, "cpu").numpy().view(np.float32)
    assert abs(float(n.std()) - 0.02) < 0.002
    m2 = ShardMeta("w", 2, 1, (1 << 16,), (0,), (1 << 16,))
    h = fills.entry_bytes(m2, 0, "normal", 7, "cpu")
    ref = torch.from_numpy(n.copy()).to(torch.bfloat16).view(torch.int16).view(torch.uint8)
    assert torch.equal(h, ref.reshape(-1))


def test_scenarios_build():
    cs = scenario_cases()
    assert len(cs) >= 12
    for c in cs:
        assert c.src.total_bytes > 0 and c.dst.total_bytes >= c.src.total_bytes
