"""Worst-fit save-side de-duplication (Sec. 4.1): oracle pins and library parity (CPU only)."""
import os

import numpy as np
import pytest

import paper_2407_20143_b200 as bcp
from paper_2407_20143_b200 import api
from oracle import reshard_oracle as orc
from workloads.configs import CONFIGS, MIXED
from workloads.layouts import Parallelism, _collect_shards, build_state, gpt_model

from helpers import GOLDEN


def read_example():
    sizes, holders, owners, loads, n = [], [], [], [], 0
    for line in open(os.path.join(GOLDEN, "worst_fit_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("ranks"):
            n = int(line.split()[1])
            continue
        a, b, c, d = [x.strip() for x in line.split("|")]
        sizes.append(int(a))
        holders.append([int(x) for x in b.split()])
        owners.append(int(c))
        loads.append([int(x) for x in d.split()])
    return n, sizes, holders, owners, loads


def test_hand_worked_example():
    n, sizes, holders, owners, loads = read_example()
    for k in range(1, len(sizes) + 1):  # every prefix reproduces the written-down state
        o, l = orc.worst_fit(sizes[:k], holders[:k], n)
        assert o == owners[:k] and l == loads[k - 1]
        assert bcp.bcp_dedup_assign(sizes[:k], holders[:k], n) == (o, l)


@pytest.mark.parametrize("seed", range(30))
def test_invariants_and_parity_random(seed):
    rng = np.random.default_rng(seed)
    n_ranks = int(rng.integers(1, 9))
    n = int(rng.integers(0, 60))
    sizes = [int(x) for x in rng.integers(0, 1000, n)]
    holders = [sorted(rng.choice(n_ranks, size=int(rng.integers(1, n_ranks + 1)), replace=False).tolist()) for _ in range(n)]
    init = [int(x) for x in rng.integers(0, 500, n_ranks)]
    owners, load = orc.worst_fit(sizes, holders, n_ranks, init)
    assert all(o in h for o, h in zip(owners, holders))
    assert sum(load) == sum(init) + sum(sizes)
    assert bcp.bcp_dedup_assign(sizes, holders, n_ranks, init) == (owners, load)


def test_list_scheduling_bound():
    """When every rank holds every shard the rule is greedy list scheduling: the spread of the
    final loads never exceeds the largest shard, and equal shards end within one shard."""
    rng = np.random.default_rng(3)
    for n_ranks in (2, 5, 16):
        sizes = [int(x) for x in rng.integers(1, 10_000, 500)]
        holders = [list(range(n_ranks))] * len(sizes)
        _, load = orc.worst_fit(sizes, holders, n_ranks)
        assert max(load) - min(load) <= max(sizes)
        _, load = orc.worst_fit([7] * 101, [list(range(n_ranks))] * 101, n_ranks)
        assert max(load) - min(load) <= 7 and sum(load) == 707


def test_matches_the_generator_on_a_real_layout():
    """Third, independent implementation: the synthetic-workload generator de-duplicates the
    saved side with the same rule; owners must agree shard by shard."""
    m = gpt_model("gpt-s", L=4, H=64, F=256, V=512, P=32)
    par = Parallelism(tp=2, pp=2, dp=2, zero="zero1")
    shards = _collect_shards(m, par, MIXED)
    sizes = [s.nbytes for s in shards]
    holders = [s.holders for s in shards]
    owners, load = bcp.bcp_dedup_assign(sizes, holders, par.world)
    state = build_state(m, par, MIXED, dedup=True)
    per_rank = [0] * par.world
    for e in state.metas:
        per_rank[e.buf_index] += e.byte_length
    assert per_rank == load


def test_errors_leave_outputs_alone():
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_dedup_assign([1, 2], [[0], []], 2)
    assert e.value.code == api.ERR_INVALID
    with pytest.raises(bcp.BcpError) as e:
        bcp.bcp_dedup_assign([1], [[3]], 2)
    assert e.value.code == api.ERR_BOUNDS
    with pytest.raises(orc.OracleError):
        orc.worst_fit([1], [[]], 2)
