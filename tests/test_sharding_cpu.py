"""Host logic of the sharded population (paper_1711_09846_b200/sharding.py) without a GPU: the partition, the copy
plan, and the two exchanges between two gloo ranks, against the oracle's copy maps (truncation selection and the
binary tournament, whose chained copies need several passes) and the definition "every recipient ends with its
donor's record as it was before the ready point"."""
import os
import socket

import numpy as np
import pytest
import torch.multiprocessing as mp

from oracle import pbt_oracle as O
from paper_1711_09846_b200 import sharding as S


def test_partition_covers_every_member_once():
    for n in range(0, 41):
        for world in (1, 2, 3, 4, 8):
            seen = []
            for r in range(world):
                a, b = S.member_range(r, world, n)
                assert 0 <= a <= b <= n and b - a in (n // world, n // world + 1)
                seen += list(range(a, b))
                for m in range(a, b):
                    assert S.owner_of(m, world, n) == r
            assert seen == list(range(n))


def _levels(src):
    """Copy pass of every recipient: one more than the deepest chain of members that read it (definition)."""
    n = len(src)
    readers = {d: [b for b in range(n) if src[b] == d and b != d] for d in range(n)}

    def depth(b):
        return 0 if not readers[b] or src[b] == b else 1 + max(depth(r) for r in readers[b])
    return [depth(b) if src[b] != b else 0 for b in range(n)]


@pytest.mark.parametrize("rule", ["truncation", "tournament"])
def test_copy_plan_against_the_oracle_copy_map(rule):
    rng = np.random.default_rng(3)
    for n in (2, 5, 7, 16, 33):
        for world in (1, 2, 3):
            f = rng.standard_normal(n).astype(np.float32)
            src = O.truncation_select(f, 0, 1, 2, 5) if rule == "truncation" else O.tournament_select(f, 0, 1)
            level = _levels([int(x) for x in src])
            plan = S.CopyPlan.from_copy_map(src, level, world)
            pairs = [(b, int(src[b])) for b in range(n) if src[b] != b]
            got = sorted(p for v in plan.local.values() for p in v) + sorted(p for v in plan.recv.values() for p in v)
            assert sorted(got) == pairs                                   # every copy exactly once
            assert sorted(p for v in plan.send.values() for p in v) == sorted(p for v in plan.recv.values() for p in v)
            for (r, l), v in plan.local.items():
                assert all(S.owner_of(b, world, n) == r == S.owner_of(d, world, n) and level[b] == l for b, d in v)
            for (r, l), v in plan.send.items():
                assert all(S.owner_of(d, world, n) == r != S.owner_of(b, world, n) and level[b] == l for b, d in v)
            for (r, l), v in plan.recv.items():
                assert all(S.owner_of(b, world, n) == r != S.owner_of(d, world, n) and level[b] == l for b, d in v)
            if rule == "truncation":
                assert plan.n_levels <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n, rule, out):
    import sys
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    from oracle import pbt_oracle as O2
    from paper_1711_09846_b200 import sharding as S2
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    a, b = S2.member_range(rank, world, n)
    # a fake shard: per local member two "slabs" whose contents identify the member
    slabs = {m: [torch.full((5,), float(m)), torch.full((3,), 100.0 + m, dtype=torch.float64)] for m in range(a, b)}
    # exchange 1: fitness of the local members -> the whole vector on every rank
    f_all = np.random.default_rng(11).standard_normal(n).astype(np.float32)           # what a single process would see
    mine = torch.from_numpy(f_all[a:b].copy())
    gathered = S2.all_gather_rows(mine, world, n).numpy()
    src = O2.truncation_select(gathered, 0, 0, 2, 5) if rule == "truncation" else O2.tournament_select(gathered, 0, 0)
    nn = len(src)
    readers = {d: [x for x in range(nn) if src[x] == d and x != d] for d in range(nn)}

    def depth(x):
        return 0 if not readers[x] or src[x] == x else 1 + max(depth(r) for r in readers[x])
    level = [depth(x) if src[x] != x else 0 for x in range(nn)]
    plan = S2.CopyPlan.from_copy_map(src, level, world)
    # exchange 2, pass by pass: local copies, then the records that cross ranks
    for lv in range(plan.n_levels):
        snapshot = {m: [t.clone() for t in ts] for m, ts in slabs.items()}
        for bb, d in plan.local.get((rank, lv), []):
            for t, s in zip(slabs[bb], snapshot[d]):
                t.copy_(s)
        S2.exchange_level(plan, rank, lv, lambda m: slabs[m])
    out[rank] = (gathered.tolist(), [int(x) for x in src], {m: [t.tolist() for t in ts] for m, ts in slabs.items()},
                 plan.crossing())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("rule,n", [("truncation", 10), ("truncation", 7), ("tournament", 12), ("tournament", 9)])
def test_two_gloo_ranks_end_with_the_donors_records(rule, n):
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        out = mgr.dict()
        port = _free_port()
        procs = [ctx.Process(target=_rank_main, args=(r, 2, port, n, rule, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(180)
            assert p.exitcode == 0
        res = dict(out)
    f_all = np.random.default_rng(11).standard_normal(n).astype(np.float32)
    want_src = O.truncation_select(f_all, 0, 0, 2, 5) if rule == "truncation" else O.tournament_select(f_all, 0, 0)
    merged = {}
    for r in range(2):
        gathered, src, slabs, crossing = res[r]
        assert np.array_equal(np.asarray(gathered, dtype=np.float32), f_all)      # identical fitness vector on every rank
        assert src == [int(x) for x in want_src]                                  # hence the identical copy map
        merged.update(slabs)
    assert sorted(merged) == list(range(n))
    for b in range(n):
        d = int(want_src[b])                                                       # the donor's record before the ready point
        assert merged[b][0] == [float(d)] * 5 and merged[b][1] == [100.0 + d] * 3, (b, d)
    assert res[0][3] == res[1][3]
    if rule == "tournament":
        assert res[0][3] > 0                                                       # some records did cross ranks
