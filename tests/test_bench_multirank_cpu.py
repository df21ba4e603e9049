"""The multi-GPU form of the benchmark is N independent replicas (no data-path collective): the only
cross-rank logic is the max-over-ranks timing and the summed value.  Checked with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import sys
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    from workloads import get_config
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    cfg = get_config("c5")
    out[rank] = (ms, bench.job_value(cfg, world, 50, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        out = mgr.dict()
        port = _free_port()
        procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert out[0] == out[1]
        ms, value = out[0]
        assert ms == 15.0
        assert value == pytest.approx(2 * 80 * 512 * 50 / 15e-3)


def test_single_process_is_the_identity():
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
