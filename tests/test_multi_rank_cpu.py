"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.  The sparse decode MLP shards as
independent replicas (no data-path collective); what the ranks share is the timing protocol:
barrier, slowest rank's time, whole-job rate = all ranks' units / that time."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import dip_inputs as di
    # every rank draws its own sequence (seed offset by rank), as the benchmark does
    w = di.WORKLOADS["phi3_mini"].scaled(d_model=64)
    xs = di.token_inputs(w.scaled(seed=w.seed + 1000 * rank), n_tokens=4, batch=1)
    local_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(local_ms, dist, torch, "cpu")
    rate = bench.whole_job_rate(40 * 8, world, ms)
    out.put((rank, ms, rate, float(xs.sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_slowest_time_and_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, rate0, sum0), (r1, ms1, rate1, sum1) = res
    assert ms0 == ms1 == 20.0                         # the maximum over ranks, on every rank
    assert rate0 == rate1 == pytest.approx(40 * 8 * 2 / 0.020)
    assert sum0 != sum1                               # the replicas run different sequences


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5, None, torch, "cpu") == 7.5
    assert bench.whole_job_rate(100, 1, 50.0) == pytest.approx(2000.0)
