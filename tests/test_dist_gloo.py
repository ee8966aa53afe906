"""The N > 1 path of the benchmark on CPU: two gloo ranks line up, take the maximum of their timings and
compute the whole-job rate the way bench.py does (replicas, no collective on the data path)."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2510_05529_b200 import dist as d
    assert d.world() == (rank, world, rank)
    assert d.init("gloo")
    d.barrier()
    ms = [10.0 + rank, 20.0 - rank]                      # rank 0: [10, 20], rank 1: [11, 19]
    mx = d.max_over_ranks(ms)
    rate = d.whole_job_rate(1.0, world, mx[0] * 1e-3)
    # ranks that share the heads of the SAME sequences (bench.py --shard heads): the job still makes one token per step
    rate_heads = d.whole_job_rate(1.0, 1, mx[0] * 1e-3)
    out.put((rank, mx, rate, rate_heads))
    d.finish()


def test_two_gloo_ranks_take_the_max_and_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, rate, rate_heads in got:
        assert mx == [11.0, 20.0]
        assert abs(rate - 2.0 / 0.011) < 1e-9           # 2 sequences' tokens over the slowest rank's time
        assert abs(rate_heads - 1.0 / 0.011) < 1e-9     # one sequence's tokens, however many ranks split its heads


def test_single_process_is_identity():
    from paper_2510_05529_b200 import dist as d
    assert d.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert d.whole_job_rate(16, 1, 0.002) == 8000.0
