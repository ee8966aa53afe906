"""The N > 1 path of the benchmark on CPU: two gloo ranks line up, take the maximum of their timings and
compute the whole-job rate the way bench.py does (replicas, no collective on the data path), and split the
heads of one model between them the way `bench.py --shard heads` does."""
import os
import socket

import numpy as np
import pytest
import torch
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


# ---------------------------------------------------------------------------------------------------------
# Head-sharded replicas: the ranks split the KV heads (and their query heads) of the SAME sequences.
# ---------------------------------------------------------------------------------------------------------
def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _shard_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as tdist

    import h1b_synth
    import oracle
    from paper_2510_05529_b200 import dist as d
    assert d.init("gloo")
    # one small GQA model (8 query heads on 4 KV heads), the same seeds on every rank
    w = h1b_synth.scaled(h1b_synth.WORKLOADS["c4_gqa_32k"], n_layers=1, n_q_heads=8, n_kv_heads=4, sketch_bits=64,
                         batch=2, context=70)
    sh = d.shard_heads(w.n_q_heads, w.n_kv_heads, rank, world, w.head_dim)
    K, V = h1b_synth.kv_rows(w, 0, w.context)
    q = h1b_synth.queries(w, 0)
    Rt = h1b_synth.projection(h1b_synth.layer_seed(w, 0, 99), w.head_dim, w.sketch_bits)
    lens = np.array([70, 33], dtype=np.int32)
    # this rank's slice of the model's inputs, and the path's result on it (the oracle stands in for the GPU here)
    Kr, Vr = d.take_heads(K, sh.kv_begin, sh.n_kv), d.take_heads(V, sh.kv_begin, sh.n_kv)
    qr = d.take_heads(q, sh.q_begin, sh.n_q)
    mine = torch.from_numpy(oracle.layer(_bits(Kr), _bits(Vr), lens, _bits(qr), Rt, 16.0, w.group_size))
    # test plumbing only: collect everybody's slice bounds and outputs to check the layout (the product never does this)
    bounds = [None] * world
    tdist.all_gather_object(bounds, tuple(sh))
    outs = [torch.empty_like(mine) for _ in range(world)]
    tdist.all_gather(outs, mine)
    whole = oracle.layer(_bits(K), _bits(V), lens, _bits(q), Rt, 16.0, w.group_size)
    out.put((rank, bounds, float(np.abs(torch.cat(outs, dim=1).numpy() - whole).max()),
             bool(np.array_equal(mine.numpy(), whole[:, sh.q_begin:sh.q_begin + sh.n_q]))))
    d.finish()


def test_two_gloo_ranks_split_the_heads_of_one_model():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, bounds, err_concat, own_rows_match in got:
        # disjoint slices whose union is the whole head set, GQA groups whole
        assert bounds == [(0, 2, 0, 4), (2, 2, 4, 4)]
        # the ranks' outputs, concatenated along the head axis in rank order, are the unsharded [B][Hq][d] tensor
        assert err_concat == 0.0 and own_rows_match


def test_shard_heads_covers_every_head_once_and_refuses_what_does_not_divide():
    from paper_2510_05529_b200 import dist as d
    for hq, hkv, world, dim in ((32, 32, 8, 128), (32, 8, 4, 128), (32, 8, 8, 128), (8, 8, 2, 64), (28, 4, 2, 64), (48, 3, 3, 128)):
        gq = hq // hkv
        kv_seen, q_seen = [], []
        for r in range(world):
            sh = d.shard_heads(hq, hkv, r, world, dim)
            assert sh.n_q == sh.n_kv * gq and sh.q_begin == sh.kv_begin * gq          # a group is never cut
            if dim == 64:
                assert sh.n_kv % 2 == 0 and sh.kv_begin % 2 == 0                      # pairs of 64-wide heads stay together
            kv_seen += list(range(sh.kv_begin, sh.kv_begin + sh.n_kv))
            q_seen += list(range(sh.q_begin, sh.q_begin + sh.n_q))
        assert kv_seen == list(range(hkv)) and q_seen == list(range(hq))
    assert d.shard_heads(32, 8, 0, 1) == (0, 8, 0, 32)
    for bad in ((32, 8, 0, 3, 128), (32, 8, 0, 16, 128), (8, 8, 0, 8, 64), (12, 6, 0, 2, 64), (30, 8, 0, 2, 128), (8, 8, 2, 2, 128)):
        with pytest.raises(ValueError):
            d.shard_heads(*bad)
