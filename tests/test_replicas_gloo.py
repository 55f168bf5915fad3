"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective);
the slowest rank's time decides the whole-job rate and every replica draws its own inputs."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_13430_b200 import inputs, replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 100.0 + 50.0 * rank                      # rank 1 is the slow one
        slowest = replicas.max_over_ranks(ms)
        mseed, tseed = replicas.rank_seeds(1000, 7, rank)
        cfg = inputs.model_cfg("tiny")
        tok, _ = inputs.tokens_and_labels(cfg, 2, 8, seed=tseed)
        dist.barrier()
        out.put((rank, slowest, replicas.whole_job_rate(5, world, slowest), mseed, tok.flatten().tolist()))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_draw_distinct_batches():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [150.0, 150.0]                 # max over ranks, seen by both
    assert all(abs(r[2] - 2 * 5 / 0.150) < 1e-9 for r in res)    # whole-job steps/s
    assert res[0][3] != res[1][3] and res[0][4] != res[1][4]     # own weights seed, own batch


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(12.5) == 12.5
    assert replicas.whole_job_rate(10, 1, 2000.0) == 5.0


def _dp_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2505_13430_b200 import data_parallel as dp
        # rank 0: 10 tokens with mean loss 2.0 / 1.0, rank 1: 30 tokens with mean loss 4.0 / 5.0
        n = 10 if rank == 0 else 30
        lp = dp.global_mean_loss(2.0 if rank == 0 else 4.0, n)
        lm = dp.global_mean_loss(1.0 if rank == 0 else 5.0, n)
        out.put((rank, lp, lm) + dp.directional_derivative(lp, lm, 1e-3, 100.0))
    finally:
        dist.destroy_process_group()


def test_data_parallel_exchange_is_two_scalars_and_every_rank_gets_the_same_d():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # token-weighted means: l+ = (10*2 + 30*4)/40 = 3.5, l- = (10*1 + 30*5)/40 = 4.0; d = -250 -> d' = -100
    for r in res:
        assert abs(r[1] - 3.5) < 1e-12 and abs(r[2] - 4.0) < 1e-12
        assert abs(r[3] + 250.0) < 1e-3 and r[4] == -100.0
    assert res[0][1:] == res[1][1:]                      # identical on both ranks -> identical seeded update
