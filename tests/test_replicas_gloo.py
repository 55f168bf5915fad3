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
