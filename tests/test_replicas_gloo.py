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


class _StubModel:
    """Stands in for qzo.Model on CPU: the begin half reports this rank's loss sums, the finish half
    records what reached it."""

    def __init__(self, sums):
        self.sums = torch.tensor(sums, dtype=torch.float32)
        self.finish_args = None
        self.finish_calls = []
        self.begin_seeds = []

    def qzo_step_begin(self, tokens, labels, seed, eps):
        self.begin_seeds.append(seed)
        return self.sums.clone()

    def qzo_step_finish(self, sums, seed, eps, lr, clip, read_back=True):
        self.finish_args = (sums.tolist(), seed, eps, lr, clip)
        self.finish_calls.append(self.finish_args)
        return None


def _dp_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2505_13430_b200 import data_parallel as dp
        # rank 0: 10 kept tokens with loss sums 20 / 10, rank 1: 30 kept tokens with loss sums 120 / 150
        stub = _StubModel([20.0, 10.0, 10.0, 10.0] if rank == 0 else [120.0, 150.0, 30.0, 30.0])
        dp.dp_step(stub, None, None, seed=77, eps=1e-3, lr=1e-5, clip=100.0, read_back=False)
        out.put((rank,) + stub.finish_args)
    finally:
        dist.destroy_process_group()


def test_data_parallel_step_exchanges_four_floats_and_every_rank_finishes_alike():
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
    # the finish half of BOTH ranks got the element-wise sums and the same seed / eps / lr / clip, so the
    # library forms the same d' and applies the same seeded update on both
    for r in res:
        assert r[1] == [140.0, 160.0, 40.0, 40.0]
        assert r[2:] == (77, 1e-3, 1e-5, 100.0)
    assert res[0][1:] == res[1][1:]


def _dp_seed_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2505_13430_b200 import data_parallel as dp
        stub = _StubModel([20.0, 10.0, 10.0, 10.0] if rank == 0 else [120.0, 150.0, 30.0, 30.0])
        dp.dp_step_seed_per_rank(stub, None, None, seed_base=500, eps=1e-3, lr_per_seed=5e-6, clip=100.0, read_back=False)
        out.put((rank, stub.begin_seeds, stub.finish_calls))
    finally:
        dist.destroy_process_group()


def test_seed_per_rank_step_gathers_the_sums_and_applies_every_ranks_update_in_rank_order():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_seed_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # each rank perturbed with its own seed ...
    assert res[0][1] == [500] and res[1][1] == [501]
    # ... and both ranks applied the same two updates in the same order: rank 0's sums with seed 500, then rank 1's
    # sums with seed 501, each with the per-seed step size (nothing is added up: the estimates stay separate)
    want = [([20.0, 10.0, 10.0, 10.0], 500, 1e-3, 5e-6, 100.0), ([120.0, 150.0, 30.0, 30.0], 501, 1e-3, 5e-6, 100.0)]
    assert res[0][2] == want and res[1][2] == want
