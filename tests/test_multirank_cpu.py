"""The N > 1 path of the bench on CPU: two gloo ranks.  The scan itself never communicates (ranks
are replicas); what the ranks share is the barrier and the max of their timings, and each rank
must draw its own inputs."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2603_14360_b200 import inputs
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        mine = [10.0 + rank, 5.0 - rank, 0.0]                # rank 1 is slower on the first, rank 0 on the second
        agreed = bench.max_over_ranks(mine, dist)
        cfg = inputs.CONFIGS["tiny_f32"]
        d = inputs.make_inputs(cfg, seed=bench.rank_input_seed(cfg.seed, rank, 0))
        q.put((rank, agreed, float(d["q"].double().sum()), bench.whole_job_tokens_per_s(cfg.tokens, world, agreed[0])))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_draw_their_own_inputs():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, s0, v0), (r1, t1, s1, v1) = got
    assert (r0, r1) == (0, 1)
    assert t0 == t1 == [11.0, 5.0, 0.0]                       # element-wise max over ranks
    assert s0 != s1                                           # different seeds -> different inputs
    assert v0 == v1 == 2 * 64 / 11e-3                         # both ranks' tokens over the slowest rank's time


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None) == [1.5, 2.5]
    assert bench.rank_input_seed(7, 0, 0) == 7 and bench.rank_input_seed(7, 1, 0) != bench.rank_input_seed(7, 0, 1)
