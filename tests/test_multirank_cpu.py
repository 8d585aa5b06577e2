"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The path shards by prompt (independent
problems, no data-path collective); what crosses ranks is the rendezvous, the per-rank workload
seeds and the max-over-ranks of the step time."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2604_06746_b200 import synth
    wl = synth.WORKLOADS["tiny"]
    mine = bench.rank_workload(wl, rank)
    pl = synth.plan(mine)
    q = synth.make_layer(mine, pl, 0, device="cpu", with_v=False)["q_win"]
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu", world)          # rank 1 is the slow one
    digests = [None] * world
    dist.all_gather_object(digests, (mine.index, float(q.double().sum())))
    if rank == 0:
        out.put((ms, digests, bench.job_tokens_per_second(wl.seq, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_get_distinct_prompts_and_the_slowest_step_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, digests, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0                                                   # the maximum over ranks
    assert digests[0][0] != digests[1][0] and digests[0][1] != digests[1][1]   # different seeds, different data
    assert np.isclose(value, 2 * 2048 / 15e-3)                          # whole-job tokens per second
