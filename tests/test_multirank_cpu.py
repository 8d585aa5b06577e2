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


def test_bare_launch_with_gpus_2_starts_two_ranks():
    """`python bench.py --gpus 2` without a launcher must start its two ranks itself; the rank
    plumbing is exercised on host memory (gloo) and rank 0 prints the job-level line."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plumbing-check"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                              # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 15.0
    assert line["prompts"][0][0] != line["prompts"][1][0] and line["prompts"][0][1] != line["prompts"][1][1]
    assert np.isclose(line["value"], 2 * 2048 / 15e-3)
