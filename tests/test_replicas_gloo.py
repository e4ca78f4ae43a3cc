"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks, no GPU.  The path has no exchange
step, so what there is to check is the timing reduction (slowest rank decides), the whole-job
rate, and that replicas draw different inputs while one rank's inputs stay reproducible."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_15475_b200 import replicas, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_here = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
        rate, ms_step = replicas.whole_job_rate(1536, 5, ms_here, dist)
        w = wl.scaled(wl.CONFIGS["c2"], B=2, V=512)
        inp = wl.make_inputs(w, call=replicas.replica_call_index(rank, 0))
        digest = float(inp["target"].float().sum())
        gathered = [None] * world
        dist.all_gather_object(gathered, (rate, ms_step, digest))
        dist.barrier()
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (rate0, ms0, d0), (rate1, ms1, d1) = got
    assert ms0 == ms1 == 5.0                           # 25 ms over 5 steps: the slow rank's time
    assert rate0 == rate1 == 2 * 1536 / 5e-3          # both replicas' rows over that time
    assert d0 != d1                                    # replicas race different batches


def test_single_rank_needs_no_process_group():
    rate, ms_step = replicas.whole_job_rate(100, 4, 8.0, None)
    assert ms_step == 2.0 and rate == 100 / 2e-3
    assert replicas.max_over_ranks(3.5) == 3.5
    a = wl.make_inputs(wl.scaled(wl.CONFIGS["c2"], B=1, V=64), call=replicas.replica_call_index(3, 1))
    b = wl.make_inputs(wl.scaled(wl.CONFIGS["c2"], B=1, V=64), call=replicas.replica_call_index(3, 1))
    assert torch.equal(a["target"], b["target"]) and torch.equal(a["seeds"], b["seeds"])
