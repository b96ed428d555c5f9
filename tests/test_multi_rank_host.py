"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own
batch, combined as (sum of units) / (max of times)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workload as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_29364_b200 import dist_util

    cfg = dist_util.rank_config(W.CONFIGS["tiny"], rank)
    meta = W.make_batch_meta(cfg)
    ms_local = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    ms, units = dist_util.combine(ms_local, cfg.batch)
    thr = dist_util.job_throughput(ms_local, cfg.batch)
    out.put((rank, cfg.seed, meta.ctx_len.tolist(), ms, units, thr))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_combine_max_time_and_sum_of_units():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, ctx0, ms0, u0, thr0), (r1, seed1, ctx1, ms1, u1, thr1) = res
    assert seed0 != seed1 and ctx0 != ctx1                    # every rank has its own batch
    assert ms0 == ms1 == 15.0                                 # the slowest rank sets the time
    assert u0 == u1 == 2 * W.CONFIGS["tiny"].batch            # the job's work is the sum
    assert thr0 == thr1 == pytest.approx(8 / 15e-3)


def test_single_process_is_identity():
    from paper_2609_29364_b200 import dist_util

    assert dist_util.combine(3.0, 7) == (3.0, 7.0)
    assert dist_util.rank_config(W.CONFIGS["tiny"], 0) is W.CONFIGS["tiny"]
