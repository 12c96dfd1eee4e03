"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_14107_b200 import inputs as I
from paper_2607_14107_b200 import replicas as R


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    m, p = I.config("c1")
    prompt = I.make_prompt(m, p, seed=R.replica_prompt_seed(1, rank))
    # rank r "measures" (10 + r) ms and decodes 64 * (r + 1) tokens
    times, counts = R.aggregate([10.0 + rank, 5.0 - rank], [64.0 * (rank + 1), 32.0])
    out[rank] = (times, counts, prompt[0, :8].tolist())
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_tokens():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        times, counts, _ = res[r]
        assert times == [11.0, 5.0]           # max over ranks
        assert counts == [192.0, 64.0]        # sum over ranks
    assert res[0][2] != res[1][2]             # replicas decode different prompts
    m, p = I.config("c1")
    assert res[1][2] == I.make_prompt(m, p, seed=2)[0, :8].tolist()
    assert R.whole_job_rate(192.0, 11.0) == 192.0 / 0.011


def test_single_process_is_identity():
    times, counts = R.aggregate([3.0], [7.0])
    assert times == [3.0] and counts == [7.0]
