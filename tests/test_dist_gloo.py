"""The multi-process path of the benchmark on CPU: two gloo ranks, rendezvous on 127.0.0.1."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2508_15212_b200 import dist_utils
from workloads import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    assert dist_utils.env_ranks() == (rank, world, rank)
    dist = dist_utils.init_process_group("gloo")
    assert dist is not None and dist.get_world_size() == world
    dist.barrier()
    slow = dist_utils.max_over_ranks(10.0 + 5.0 * rank, dist)            # rank 1 is the slow one
    # every rank draws its own data: same shapes, different bytes, no exchange
    wl = inputs.make_workload(batch=1, n_q_heads=4, n_kv_heads=1, seq_lens=64, window=4, dtype="bf16",
                              seed=7 + 1000003 * dist_utils.rank_seed_offset(rank))
    digest = int(wl.k.view(torch.int16).to(torch.int64).sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, digest)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, slow, gathered))


def test_two_gloo_ranks_time_is_max_and_data_is_per_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert res[0][2] == res[1][2] and res[0][2][0] != res[0][2][1]
    assert dist_utils.aggregate_throughput(100.0, 2, 0.5) == 400.0
    assert dist_utils.max_over_ranks(3.5, None) == 3.5 and dist_utils.rank_seed_offset(2, 3) == 131
