"""Host-side logic of the N > 1 path with two gloo ranks on CPU: disjoint replica groups and the
max-over-ranks reduction of step times that bench.py reports."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_22418_b200 import dist as pd, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    group = pd.replica_group(4, world, rank)
    pd.barrier()
    times = pd.max_over_ranks([10.0 + rank, 5.0 - rank])
    tok = synth.tokens(1, group[0], 0, 0, 2, 8, 100)
    gathered = [None] * world
    dist.all_gather_object(gathered, (group, times, tok.tolist()))
    if rank == 0:
        out.put(gathered)
    dist.destroy_process_group()


def test_two_ranks_disjoint_replicas_and_max_times():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (g0, t0, k0), (g1, t1, k1) = res
    assert g0 == [0, 1, 2, 3] and g1 == [4, 5, 6, 7]
    assert t0 == t1 == [11.0, 5.0]
    assert k0 != k1                     # each rank draws its own batches


def test_single_process_is_identity():
    assert pd.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert pd.replica_group(2, 3, 2) == [4, 5]
