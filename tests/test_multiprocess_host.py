"""Host-side logic of the N > 1 path with two gloo ranks on CPU: disjoint replica groups, the
max-over-ranks reduction of step times that bench.py reports, and the exchange step of the
outer sync (Algorithm 1, the count-normalised average): every rank ends up with every owner's end values."""
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


def _exchange_worker(rank, world, port, sizes, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    K = len(sizes)
    mine = pd.my_replicas(K, world, rank)
    # the owner holds the end values (a function of the replica id), everyone else stale numbers
    vals = [torch.full((n,), -1.0 - rank) for n in sizes]
    for k in mine:
        vals[k] = torch.arange(sizes[k], dtype=torch.float32) * 0.5 + 1000.0 * k
    received = pd.exchange_replica_values(vals, world, rank)
    ok = all(torch.equal(vals[k], torch.arange(sizes[k], dtype=torch.float32) * 0.5 + 1000.0 * k) for k in range(K))
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, ok, received))
    if rank == 0:
        out.put(gathered)
    dist.destroy_process_group()


def _run_exchange(sizes):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_exchange_worker, args=(r, 2, port, sizes, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    return res


def test_exchange_step_two_ranks_equal_and_ragged_replicas():
    # six equal replicas: three all-gather rounds; every rank receives exactly the other's three
    (m0, ok0, r0), (m1, ok1, r1) = _run_exchange([4096] * 6)
    assert m0 == [0, 2, 4] and m1 == [1, 3, 5] and ok0 and ok1
    assert r0 == r1 == 3 * 4096 * 4
    # ragged sizes, an odd replica count and an empty replica: broadcasts
    sizes = [1000, 24, 0, 512, 77]
    (m0, ok0, r0), (m1, ok1, r1) = _run_exchange(sizes)
    assert m0 == [0, 2, 4] and m1 == [1, 3] and ok0 and ok1
    assert r0 == (24 + 512) * 4 and r1 == (1000 + 0 + 77) * 4


def test_exchange_plan_covers_every_replica_once():
    for sizes, world in (([8] * 8, 4), ([8, 8, 8, 4, 8, 8], 3), ([5], 2), ([0, 3, 3, 3], 2), ([7] * 5, 8)):
        seen = []
        for kind, item in pd.exchange_plan(sizes, world):
            seen.extend(item if kind == "all_gather" else [item])
            if kind == "all_gather":
                assert len(item) == world and [pd.owner_rank(k, world) for k in item] == list(range(world))
        assert sorted(seen) == [k for k in range(len(sizes)) if sizes[k] > 0]
    assert pd.my_replicas(7, 3, 1) == [1, 4] and pd.owner_rank(5, 4) == 1
