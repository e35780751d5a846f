"""Multi-GPU plumbing: one process per GPU.

Between outer syncs the replicas of Algorithm 1 never exchange data, so G GPUs run G disjoint
sets of replicas with no data-path collective.  Every H steps the paper all-reduces the sparse
deltas and divides by the count vector m (Algorithm 1, the count-normalised average, Eq. 2.4).  Here that exchange
step is an all-gather of the replicas' end values: replica k lives on GPU k mod G, every GPU
holds a buffer for every replica's packed trained values (ppu_replica_values), the owners'
values are gathered into those buffers, and every GPU then runs the same ppu_outer_sync over
all K replicas - the sum over owners, the division by m and the Nesterov step happen in that
one kernel, in the same order on every GPU, so all GPUs end with bit-identical parameters, equal
to what one GPU simulating all K replicas computes.  For disjoint slices this moves exactly the
trained values once (what an all-reduce of sparse deltas would move); where owners overlap
(m > 1) it moves each owner's copy, and no separate reduce-scatter is needed.

The collectives run on local buffers only (NCCL on GPUs, gloo in the CPU tests): no kernel of
this library reads another GPU's memory.
"""
from __future__ import annotations


def replica_group(n_replicas_per_rank: int, world: int, rank: int):
    """Global ids of the replicas rank `rank` simulates when every rank runs its own independent
    block of replicas (the benchmark's replicas-only mode)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    lo = rank * n_replicas_per_rank
    return list(range(lo, lo + n_replicas_per_rank))


def owner_rank(replica: int, world: int) -> int:
    """Replica k is stepped by GPU k mod G."""
    return replica % world


def my_replicas(n_replicas: int, world: int, rank: int):
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    return [k for k in range(n_replicas) if owner_rank(k, world) == rank]


def exchange_plan(sizes, world: int):
    """How the exchange is issued.  sizes[k] = number of packed values of replica k.  Replicas
    j*G .. j*G + G - 1 form round j, one replica per rank; a complete round whose buffers are all
    the same size goes as one all-gather, anything else as one broadcast per replica.
    Returns a list of ("all_gather", [k ...]) / ("broadcast", k) items; every replica appears
    exactly once."""
    K = len(sizes)
    plan = []
    for j in range(0, K, world):
        ks = list(range(j, min(j + world, K)))
        if len(ks) == world and len({sizes[k] for k in ks}) == 1 and sizes[ks[0]] > 0:
            plan.append(("all_gather", ks))
        else:
            plan.extend(("broadcast", k) for k in ks if sizes[k] > 0)
    return plan


def exchange_replica_values(values, world: int, rank: int, group=None):
    """values[k]: this rank's 1-D buffer for replica k's packed trained values (a view into the
    context's arena on a GPU; any tensor in the CPU tests).  On return every buffer holds its
    owner's values.  Returns the number of bytes this rank received."""
    import torch.distributed as dist
    if world == 1:
        return 0
    received = 0
    for kind, item in exchange_plan([int(v.numel()) for v in values], world):
        if kind == "all_gather":
            mine = values[item[rank]]
            dist.all_gather([values[k] for k in item], mine, group=group)
            received += sum(values[k].numel() * values[k].element_size() for k in item if k != item[rank])
        else:
            src = owner_rank(item, world)
            dist.broadcast(values[item], src=src, group=group)
            if src != rank:
                received += values[item].numel() * values[item].element_size()
    return received


def outer_sync_all_gpus(ctx, n_replicas: int, world: int, rank: int, group=None):
    """The exchange step followed by the outer step of Algorithm 1 on every GPU.
    ctx: this rank's ppu.Context holding all n_replicas replicas, of which it stepped
    my_replicas(n_replicas, world, rank).  Returns the bytes received."""
    ctx.ppu_sync()                       # the local steps that produced the values have finished
    vals = [ctx.ppu_replica_values(k) for k in range(n_replicas)]
    n = exchange_replica_values(vals, world, rank, group)
    ctx.ppu_outer_sync(list(range(n_replicas)))
    return n


def exchange_between_contexts(ctxs, n_replicas: int):
    """The same exchange between several contexts that live in ONE process (ranks emulated one
    after the other on one GPU, for tests): context r plays GPU r, the owners' values are copied
    into the other contexts' buffers with plain device copies."""
    world = len(ctxs)
    for k in range(n_replicas):
        src = ctxs[owner_rank(k, world)].ppu_replica_values(k)
        for r, c in enumerate(ctxs):
            if r != owner_rank(k, world):
                c.ppu_replica_values(k).copy_(src)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
