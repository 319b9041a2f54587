"""Multi-GPU use of the selection path: layers are independent (Algorithm 1's outer loop), so a model is
split by layers across ranks and the per-layer records are gathered on the host.  No tensor data moves
between GPUs; the only communication is the gather of a few dozen bytes per layer (and the barrier /
max-over-ranks of a timing).  Works with any torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
import torch
import torch.distributed as dist


def partition_layers(costs, world):
    """Split layer indices into `world` lists with balanced total cost (bytes or flops).

    Deterministic longest-processing-time greedy: layers sorted by (-cost, index) go to the currently
    lightest rank (ties to the lowest rank); each rank's list is returned in ascending layer order.
    """
    if world < 1:
        raise ValueError("world must be >= 1")
    load = [0] * world
    parts = [[] for _ in range(world)]
    for i in sorted(range(len(costs)), key=lambda k: (-costs[k], k)):
        r = min(range(world), key=lambda k: (load[k], k))
        parts[r].append(i)
        load[r] += costs[i]
    return [sorted(p) for p in parts]


def layer_costs(shapes, metric="tensor", tokens=0):
    """Per-layer balancing cost for [(name, out_features, in_features)]: bytes of W under the tensor criterion (the
    scoring kernels are bound by the read of W), multiply-adds of the layer under the layer-output criterion."""
    if metric == "layer_output":
        return [o * i * max(1, tokens) for _, o, i in shapes]
    return [2 * o * i for _, o, i in shapes]


def select_formats_sharded(costs, score_fn, group=None):
    """Score this rank's share of the layers and return the records of ALL layers, in layer order, on every rank.

    costs     per-layer cost used for balancing (e.g. bytes of W for the tensor metric, flops for the layer metric)
    score_fn  callable(list_of_layer_indices) -> list of records (one per index, any picklable object); on a GPU
              rank it builds/loads those layers and calls mofq.select_formats on them
    """
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    parts = partition_layers(costs, world)
    mine = score_fn(parts[rank])
    if len(mine) != len(parts[rank]):
        raise ValueError("score_fn must return one record per layer index")
    if world == 1:
        gathered = [list(zip(parts[0], mine))]
    else:
        gathered = [None] * world
        dist.all_gather_object(gathered, list(zip(parts[rank], mine)), group=group)
    out = [None] * len(costs)
    for chunk in gathered:
        for idx, rec in chunk:
            out[idx] = rec
    return out


def max_over_ranks(value, device="cpu", group=None):
    """Largest `value` over all ranks (a device-side timing is reported as the slowest rank's)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
