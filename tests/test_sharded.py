"""The N>1 path on CPU: two gloo ranks split a layer list, score their shares with a stand-in scorer and
gather the records; the timing reduction takes the slowest rank."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2305_12356_b200 import inputs
from paper_2305_12356_b200.sharded import max_over_ranks, partition_layers, select_formats_sharded


def test_partition_is_balanced_and_complete():
    shapes = inputs.workload_layers("llama7b_w4_group128", blocks=4)
    costs = [o * i * 2 for _, o, i in shapes]
    for world in (1, 2, 3, 8):
        parts = partition_layers(costs, world)
        assert sorted(i for p in parts for i in p) == list(range(len(costs)))
        loads = [sum(costs[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(costs)
        assert parts == partition_layers(costs, world)                # deterministic
    assert partition_layers([], 2) == [[], []]
    with pytest.raises(ValueError):
        partition_layers(costs, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, costs, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seen = []

        def score(indices):                                           # stand-in for mofq.select_formats on this rank's layers
            seen.extend(indices)
            return [dict(layer=i, chosen=i % 2, rank=rank) for i in indices]

        recs = select_formats_sharded(costs, score)
        slowest = max_over_ranks(10.0 + rank)
        torch.save(dict(recs=recs, seen=seen, slowest=slowest), os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_gather_all_records(tmp_path):
    shapes = inputs.workload_layers("llama13b_w8a8_layer", blocks=2)
    costs = [o * i for _, o, i in shapes]
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, costs, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(tmp_path / f"r{r}.pt") for r in range(world)]
    parts = partition_layers(costs, world)
    for r, o in enumerate(outs):
        assert o["seen"] == parts[r]                                   # each rank scored only its share
        assert [rec["layer"] for rec in o["recs"]] == list(range(len(costs)))
        assert [rec["chosen"] for rec in o["recs"]] == [i % 2 for i in range(len(costs))]
        assert o["slowest"] == 11.0
    assert outs[0]["recs"] == outs[1]["recs"]
    assert {rec["rank"] for rec in outs[0]["recs"]} == {0, 1}
