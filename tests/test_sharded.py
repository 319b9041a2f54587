"""The N>1 path on CPU: two gloo ranks split one model's layer list by cost, each rank "scores" its share by parsing
its slice of a recorded buffer of selection records (the bytes a device would hold after mofq_select_formats), and the
records are gathered on every rank; the timing reduction takes the slowest rank."""
import ctypes as C
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2305_12356_b200 import binding as B
from paper_2305_12356_b200 import inputs
from paper_2305_12356_b200.sharded import layer_costs, max_over_ranks, partition_layers, select_formats_sharded


def test_partition_is_balanced_and_complete():
    shapes = inputs.workload_layers("llama7b_w4_group128", blocks=4)
    costs = layer_costs(shapes)
    assert costs[0] == 2 * 4096 * 4096
    for world in (1, 2, 3, 8):
        parts = partition_layers(costs, world)
        assert sorted(i for p in parts for i in p) == list(range(len(costs)))
        loads = [sum(costs[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(costs)
        assert parts == partition_layers(costs, world)                # deterministic
    assert partition_layers([], 2) == [[], []]
    with pytest.raises(ValueError):
        partition_layers(costs, 0)


def test_whole_models_split_evenly_by_cost():
    """The shares of a whole model differ by far less than one layer: the slowest rank bounds the sharded time."""
    for name in ("llama33b_w4_channel_and_group128", "llama65b_w8a8_layer"):
        wl = inputs.WORKLOADS[name]
        costs = layer_costs(inputs.workload_layers(name), wl["metric"], wl["tokens"])
        for world in (2, 4, 8):
            loads = [sum(costs[i] for i in p) for p in partition_layers(costs, world)]
            assert max(loads) / (sum(loads) / world) < 1.01, (name, world, loads)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _recorded_results(n_layers, n_sets, n_cand):
    """Bytes of n_layers * n_sets selection records, as a device buffer would hold them."""
    recs = (B.MofqResult * (n_layers * n_sets))()
    for k, r in enumerate(recs):
        r.chosen = (k * 7 + 3) % n_cand
        r.status = 0
        for c in range(n_cand):
            r.error[c] = 1e-5 * (1 + ((k * 13 + c * 5) % 17))
            r.nsr[c] = 0.0
        r.rel_margin = 0.25 + k
    return bytes(recs)


def _worker(rank, world, port, costs, n_sets, n_cand, blob, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seen = []
        rb = B.RESULT_BYTES

        def score(indices):        # what a GPU rank does after mofq.select_formats on its layers: parse its records
            seen.extend(indices)
            mine = b"".join(blob[i * n_sets * rb:(i + 1) * n_sets * rb] for i in indices)
            parsed = B._parse_results(mine, len(indices) * n_sets, n_cand)
            return [parsed[k * n_sets:(k + 1) * n_sets] for k in range(len(indices))]

        recs = select_formats_sharded(costs, score)
        slowest = max_over_ranks(10.0 + rank)
        torch.save(dict(recs=recs, seen=seen, slowest=slowest), os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_gather_the_records_of_one_model(tmp_path):
    name = "llama33b_w4_channel_and_group128"
    wl = inputs.WORKLOADS[name]
    shapes = inputs.workload_layers(name, blocks=2)
    costs = layer_costs(shapes, wl["metric"], wl["tokens"])
    n_sets, n_cand = len(wl["w_gran"]), len(wl["candidates"])
    blob = _recorded_results(len(shapes), n_sets, n_cand)
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, costs, n_sets, n_cand, blob, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(tmp_path / f"r{r}.pt") for r in range(world)]
    parts = partition_layers(costs, world)
    single = B._parse_results(blob, len(shapes) * n_sets, n_cand)               # what one rank scoring everything gets
    want = [single[k * n_sets:(k + 1) * n_sets] for k in range(len(shapes))]
    for r, o in enumerate(outs):
        assert o["seen"] == parts[r]                                   # each rank scored only its share
        assert o["recs"] == want                                       # and every rank holds the whole model's records
        assert o["slowest"] == 11.0
    assert C.sizeof(B.MofqResult) == B.RESULT_BYTES == 48
