"""Host logic of the N > 1 path, on CPU with two gloo ranks: blocks are dealt to ranks whole (no collective on
the data path), each rank works on its own share, and the reported time is the slowest rank's."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_04711_b200 import build as _build
from paper_2605_04711_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2605_04711_b200 import harness
        from oracle import baoc_oracle as O
        wl = W.make_workload("resnet50", seed=0)
        weights = [26.0 * b.numel for b in wl.blocks]
        mine = harness.partition_blocks(weights, world)[rank]
        # every rank owns whole blocks and can run its share of the path alone: here the statistics step of
        # the oracle on its three smallest blocks, standing in for the device work
        o = O.Opts()
        for i in sorted(mine, key=lambda k: wl.blocks[k].numel)[:3]:
            st = O.stats_init(wl.blocks[i].numel)
            O.stats_step(st, W.block_grad(wl, i, 1).double().numpy(), o)
            O.stats_step(st, W.block_grad(wl, i, 2).double().numpy(), o)
            assert -1.0 <= st.rho_bar <= 1.0
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        my_ms = 3.0 + 2.0 * rank                                     # rank 1 is the slow one
        slowest = harness.max_over_ranks(my_ms, dist)
        total = harness.sum_over_ranks(sum(wl.blocks[i].numel for i in mine), dist)
        if rank == 0:
            out.put((gathered, slowest, total, wl.numel, weights))
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_whole_blocks_and_report_the_slowest_time():
    _build.build()
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=300)
        assert p.exitcode == 0
    parts, slowest, total, numel, weights = out.get()
    assert sorted(parts[0] + parts[1]) == list(range(len(weights)))       # disjoint and complete
    assert set(parts[0]).isdisjoint(parts[1])
    loads = [sum(weights[i] for i in p) for p in parts]
    assert abs(loads[0] - loads[1]) <= max(weights)                        # greedy balance: within one block
    assert slowest == 5.0 and total == numel


def test_partition_is_deterministic_and_handles_edge_cases():
    from paper_2605_04711_b200 import harness
    w = [5.0, 5.0, 3.0, 3.0, 1.0]
    assert harness.partition_blocks(w, 1) == [[0, 1, 2, 3, 4]]
    assert harness.partition_blocks(w, 2) == harness.partition_blocks(w, 2) == [[0, 2, 4], [1, 3]]
    parts = harness.partition_blocks(w, 8)                                  # more ranks than blocks: some ranks idle
    assert sorted(i for p in parts for i in p) == [0, 1, 2, 3, 4] and sum(1 for p in parts if not p) == 3
    assert harness.partition_blocks([], 3) == [[], [], []]
