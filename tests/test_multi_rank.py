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


def _oracle_two_steps(wl, ids):
    """Statistics pass + optimizer step of the oracle on the given blocks of the toy workload (the oracle stands in for
    the device work), two steps; returns {block: (fp32 parameters, rho_bar)}."""
    from oracle import baoc_oracle as O
    o = O.Opts()
    cfgs = O.default_configs()
    out = {}
    for i in ids:
        b = wl.blocks[i]
        c = cfgs[i % 5 if not (i % 5 == 3 and b.cols <= 1) else 2]
        th = W.block_param(wl, i).double().numpy()
        ss, st = O.stats_init(b.numel), O.step_init(c, b.numel, b.rows, b.cols)
        for t in (1, 2):
            g = W.block_grad(wl, i, t).double().numpy()
            O.stats_step(ss, g, o)
            th = O.step(th, g, st, c, b.rows, b.cols)
        out[i] = (th.astype(np.float32), ss.rho_bar)
    return out


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2605_04711_b200 import harness
        wl = W.make_workload("toy", seed=0)
        parts = harness.partition_blocks([26.0 * b.numel for b in wl.blocks], world)
        mine = parts[rank]
        # this rank's shard, laid out as the harness lays a session out: a flat buffer at the longest shard's length
        shard = W.Workload("shard", [wl.blocks[i] for i in mine], window=wl.window, mem_budget_frac=wl.mem_budget_frac,
                           time_budget=wl.time_budget, seed=wl.seed)
        offs, total = W.flat_layout(shard, 128)
        cap = int(harness.max_over_ranks(total, dist))
        local = torch.zeros(cap, dtype=torch.float32)
        res = _oracle_two_steps(wl, mine)                           # no collective: whole blocks are local work
        for o, i in zip(offs, mine):
            local[o:o + wl.blocks[i].numel] = torch.from_numpy(res[i][0])
        gathered = torch.empty(world * cap, dtype=torch.float32)
        harness.all_gather_params(local, gathered, dist)           # the one exchange of the sharded step
        layouts = [None] * world
        dist.all_gather_object(layouts, (mine, offs))
        rho = [None] * world
        dist.all_gather_object(rho, {i: res[i][1] for i in mine})
        if rank == 0:
            out.put((gathered.numpy(), cap, layouts, rho))
    finally:
        dist.destroy_process_group()


def test_a_sharded_run_reproduces_the_unsharded_one_block_by_block():
    """Two ranks that each own whole blocks, followed by the all-gather of the updated parameters, leave every rank
    with exactly the parameters (and per-block statistics) one rank computes alone."""
    _build.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, cap, layouts, rho = out.get(timeout=300)      # before the join: a rank blocks in put() until a large result is taken
    for p in procs:
        p.join(timeout=300)
        assert p.exitcode == 0
    wl = W.make_workload("toy", seed=0)
    alone = _oracle_two_steps(wl, range(len(wl.blocks)))
    seen = set()
    for r, (mine, offs) in enumerate(layouts):
        for o, i in zip(offs, mine):
            got = gathered[r * cap + o: r * cap + o + wl.blocks[i].numel]
            np.testing.assert_array_equal(got, alone[i][0])
            assert rho[r][i] == alone[i][1]
            seen.add(i)
    assert seen == set(range(len(wl.blocks)))


def test_partition_is_deterministic_and_handles_edge_cases():
    from paper_2605_04711_b200 import harness
    w = [5.0, 5.0, 3.0, 3.0, 1.0]
    assert harness.partition_blocks(w, 1) == [[0, 1, 2, 3, 4]]
    assert harness.partition_blocks(w, 2) == harness.partition_blocks(w, 2) == [[0, 2, 4], [1, 3]]
    parts = harness.partition_blocks(w, 8)                                  # more ranks than blocks: some ranks idle
    assert sorted(i for p in parts for i in p) == [0, 1, 2, 3, 4] and sum(1 for p in parts if not p) == 3
    assert harness.partition_blocks([], 3) == [[], [], []]
