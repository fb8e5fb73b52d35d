"""Device-side plumbing shared by the tests, the smoke check and the benchmark.

Allocates the flat parameter / gradient buffers and the library's workspaces
with PyTorch, fills them from the seeded generators in ``workloads`` and drives
the C ABI through ``binding``.  No arithmetic of the method lives here.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import workloads as W


def partition_blocks(weights: Sequence[float], world: int) -> List[List[int]]:
    """Whole blocks to ranks, no block split: longest-processing-time greedy on the given per-block weights
    (bytes a step moves for the block, say).  Deterministic: ties go to the lower block index and the lower
    rank.  Statistics are per-block sums and every update rule is local to its block, so ranks that own whole
    blocks need no collective on the data path."""
    if world < 1:
        raise ValueError("world must be at least 1")
    order = sorted(range(len(weights)), key=lambda i: (-float(weights[i]), i))
    load = [0.0] * world
    parts: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        parts[r].append(i)
        load[r] += float(weights[i])
    for p in parts:
        p.sort()
    return parts


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's value (device-timed milliseconds), as every rank sees it."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist=None, device="cpu") -> float:
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


GUARD_BYTES = 4096
GUARD_BYTE = 0xC5


def guarded_alloc(n_bytes: int, device, fill_zero: bool = False):
    """A buffer of n_bytes bytes with GUARD_BYTES guard bytes of a fixed pattern before and after it, for tests of memory
    safety where no memory checker can be run: returns (whole allocation, the usable view).  The view keeps the 256-byte
    alignment of the allocation."""
    whole = torch.empty(n_bytes + 2 * GUARD_BYTES, dtype=torch.uint8, device=device)
    whole[:GUARD_BYTES] = GUARD_BYTE
    whole[GUARD_BYTES + n_bytes:] = GUARD_BYTE
    view = whole[GUARD_BYTES:GUARD_BYTES + n_bytes]
    if fill_zero:
        view.zero_()
    return whole, view


def guards_intact(whole: torch.Tensor) -> bool:
    """True while nothing has written into the guard bytes around a buffer from ``guarded_alloc``."""
    n = whole.numel() - 2 * GUARD_BYTES
    return bool((whole[:GUARD_BYTES] == GUARD_BYTE).all().item() and (whole[GUARD_BYTES + n:] == GUARD_BYTE).all().item())


def all_gather_params(local: torch.Tensor, out: torch.Tensor, dist) -> None:
    """The one exchange of a whole-block sharded step when replicas hold full weights: every rank contributes its flat
    parameter buffer ``local`` (all ranks' buffers have the same length, the longest shard's) and receives all of them
    in ``out`` (world x that length; rank r's block that starts at offset o of its buffer lies at r * len(local) + o).
    Queued behind the step on the current stream; NCCL on GPUs, gloo in the CPU tests."""
    if out.numel() != local.numel() * dist.get_world_size():
        raise ValueError("out must hold one buffer of local's length per rank")
    try:
        dist.all_gather_into_tensor(out, local)
    except (RuntimeError, NotImplementedError):               # a backend without the flat form
        dist.all_gather(list(out.view(dist.get_world_size(), -1).unbind(0)), local)


LIVE_SESSIONS = None        # a weakref.WeakSet, created on first use: the sessions whose guards a test fixture verifies


class Session:
    """One workload resident on one GPU.

    params: one flat fp32 buffer, block i at ``offs[i]`` (128-element aligned).
    grads:  ``n_grad_sets`` flat bf16 buffers with the same offsets; set k holds
    the gradients of step t for t % n_grad_sets == k once ``fill_grads(t)`` ran.
    """

    def __init__(self, wl: W.Workload, configs: Optional[Sequence[B.Config]] = None, opts: Optional[B.Opts] = None,
                 n_grad_sets: int = 2, device: str = "cuda:0", pinned_host_grads: bool = False, samples=None,
                 param_capacity: int = 0, factored_group_bytes: int = 0, param_skew_elems: int = 0):
        global LIVE_SESSIONS
        if LIVE_SESSIONS is None:
            import weakref
            LIVE_SESSIONS = weakref.WeakSet()
        LIVE_SESSIONS.add(self)
        self.wl = wl
        self.device = torch.device(device)
        self.configs = list(configs) if configs is not None else B.default_configs()
        self.h = B.Baoc(wl.blocks, self.configs, opts)
        self.offs, self.total = W.flat_layout(wl, 128)
        self.n_grad_sets = n_grad_sets
        # param_capacity: allocate the parameter buffer at least this long (the longest shard's length, so that the
        # buffers of all ranks can be all-gathered as they are)
        # every device buffer sits between guard bytes (``verify_guards``)
        self._guarded = []

        def alloc(n_bytes, zero=False):
            whole, view = guarded_alloc(n_bytes, self.device, zero)
            self._guarded.append(whole)
            return view

        self._alloc = alloc
        # param_skew_elems: start the parameter buffer this many elements into its allocation (4: every block pointer is
        # then 16-byte but not 32-byte aligned, the least the interface accepts)
        self.params = alloc(4 * (max(self.total, int(param_capacity)) + int(param_skew_elems)), True).view(torch.float32)[int(param_skew_elems):]
        self.grads = [alloc(2 * self.total, True).view(torch.bfloat16) for _ in range(n_grad_sets)]
        self.param_views = [self.params[o:o + b.numel] for o, b in zip(self.offs, wl.blocks)]
        self.grad_views = [[g[o:o + b.numel] for o, b in zip(self.offs, wl.blocks)] for g in self.grads]
        self.param_table = B.pointer_table(self.param_views)
        self.grad_tables = [B.pointer_table(v) for v in self.grad_views]
        self.host_grads = None
        if pinned_host_grads:
            self.host_grads = [torch.zeros(self.total, dtype=torch.bfloat16).pin_memory() for _ in range(n_grad_sets)]
            self.host_tables = [B.pointer_table([hg[o:o + b.numel] for o, b in zip(self.offs, wl.blocks)])
                                for hg in self.host_grads]
        if factored_group_bytes:
            self.h.set_factored_schedule(factored_group_bytes)
        self.samples = samples
        if samples is not None:
            self.h.set_sampling(samples)
        self.ws = alloc(self.h.stats_workspace_bytes())
        self.h.bind_stats_workspace(self.ws)
        self.state = None
        self.assign = None
        self._fixed_cache = {}

    def verify_guards(self) -> bool:
        """True while no kernel (or copy) has written outside any of this session's device buffers."""
        torch.cuda.synchronize(self.device)
        return all(guards_intact(w) for w in self._guarded)

    # ---- inputs -------------------------------------------------------------
    def init_params(self):
        for i, v in enumerate(self.param_views):
            v.copy_(W.block_param(self.wl, i, device=self.device))

    def fill_grads(self, t: int, blocks: Optional[Sequence[int]] = None, cache_fixed: bool = False):
        """Generate the gradients of step t (1-based) into set t % n_grad_sets."""
        k = t % self.n_grad_sets
        for i in (range(len(self.wl.blocks)) if blocks is None else blocks):
            fixed = None
            if cache_fixed:
                if i not in self._fixed_cache:
                    self._fixed_cache[i] = W.block_fixed_parts(self.wl, i, self.device)
                fixed = self._fixed_cache[i]
            W.block_grad(self.wl, i, t, device=self.device, fixed=fixed, out=self.grad_views[k][i])
        return k

    def host_copy_of_grads(self, k: int):
        if self.host_grads is not None:
            self.host_grads[k].copy_(self.grads[k])

    # ---- the path -------------------------------------------------------------
    def sample_stats(self, k: int):
        self.h.sample_stats(self.grad_tables[k])

    def risk(self):
        return self.h.risk(self.param_table)

    def allocate(self, risk, time_ratio=None, forbid=None, pref=None):
        mem, ratio = self.h.cost_model()
        if time_ratio is not None:
            ratio = np.asarray(time_ratio, np.float64)
        b_mem = int(np.floor(self.wl.mem_budget_frac * 8.0 * self.wl.numel))
        return self.h.allocate(risk, mem, ratio, b_mem, self.wl.time_budget, forbid, pref)

    def configure(self, assign):
        self.assign = np.asarray(assign, np.int32)
        self.state = self._alloc(self.h.state_bytes(self.assign))
        self.h.configure(self.assign, self.state)

    def configure_from_window(self, assign):
        """Instantiate the optimizer with the window's moments as its initial moments."""
        self.assign = np.asarray(assign, np.int32)
        self.state = self._alloc(self.h.state_bytes(self.assign))
        self.h.configure_from_window(self.assign, self.state)

    def reconfigure(self, assign, steps_done: int, inherit: bool = True):
        """Move to a new assignment in a fresh state buffer (the old one stays alive until the stream has passed)."""
        self.assign = np.asarray(assign, np.int32)
        new_state = self._alloc(self.h.state_bytes(self.assign))
        self.h.reconfigure(self.assign, new_state, steps_done, inherit)
        self.state = new_state

    def step(self, k: int, t: int):
        self.h.step(self.grad_tables[k], self.param_table, t)

    def step_from_host(self, k: int, do_stats: bool, t: int):
        self.h.step_from_host(self.host_tables[k], self.grad_tables[k], self.param_table, do_stats, t)

    # ---- read-back for checks ---------------------------------------------------
    def block_grad_host(self, k: int, i: int) -> np.ndarray:
        return self.grad_views[k][i].double().cpu().numpy()

    def block_param_host(self, i: int) -> np.ndarray:
        return self.param_views[i].double().cpu().numpy()

    def sampled(self, i: int, full: np.ndarray) -> np.ndarray:
        """The entries of block i's flat array that the statistics see (all of them without sampling)."""
        if self.samples is None:
            return full
        rows, cols = self.samples[i]
        b = self.wl.blocks[i]
        return full[rows] if cols is None else full.reshape(b.rows, b.cols)[np.ix_(rows, cols)].reshape(-1)
