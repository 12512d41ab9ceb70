"""Several GPUs as the paper's parameter servers, one process per GPU.

Section 1.1: the parameters are split over servers; server j holds theta[j], every worker sends it the part
G[j] of its gradient (Algorithm 3) and reads theta[j] back; Algorithm 4 runs on every server.  Here GPU j is
server j for one contiguous range of columns AND the machine that some of the workers run on: their
gradients are whole rows in its memory, and it keeps a full copy of theta for them to read.

One iteration on GPU j is ONE launch of the library's row-streaming kernel (`sgdb_step_rows`): it takes the
selection in its prologue (every server computes the same one from the same W numbers), pulls its columns of
the kept rows from whichever GPU holds them with bulk copies over NVLink (never multicast), applies the
optimizer rule to its range and stores the new parameters into every GPU's copy.  There is no separate
reduce-scatter or all-gather and no kernel waits for another GPU; the two points of the synchronous protocol
where GPUs must agree (all gradients written before any server reads; all copies written before any worker
reads) are fences between launches, enqueued on the stream.

This module is plumbing only: which columns and workers belong to whom, the exchange of buffer addresses
between processes, and the fences.  Every arithmetic step runs in the CUDA library.
"""
from __future__ import annotations

import pickle
from dataclasses import dataclass
from multiprocessing.reduction import ForkingPickler

import torch
import torch.distributed as dist
import torch.multiprocessing  # noqa: F401  (registers how tensors are passed between processes)


@dataclass(frozen=True)
class Plan:
    """Who holds what: column ranges per server, workers per machine.  Pure host arithmetic."""

    P: int
    W: int
    G: int
    ranges: tuple  # ((first column, columns), ...) per server, from sgdb_shard_range

    @property
    def workers_per_machine(self) -> int:
        return -(-self.W // self.G)

    def machine_of(self, w: int) -> int:
        """The GPU whose memory holds worker w's gradient: neighbours share a machine."""
        return w // self.workers_per_machine

    def local_index(self, w: int) -> int:
        return w % self.workers_per_machine

    def workers_of(self, g: int) -> range:
        k = self.workers_per_machine
        return range(min(self.W, g * k), min(self.W, (g + 1) * k))

    def groups(self):
        """Machine id of every worker (the d_group array of the two-level calls)."""
        return [self.machine_of(w) for w in range(self.W)]


def make_plan(P: int, W: int, G: int, shard_range=None) -> Plan:
    if shard_range is None:
        from .binding import sgdb_shard_range as shard_range
    if P < 0 or W < 1 or G < 1:
        raise ValueError("need P >= 0, W >= 1, G >= 1")
    return Plan(P, W, G, tuple(tuple(shard_range(P, G, j)) for j in range(G)))


def row_addresses(plan: Plan, j: int, grad_bases, row_pitch_bytes: int, elem_bytes: int):
    """Address, as seen from this process, of column first_j of every worker's gradient.
    grad_bases[g] = address of machine g's gradient buffer ([its workers x row pitch]) mapped into this process."""
    first = plan.ranges[j][0]
    return [grad_bases[plan.machine_of(w)] + plan.local_index(w) * row_pitch_bytes + first * elem_bytes
            for w in range(plan.W)]


def replica_addresses(plan: Plan, j: int, theta_bases):
    """Address of column first_j in every OTHER GPU's copy of theta (server j's own copy is its d_theta)."""
    first = plan.ranges[j][0]
    return [theta_bases[g] + first * 4 for g in range(plan.G) if g != j]


def share_with_peers(tensor: torch.Tensor, group=None):
    """Every process passes its tensor; returns one tensor per rank, each an alias of that rank's memory
    (this rank's entry is `tensor` itself).  Device memory travels as a CUDA IPC handle, host memory as a
    shared-memory file; the owner must keep its tensor alive while the peers use theirs."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    if world == 1:
        return [tensor]
    payload = bytes(ForkingPickler.dumps(tensor))
    gathered = [None] * world
    dist.all_gather_object(gathered, payload, group=group)
    return [tensor if g == rank else pickle.loads(gathered[g]) for g in range(world)]


def fence(group=None, flag: torch.Tensor | None = None) -> None:
    """Everything enqueued before the fence on any rank's current stream is complete, on every rank, before
    anything enqueued after it starts.  With NCCL this is a one-word all-reduce on the stream (no host wait);
    with another backend the host waits for its stream and meets the others at a barrier."""
    if dist.get_world_size(group) == 1:
        return  # the stream's own order is all there is to keep
    backend = dist.get_backend(group)
    if backend == "nccl":
        dist.all_reduce(flag, group=group)
        return
    if torch.cuda.is_available() and torch.cuda.is_initialized():
        torch.cuda.current_stream().synchronize()
    dist.barrier(group=group)


class ServerGroup:
    """This process's member of a group of G parameter servers (rank j = server j = machine j).

    Buffers, all on `device`:
      grads  [workers of this machine, ld]  rows the local workers write before `step` (dtype f32 or bf16)
      theta  [P] fp32                       this GPU's full copy; columns of range j are the master copy
      state0, state1 [columns of range j]   optimizer state of range j (as the rule needs)
    `step` and `step_two_level` take the arrival times and tags of ALL W workers as tensors on `device`,
    identical on every rank.
    """

    def __init__(self, P: int, W: int, N: int, b: int, grad_dtype: torch.dtype, opt_kw: dict, device, group=None,
                 launch=None, two_level_launch=None):
        from . import binding  # fails loudly when the CUDA library is not built: there is no fallback

        self.sgdb = binding
        self.group = group
        self.rank = dist.get_rank(group)
        G = dist.get_world_size(group)
        if N + b != W:
            raise ValueError("W must equal N + b")
        self.N, self.b, self.device, self.opt_kw = N, b, torch.device(device), dict(opt_kw)
        self.grad_dtype = grad_dtype
        self.plan = make_plan(P, W, G, binding.sgdb_shard_range)
        es = 2 if grad_dtype == torch.bfloat16 else 4
        self.ld = -(-P // 8) * 8  # rows start on 16-byte boundaries for both element types
        n_local = len(self.plan.workers_of(self.rank))
        self.grads = torch.zeros((max(n_local, 1), max(self.ld, 8)), dtype=grad_dtype, device=self.device)
        self.theta = torch.zeros(max(P, 1), dtype=torch.float32, device=self.device)
        self.first, self.len = self.plan.ranges[self.rank]
        n_state = {"sgd": 0, "momentum": 1, "rmsprop": 2, "adam": 2, "adagrad": 1}[opt_kw["kind"]]
        self.state0 = torch.zeros(max(self.len, 1), dtype=torch.float32, device=self.device) if n_state >= 1 else None
        self.state1 = torch.zeros(max(self.len, 1), dtype=torch.float32, device=self.device) if n_state >= 2 else None
        self.message = torch.zeros(max(self.ld, 8), dtype=torch.float32, device=self.device)  # two-level: this machine's mean
        self.mask = torch.zeros(W, dtype=torch.uint8, device=self.device)
        self.order = torch.zeros(W, dtype=torch.int32, device=self.device)
        self.group_order = torch.zeros(G, dtype=torch.int32, device=self.device)
        self.info = torch.zeros(3, dtype=torch.int32, device=self.device)
        self.local_info = torch.zeros(2, dtype=torch.int32, device=self.device)
        self.local_mask = torch.zeros(max(n_local, 1), dtype=torch.uint8, device=self.device)
        self.local_order = torch.zeros(max(n_local, 1), dtype=torch.int32, device=self.device)
        self.groups = torch.tensor(self.plan.groups(), dtype=torch.int32, device=self.device)
        self._flag = torch.zeros(1, dtype=torch.int32, device=self.device)

        # the peers' buffers, mapped into this process (kept alive here for as long as the tables are used)
        self._peer_grads = share_with_peers(self.grads, group)
        self._peer_theta = share_with_peers(self.theta, group)
        self._peer_message = share_with_peers(self.message, group)
        if self.device.type == "cuda":
            # kernels on this GPU will read the peers' rows and write the peers' copies of theta
            with torch.cuda.device(self.device):
                for x in self._peer_grads:
                    if x.device != self.grads.device:
                        binding.sgdb_enable_peer_access(x.device.index)
        pitch = self.grads.stride(0) * es
        self.row_addr = row_addresses(self.plan, self.rank, [x.data_ptr() for x in self._peer_grads], pitch, es)
        self.replica_addr = replica_addresses(self.plan, self.rank, [x.data_ptr() for x in self._peer_theta])
        self.message_addr = [x.data_ptr() + self.first * 4 for x in self._peer_message]
        if self.device.type == "cuda":
            self.rows_table = binding.make_address_table(self.row_addr, self.device)
            self.replica_table = binding.make_address_table(self.replica_addr, self.device) if self.replica_addr else None
            self.message_table = binding.make_address_table(self.message_addr, self.device)
        self._launch = launch if launch is not None else ServerGroup._launch_step_rows
        self._launch_two_level = two_level_launch if two_level_launch is not None else ServerGroup._launch_two_level_rows
        fence(group, self._flag)

    def my_theta(self) -> torch.Tensor:
        """The master copy of this server's range (a view into this GPU's copy of theta)."""
        return self.theta[self.first:self.first + self.len] if self.len else self.theta[:1]

    def _opt(self, update: int):
        return self.sgdb.Opt(step=update, **self.opt_kw)

    def _launch_step_rows(self, t: int, arrival, tags, update: int) -> None:
        self.sgdb.sgdb_step_rows(self.rows_table, self.grad_dtype, self.len, arrival, tags, t, self.N, self.b,
                                 self.my_theta(), self.state0, self.state1, self._opt(update), self.replica_table,
                                 self.mask, self.order[:self.N], self.info[:2])

    def step(self, t: int, arrival, tags, update: int = 1) -> None:
        """Iteration t on this server: fence, one launch, fence.  Afterwards every GPU's `theta` holds the new
        parameters of every range and `info[:2]` = {current gradients, status}.  `update` is the 1-based count of
        updates including this one (sgdb_opt_t's `step`; it matters to Adam only)."""
        fence(self.group, self._flag)  # every worker's gradient is in place
        self._launch(self, t, arrival, tags, update)
        fence(self.group, self._flag)  # every copy of theta is complete

    def _launch_two_level_rows(self, t: int, arrival, tags, n_machines: int, update: int) -> None:
        sgdb = self.sgdb
        sgdb.sgdb_select_grouped(arrival, tags, self.groups, t, self.plan.G, n_machines, self.mask, self.group_order[:n_machines],
                                 self.order, self.info)
        sgdb.sgdb_step_rows_ordered(self.message_table, torch.float32, self.len, n_machines, self.group_order[:n_machines],
                                    self.info, self.my_theta(), self.state0, self.state1, self._opt(update), self.replica_table)

    def step_two_level(self, t: int, arrival, tags, n_machines: int, update: int = 1) -> None:
        """Iteration t with the gradients of each machine's workers combined before they leave the machine
        (Section 6): every machine writes the mean of its workers' rows if all of them are current, then the
        servers take the first n_machines messages as rows.  One row per machine crosses instead of one per worker."""
        sgdb = self.sgdb
        mine = self.plan.workers_of(self.rank)
        fence(self.group, self._flag)
        if len(mine) and self.plan.P:
            a, g = arrival[mine.start:mine.stop], tags[mine.start:mine.stop]
            sgdb.sgdb_select(a, g, t, len(mine), 0, self.local_mask, self.local_order, self.local_info)
            sgdb.sgdb_aggregate(self.grads, self.plan.P, len(mine), self.local_order, self.local_info, self.message[:self.plan.P],
                                ld=self.grads.stride(0))
        fence(self.group, self._flag)  # every machine's message is in place
        self._launch_two_level(self, t, arrival, tags, n_machines, update)
        fence(self.group, self._flag)
