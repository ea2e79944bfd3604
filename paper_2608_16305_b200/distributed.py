"""Multi-worker plumbing around the step: the boundary cache refresh as one all-to-all of packed rows,
the coordinator's refresh flag, and the synchronised gradient (Algorithm 2, dynamic cache
synchronisation).  One process per GPU; `torch.distributed` carries the bytes (NCCL on GPUs), the
library's kernels do everything that touches the model state:

    offline   tgnn_backward_scan (N_sync flags)  ->  tgnn_refresh_plan (who sends what, per window)
    boundary  tgnn_pack_rows -> all_to_all_single -> tgnn_unpack_rows         (only when S_r = 1)
    step      step with the gradient left in the context's buffer -> all_reduce -> tgnn_apply_gradient

Received rows land in this GPU's own memory before any kernel reads them.  The row movers are
arguments so that the host logic (splits, routing, flag) can be exercised by CPU processes over gloo
with stand-ins; the defaults are the library's kernels and there is no other implementation here.
"""
from __future__ import annotations

from typing import Callable, List, Optional

import numpy as np
import torch
import torch.distributed as dist

from . import binding as B


class RefreshPlan:
    """Worker `me`'s receive and send lists for every window, computed on the device by
    tgnn_refresh_plan from the backward scan's N_sync flags; the per-peer counts are kept on the host
    because the collective wants its split sizes there."""

    def __init__(self, sync: torch.Tensor, owner: torch.Tensor, n_sync_host: np.ndarray, P: int, me: int):
        Q = int(n_sync_host.shape[1]) if n_sync_host.size else 0
        self.P, self.Q, self.me = P, Q, me
        self.cap = max(1, int(n_sync_host.sum(axis=0).max()) if Q else 1)
        dev = sync.device
        self.recv_nodes = torch.zeros((max(Q, 1), self.cap), dtype=torch.int32, device=dev)
        self.send_nodes = torch.zeros((max(Q, 1), self.cap), dtype=torch.int32, device=dev)
        recv_off = torch.zeros((max(Q, 1), P + 1), dtype=torch.int32, device=dev)
        send_off = torch.zeros((max(Q, 1), P + 1), dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.refresh_plan(sync, owner, P, Q, me, self.cap, self.recv_nodes, recv_off, self.send_nodes, send_off, status)
        st = int(status.item())
        if st:
            raise RuntimeError(f"refresh plan reported device status {st}")
        self.recv_off = recv_off.cpu().numpy().astype(np.int64)
        self.send_off = send_off.cpu().numpy().astype(np.int64)

    @classmethod
    def from_lists(cls, recv_nodes, recv_off, send_nodes, send_off, P: int, me: int) -> "RefreshPlan":
        """A plan from ready-made lists (tensors [Q, cap] and host offsets [Q, P + 1])."""
        self = cls.__new__(cls)
        self.P, self.me, self.Q, self.cap = P, me, int(recv_off.shape[0]), int(recv_nodes.shape[1])
        self.recv_nodes, self.send_nodes = recv_nodes, send_nodes
        self.recv_off, self.send_off = np.asarray(recv_off, np.int64), np.asarray(send_off, np.int64)
        return self

    def recv_counts(self, q: int) -> List[int]:
        return np.diff(self.recv_off[q]).tolist()

    def send_counts(self, q: int) -> List[int]:
        return np.diff(self.send_off[q]).tolist()


class BoundaryRefresh:
    """The refresh of one worker's remote-node states at a window boundary."""

    def __init__(self, plan: RefreshPlan, d: int, group=None, pack: Callable = B.pack_rows, unpack: Callable = B.unpack_rows):
        self.plan, self.d, self.group = plan, d, group
        self._pack, self._unpack = pack, unpack
        dev = plan.recv_nodes.device
        self.send_buf = torch.zeros(plan.cap * (d + 2), dtype=torch.float32, device=dev)
        self.recv_buf = torch.zeros(plan.cap * (d + 2), dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.rows_sent = self.rows_received = 0

    def pack(self, q: int, memory: torch.Tensor, last_update: torch.Tensor) -> int:
        """Phase 1: the rows this worker owes the others, grouped by requester, into send_buf."""
        ns = int(self.plan.send_off[q, -1])
        if ns:
            self._pack(memory, last_update, self.plan.send_nodes[q, :ns], self.send_buf, self.status)
        return ns

    def exchange(self, q: int) -> None:
        """Phase 2: one all-to-all; segment r of send_buf goes to worker r, segment o of recv_buf comes from o."""
        pl, w = self.plan, self.d + 2
        sc, rc = pl.send_counts(q), pl.recv_counts(q)
        if pl.P == 1 and sum(sc) == 0 and sum(rc) == 0:
            return                                      # a single worker owns every node: nothing to move
        dist.all_to_all_single(self.recv_buf[:sum(rc) * w], self.send_buf[:sum(sc) * w],
                               output_split_sizes=[c * w for c in rc], input_split_sizes=[c * w for c in sc],
                               group=self.group)

    def unpack(self, q: int, memory: torch.Tensor, last_update: torch.Tensor) -> int:
        """Phase 3: received rows replace this worker's copies of its N_sync nodes."""
        nr = int(self.plan.recv_off[q, -1])
        if nr:
            self._unpack(memory, last_update, self.plan.recv_nodes[q, :nr], self.recv_buf, self.status)
        return nr

    def run(self, q: int, memory: torch.Tensor, last_update: torch.Tensor) -> None:
        """Executes the refresh of window q (every worker of the group must call it)."""
        self.rows_sent += self.pack(q, memory, last_update)
        self.exchange(q)
        self.rows_received += self.unpack(q, memory, last_update)


def broadcast_decision(sync: int, device, group=None, coordinator: int = 0) -> int:
    """The coordinator's refresh decision S_r as a constant-size flag to all workers."""
    flag = torch.tensor([int(sync)], dtype=torch.int32, device=device)
    dist.broadcast(flag, src=coordinator, group=group)
    return int(flag.item())


def synchronise_gradient(lib: "B.Tgnn", gradnorm_out: Optional[torch.Tensor], group=None, grads: Optional[torch.Tensor] = None) -> None:
    """Sum of the workers' gradient buffers, then norm and Adam on their mean (in stream order)."""
    g = lib.grad_buffer() if grads is None else grads
    world = dist.get_world_size(group)
    if world > 1:
        dist.all_reduce(g, op=dist.ReduceOp.SUM, group=group)
    lib.apply_gradient(1.0 / world, gradnorm_out)
