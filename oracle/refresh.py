"""Oracle for the multi-worker exchanges around the step: the boundary cache refresh and the
synchronised gradient (Algorithm 2, dynamic cache synchronisation section).

TEST INFRASTRUCTURE: only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module.  It shares no code with the library.

All workers are simulated in one process with plain Python loops over numpy rows.

    boundary refresh   at an executed window boundary (S_r = 1) worker p fetches the state of every
                       node in N_sync[p] from the worker that owns it: afterwards p's copy of such a
                       node equals the owner's copy.  Nothing else changes on any worker.
    gradient           the model gradient a worker applies is the mean over workers of their local
                       gradients (data-parallel training); its norm is the controller's g_r, the same
                       number on every worker.

Readings where the paper is silent:
  * a node's "data state" is its memory row together with its last-update time (the pair the memory
    module keeps per node);
  * every worker reads the owners' states as they were BEFORE the refresh (one collective exchange, not
    a chain), which matters only if an owner could itself receive the node -- it cannot, a worker never
    requests a node it owns, and the plan asserts that;
  * "synchronised gradients" are averaged, as the data-parallel baseline of the evaluation does; a sum
    would only rescale g_r and the learning rate.
"""
from __future__ import annotations

from typing import List, Sequence, Set, Tuple

import numpy as np


def refresh_plan(n_sync: Sequence[Set[int]], owner: Sequence[int]) -> List[List[List[int]]]:
    """send[o][p] = the nodes worker o sends to worker p, in ascending id order.

    n_sync[p] is worker p's candidate refresh set for the window that starts at this boundary.
    """
    P = len(n_sync)
    send: List[List[List[int]]] = [[[] for _ in range(P)] for _ in range(P)]
    for p in range(P):
        for n in sorted(n_sync[p]):
            o = int(owner[n])
            if o == p:
                raise ValueError(f"worker {p} asks for node {n}, which it owns")
            send[o][p].append(int(n))
    return send


def boundary_refresh(memory: Sequence[np.ndarray], last_update: Sequence[np.ndarray], n_sync: Sequence[Set[int]],
                     owner: Sequence[int]) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Tables of all workers after an executed refresh (inputs are not modified)."""
    P = len(n_sync)
    send = refresh_plan(n_sync, owner)
    mem_new = [np.array(m, copy=True) for m in memory]
    lu_new = [np.array(t, copy=True) for t in last_update]
    for o in range(P):
        for p in range(P):
            for n in send[o][p]:
                mem_new[p][n, :] = memory[o][n, :]      # the owner's state before the exchange
                lu_new[p][n] = last_update[o][n]
    return mem_new, lu_new


def synchronised_gradient(grads: Sequence[np.ndarray]) -> Tuple[np.ndarray, float]:
    """Mean of the workers' gradients (fp64) and its Euclidean norm g_r."""
    acc = np.zeros_like(np.asarray(grads[0], dtype=np.float64))
    for g in grads:
        acc = acc + np.asarray(g, dtype=np.float64)
    mean = acc / float(len(grads))
    return mean, float(np.sqrt(np.sum(mean * mean)))
