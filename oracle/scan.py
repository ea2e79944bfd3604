"""Oracle for the source-based backward dependency scan and mixed-batch construction (Algorithm 1).

TEST INFRASTRUCTURE: only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module.  It shares no code with the library.

Pure Python sets and loops, in the algorithm's order and notation: for worker p
and synchronisation window W_q (K consecutive global batches B^s of the
timestamp-ordered stream) it walks the batches backward, keeps

    F      the dependency frontier (remote nodes whose state worker p will need)
    I_aux  ids of the auxiliary replay events inserted so far

and returns, per batch, the target events {e in B^s : pi(u) = p}, the auxiliary
events, and the candidate refresh set N_sync = F after the scan.  The mixed batch
(Eq. 5) is the timestamp-ordered union of the two with its event-type mask.

Readings where the algorithm is silent:
  * inside a batch the inner loop visits the events in reverse chronological
    order too (by (t, id) descending): the scan is a backward trace, so an
    event can be pulled in only by events that come after it in time -- except
    for the batch's own target events, whose remote destinations enter F before
    the batch is walked, exactly as the listing has it;
  * events are identified by their position in the stream, so I_aux never
    matters inside one worker's scan (a batch is visited once); it is kept
    because the listing keeps it;
  * the last window of the stream may hold fewer than K batches, the last batch
    fewer than B events.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Set, Tuple

import numpy as np


def window_batches(num_events: int, batch: int, K: int, q: int) -> List[range]:
    """Event-id ranges of the global batches of window W_q (Definition of the synchronisation window)."""
    nb = (num_events + batch - 1) // batch
    return [range(s * batch, min((s + 1) * batch, num_events)) for s in range(q * K, min((q + 1) * K, nb))]


def backward_scan(src: Sequence[int], dst: Sequence[int], owner: Sequence[int], p: int, batch: int, K: int, q: int
                  ) -> Tuple[Dict[int, List[int]], Dict[int, List[int]], Set[int]]:
    """Algorithm 1 for worker p and window q.

    Returns (targets, aux, n_sync): event ids per global batch index s (ascending ids = timestamp
    order, the stream being sorted) and the candidate boundary refresh set.
    """
    batches = window_batches(len(src), batch, K, q)
    tar: Dict[int, List[int]] = {}
    aux: Dict[int, List[int]] = {}
    F: Set[int] = set()
    I_aux: Set[int] = set()
    for j in reversed(range(len(batches))):            # batches in reverse chronological order
        s = q * K + j
        B_s = batches[j]
        tar[s] = [e for e in B_s if owner[src[e]] == p]
        F |= {int(dst[e]) for e in tar[s] if owner[dst[e]] != p}
        aux[s] = []
        for e in reversed(B_s):                        # reading: backward inside the batch as well
            u, v = int(src[e]), int(dst[e])
            if (u in F or v in F) and owner[u] != p:
                if e not in I_aux:
                    aux[s].append(e)
                    I_aux.add(e)
                F |= {i for i in (u, v) if owner[i] != p}
        aux[s].sort()
    return tar, aux, F


def mixed_batch(tar: List[int], aux: List[int]) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 5: timestamp-ordered union (ids ascend with time) and its event-type mask (1 = auxiliary)."""
    ids = np.array(sorted(set(tar) | set(aux)), dtype=np.int64)
    aux_set = set(aux)
    return ids, np.array([1 if int(e) in aux_set else 0 for e in ids], dtype=np.uint8)


def scan_stream(src, dst, owner, P: int, batch: int, K: int):
    """All workers and windows: role[p][e] in {0 absent, 1 target, 2 auxiliary} and N_sync[p][q]."""
    E = len(src)
    nb = (E + batch - 1) // batch
    Q = (nb + K - 1) // K
    role = np.zeros((P, E), dtype=np.uint8)
    n_sync: List[List[Set[int]]] = [[set() for _ in range(Q)] for _ in range(P)]
    for p in range(P):
        for q in range(Q):
            tar, aux, F = backward_scan(src, dst, owner, p, batch, K, q)
            for ids in tar.values():
                role[p, ids] = 1
            for ids in aux.values():
                role[p, ids] = 2
            n_sync[p][q] = F
    return role, n_sync
