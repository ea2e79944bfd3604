"""Backward dependency scan and mixed-batch construction (Algorithm 1, Eq. 5): the oracle against a
hand-worked window, an independent fixed-point formulation, and the invariants the construction promises."""
import os

import numpy as np
import pytest

from oracle import scan as osc

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    ev, rows = [], []
    with open(os.path.join(HERE, "golden", "scan_worked.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            if line[0] == "e":
                _, i, u, v = line.split()
                assert int(i) == len(ev)
                ev.append((int(u), int(v)))
            else:
                head, tar, aux, ns = [x.strip() for x in line[1:].split("|")]
                ids = lambda s: [] if s == "-" else [int(x) for x in s.split()]
                p, q = [int(x) for x in head.split()]
                rows.append((p, q, ids(tar), ids(aux), set(ids(ns))))
    return ev, rows


def test_oracle_hand_worked_window():
    ev, rows = _golden()
    src, dst = [u for u, _ in ev], [v for _, v in ev]
    owner = [0, 0, 0, 1, 1, 1]
    for p, q, tar, aux, ns in rows:
        t, a, F = osc.backward_scan(src, dst, owner, p, batch=3, K=2, q=q)
        assert sorted(sum(t.values(), [])) == tar, (p, q)
        assert sorted(sum(a.values(), [])) == aux, (p, q)
        assert F == ns, (p, q)
    ids, mask = osc.mixed_batch([3, 5], [4])
    assert ids.tolist() == [3, 4, 5] and mask.tolist() == [0, 1, 0]      # Eq. 5 on batch 1 of worker 0


def _random_stream(rng, N, E, P, hub=0.3):
    w = 1.0 / np.arange(1, N + 1) ** hub
    w /= w.sum()
    src = rng.choice(N, size=E, p=w).astype(np.int32)
    dst = rng.choice(N, size=E, p=w).astype(np.int32)
    owner = rng.integers(0, P, size=N).astype(np.int32)
    return src, dst, owner


def _fixed_point(src, dst, owner, p, batch, K, q):
    """The same sets from a different route: entry positions relaxed to their least fixed point.

    Scan position i counts events of the window backward from its last event.  entry[x] = position
    from which node x is in the frontier: the first scanned position of batch s for remote destinations
    of the batch's targets, i + 1 for remote endpoints of an inserted event at position i.  An event at
    position i with a remote source is inserted iff some endpoint has entry <= i.  All events are
    relaxed together until nothing changes."""
    E = len(src)
    nb = (E + batch - 1) // batch
    lo, hi = q * K * batch, min(E, min((q + 1) * K, nb) * batch)
    n = hi - lo
    pos_of = lambda e: hi - 1 - e
    INF = 1 << 30
    entry = np.full(len(owner), INF, dtype=np.int64)
    for e in range(lo, hi):
        if owner[src[e]] == p and owner[dst[e]] != p:
            s_end = min(hi, (e // batch + 1) * batch)          # one past the batch's last event
            entry[dst[e]] = min(entry[dst[e]], pos_of(s_end - 1))
    ins = np.zeros(n, bool)
    changed = True
    while changed:
        changed = False
        for e in range(lo, hi):                                  # any order: a relaxation sweep
            i = pos_of(e)
            if owner[src[e]] != p and min(entry[src[e]], entry[dst[e]]) <= i:
                if not ins[i]:
                    ins[i] = changed = True
                for x in (src[e], dst[e]):
                    if owner[x] != p and entry[x] > i + 1:
                        entry[x] = i + 1
                        changed = True
    aux = sorted(hi - 1 - i for i in np.nonzero(ins)[0])
    return aux, set(int(x) for x in np.nonzero(entry < INF)[0])


@pytest.mark.parametrize("seed,N,E,P,batch,K", [(1, 12, 60, 2, 5, 3), (2, 30, 200, 4, 16, 4), (3, 50, 333, 3, 20, 6),
                                                (4, 8, 90, 2, 9, 1), (5, 200, 1000, 8, 50, 6)])
def test_oracle_equals_fixed_point_formulation(seed, N, E, P, batch, K):
    rng = np.random.default_rng(seed)
    src, dst, owner = _random_stream(rng, N, E, P)
    nb = (E + batch - 1) // batch
    for p in range(P):
        for q in range((nb + K - 1) // K):
            t, a, F = osc.backward_scan(src, dst, owner, p, batch, K, q)
            aux_fp, F_fp = _fixed_point(src, dst, owner, p, batch, K, q)
            assert sorted(sum(a.values(), [])) == aux_fp, (p, q)
            assert F == F_fp, (p, q)


def test_oracle_invariants_of_the_construction():
    rng = np.random.default_rng(9)
    N, E, P, batch, K = 40, 400, 4, 25, 4
    src, dst, owner = _random_stream(rng, N, E, P, hub=0.8)
    role, n_sync = osc.scan_stream(src, dst, owner, P, batch, K)
    nb = (E + batch - 1) // batch
    for p in range(P):
        assert np.array_equal(role[p] == 1, owner[src] == p)                 # targets: exactly the source-owned events
        assert not np.any((role[p] == 2) & (owner[src] == p))                # no target is ever auxiliary
        for q in range((nb + K - 1) // K):
            F = n_sync[p][q]
            assert all(owner[x] != p for x in F)                             # only remote nodes are refresh candidates
            lo, hi = q * K * batch, min(E, (q + 1) * K * batch)
            for e in range(lo, hi):
                if role[p, e] == 1 and owner[dst[e]] != p:
                    assert dst[e] in F                                        # every remote destination of a target
                    s0 = (e // batch) * batch
                    # every event of the window up to the end of the target's batch that touches that
                    # destination from a remote source is replayed
                    for e2 in range(lo, min(hi, s0 + batch)):
                        if owner[src[e2]] != p and (src[e2] == dst[e] or dst[e2] == dst[e]):
                            assert role[p, e2] == 2, (p, e, e2)
                if role[p, e] == 2:
                    assert all(x in F for x in (src[e], dst[e]) if owner[x] != p)
    # one worker owns everything: nothing is remote, nothing is replayed
    r1, s1 = osc.scan_stream(src, dst, np.zeros(N, np.int32), 1, batch, K)
    assert (r1 == 1).all() and all(not F for F in s1[0])
    # a longer window can only add replay events for the batches it already covered
    role_k1, _ = osc.scan_stream(src, dst, owner, P, batch, 1)
    assert np.all((role_k1 == 2) <= (role == 2))
