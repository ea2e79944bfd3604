"""Boundary cache refresh and synchronised gradient: the oracle against a hand-worked exchange, the
properties the refresh promises, the scan's N_sync sets, and the model oracle's own gradients."""
import os

import numpy as np
import pytest

from oracle import refresh as orf
from oracle import scan as osc

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    owner, nsync, send, after = None, {}, {}, {}
    with open(os.path.join(HERE, "golden", "refresh_worked.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, rest = line.split(None, 1)
            if key == "owner":
                owner = [int(x) for x in rest.split()]
                continue
            head, tail = [x.strip() for x in rest.split(":")]
            h = [int(x) for x in head.split()]
            vals = [] if tail == "-" else [int(x) for x in tail.split()]
            if key == "nsync":
                nsync[h[0]] = set(vals)
            elif key == "send":
                send[(h[0], h[1])] = vals
            elif key == "after":
                after[(h[0], h[1])] = vals
    return owner, nsync, send, after


def _tables(P, N, d=2):
    mem = [np.array([[100 * w + 10 * n + 1 + j for j in range(d)] for n in range(N)], dtype=np.float64) for w in range(P)]
    lu = [np.array([1000 * w + n for n in range(N)], dtype=np.float64) for w in range(P)]
    return mem, lu


def test_hand_worked_exchange():
    owner, nsync, send, after = _golden()
    P, N = 3, len(owner)
    ns = [nsync[p] for p in range(P)]
    plan = orf.refresh_plan(ns, owner)
    for o in range(P):
        for p in range(P):
            assert plan[o][p] == send.get((o, p), []), (o, p)
    mem, lu = _tables(P, N)
    m2, t2 = orf.boundary_refresh(mem, lu, ns, owner)
    for w in range(P):
        for n in range(N):
            if (w, n) in after:
                a = after[(w, n)]
                assert list(m2[w][n]) == a[:2] and t2[w][n] == a[2], (w, n)
            else:
                assert np.array_equal(m2[w][n], mem[w][n]) and t2[w][n] == lu[w][n], (w, n)


def test_requesting_an_owned_node_is_an_error():
    with pytest.raises(ValueError):
        orf.refresh_plan([{0}, set()], [0, 1])


def test_refresh_properties_on_scanned_windows():
    """N_sync from the backward dependency scan (Algorithm 1) on a random stream: every requested node is
    remote, travels exactly once and from its owner; afterwards the requester's copy equals the owner's,
    every other row everywhere is untouched, owners' own rows never change, and a second refresh changes
    nothing."""
    rng = np.random.default_rng(3)
    P, N, E, B, K, d = 4, 60, 600, 25, 3, 5
    src, dst = rng.integers(0, N, E), rng.integers(0, N, E)
    owner = rng.integers(0, P, N)
    Q = (E // B + K - 1) // K
    for q in range(Q):
        ns = [osc.backward_scan(src, dst, owner, p, B, K, q)[2] for p in range(P)]
        assert any(ns)
        plan = orf.refresh_plan(ns, owner)
        for p in range(P):
            got = sorted(n for o in range(P) for n in plan[o][p])
            assert got == sorted(ns[p])
            assert all(owner[n] == o for o in range(P) for n in plan[o][p])
            assert plan[p][p] == []
        mem = [rng.standard_normal((N, d)) for _ in range(P)]
        lu = [rng.random(N) * 100 for _ in range(P)]
        m2, t2 = orf.boundary_refresh(mem, lu, ns, owner)
        for p in range(P):
            for n in range(N):
                if n in ns[p]:
                    o = owner[n]
                    assert np.array_equal(m2[p][n], mem[o][n]) and t2[p][n] == lu[o][n]
                else:
                    assert np.array_equal(m2[p][n], mem[p][n]) and t2[p][n] == lu[p][n]
        m3, t3 = orf.boundary_refresh(m2, t2, ns, owner)
        assert all(np.array_equal(a, b) for a, b in zip(m2, m3)) and all(np.array_equal(a, b) for a, b in zip(t2, t3))


def test_synchronised_gradient_closed_form():
    """Workers minimising 0.5 |x - a_p|^2 have local gradients x - a_p; their mean is x - mean(a_p), the
    gradient of the mean loss, with norm |x - mean(a_p)|."""
    rng = np.random.default_rng(0)
    x = rng.standard_normal(40)
    a = [rng.standard_normal(40) for _ in range(5)]
    mean, g = orf.synchronised_gradient([x - ap for ap in a])
    want = x - sum(a) / 5.0
    assert np.allclose(mean, want, rtol=0, atol=1e-15)
    assert abs(g - np.linalg.norm(want)) <= 1e-14
    one, g1 = orf.synchronised_gradient([x])
    assert np.array_equal(one, x) and g1 == float(np.sqrt(np.sum(x * x)))


def test_synchronised_gradient_of_two_half_batches_is_the_full_batch_gradient(oracle):
    """Eq. 13 averages over the unmasked events, so two workers that score the two equal halves of a batch
    (complementary masks) hold local gradients whose mean is the gradient of the whole batch."""
    from paper_2608_16305_b200 import workload as wl
    o = oracle
    cfg = wl.CONFIGS["tiny"]
    stream = wl.make_stream(cfg)
    W = wl.make_weights(cfg.d, cfg.d_e, cfg.seed, bias_scale=0.1)
    ocfg = o.make_config(cfg.num_nodes, cfg.d, cfg.d_e, cfg.k, cfg.heads)
    params = o.pack_params(ocfg, W).astype(np.float64)
    rng = np.random.default_rng(1)
    memory = rng.standard_normal((cfg.num_nodes, cfg.d)) * 0.3
    last_update = np.zeros(cfg.num_nodes)
    b = 7
    q = slice(b * cfg.batch, (b + 1) * cfg.batch)
    u = slice((b - 1) * cfg.batch, b * cfg.batch)
    nq = cfg.batch
    assert nq % 2 == 0
    nodes = np.concatenate([stream.src[q], stream.dst[q], stream.neg[q]])
    times = np.concatenate([stream.t[q]] * 3)
    nb = o.sample_recent(stream.indptr, stream.nbr, stream.eid, stream.ts, nodes, times, cfg.k)
    upd = (stream.src[u], stream.dst[u], stream.t[u], np.arange(u.start, u.stop, dtype=np.int32), None)
    roots = (nodes, times) + nb
    first = (np.arange(nq) < nq // 2).astype(np.uint8)
    run = lambda mask: o.loss_and_grads(ocfg, params, memory, last_update, stream.efeat() if cfg.d_e else None, upd,
                                        roots, nq, mask)
    full, a, c = run(None), run(first), run(1 - first)
    mean, g = orf.synchronised_gradient([a.grads, c.grads])
    scale = np.abs(full.grads).max()
    assert np.abs(mean - full.grads).max() <= 1e-12 * scale
    assert abs(g - full.gradnorm) <= 1e-12 * full.gradnorm
    assert abs(0.5 * (a.loss + c.loss) - full.loss) <= 1e-13


def test_two_rank_refresh_flag_and_gradient_sum_over_gloo():
    """The host side of the exchanges with two CPU processes: split sizes and routing of the all-to-all
    from each rank's plan, the coordinator's flag, and the gradient all-reduce followed by the apply call.
    The row movers are replaced by index copies (the kernels are covered on the GPU); the tables after the
    refresh must equal the oracle's."""
    import socket
    import subprocess
    import sys
    root = os.path.dirname(HERE)
    code = r"""
import os, sys, numpy as np, torch, torch.distributed as dist
sys.path.insert(0, %r)
from oracle import refresh as orf, scan as osc
from paper_2608_16305_b200 import distributed as D
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", rank=rank, world_size=2, init_method="tcp://127.0.0.1:" + os.environ["PORT"])
rng = np.random.default_rng(5)                       # same stream on both ranks
P, N, E, Bsz, K, d = 2, 80, 400, 20, 4, 6
src, dst = rng.integers(0, N, E), rng.integers(0, N, E)
owner = rng.integers(0, P, N)
Q = (E // Bsz + K - 1) // K
mem = [rng.standard_normal((N, d)).astype(np.float32) for _ in range(P)]
lu = [rng.random(N) * 50 for _ in range(P)]
sets = [[osc.backward_scan(src, dst, owner, p, Bsz, K, q)[2] for p in range(P)] for q in range(Q)]
cap = max(sum(len(s) for s in sets[q]) for q in range(Q))
rn, sn = np.zeros((Q, cap), np.int32), np.zeros((Q, cap), np.int32)
ro, so = np.zeros((Q, P + 1), np.int64), np.zeros((Q, P + 1), np.int64)
for q in range(Q):
    plan = orf.refresh_plan(sets[q], owner)
    r_list = [plan[o][rank] for o in range(P)]
    s_list = [plan[rank][r] for r in range(P)]
    ro[q, 1:], so[q, 1:] = np.cumsum([len(x) for x in r_list]), np.cumsum([len(x) for x in s_list])
    rn[q, :ro[q, -1]], sn[q, :so[q, -1]] = sum(r_list, []), sum(s_list, [])
plan = D.RefreshPlan.from_lists(torch.from_numpy(rn), ro, torch.from_numpy(sn), so, P, rank)

def pack(memory, last_update, nodes, packed, status):
    n = nodes.numel()
    rows = packed[:n * (d + 2)].view(n, d + 2)
    rows[:, :d] = memory[nodes.long()]
    rows[:, d:] = last_update[nodes.long()].view(torch.float32).view(n, 2)

def unpack(memory, last_update, nodes, packed, status):
    n = nodes.numel()
    rows = packed[:n * (d + 2)].view(n, d + 2)
    memory[nodes.long()] = rows[:, :d]
    last_update[nodes.long()] = rows[:, d:].contiguous().view(torch.float64).view(n)

ref = D.BoundaryRefresh(plan, d, pack=pack, unpack=unpack)
my_mem, my_lu = torch.from_numpy(mem[rank].copy()), torch.from_numpy(lu[rank].copy())
moved = 0
for q in range(Q):
    # the coordinator (rank 0) decides; rank 1's own opinion is overruled
    s = D.broadcast_decision(q %% 2 if rank == 0 else 1 - q %% 2, torch.device("cpu"))
    assert s == q %% 2
    if s:
        ref.run(q, my_mem, my_lu)
        mem, lu = orf.boundary_refresh(mem, lu, sets[q], owner)
    assert np.array_equal(my_mem.numpy(), mem[rank]) and np.array_equal(my_lu.numpy(), lu[rank]), q
moved = ref.rows_received
assert moved == sum(len(sets[q][rank]) for q in range(Q) if q %% 2) and moved > 0

class FakeLib:                                          # records what the gradient synchronisation asks of the library
    def __init__(self):
        self.g = torch.arange(5, dtype=torch.float32) * (rank + 1)
        self.applied = None
    def grad_buffer(self):
        return self.g
    def apply_gradient(self, scale, out):
        self.applied = (scale, self.g.clone())
lib = FakeLib()
D.synchronise_gradient(lib, None)
scale, g = lib.applied
mean, norm = orf.synchronised_gradient([np.arange(5.0), 2 * np.arange(5.0)])
assert scale == 0.5 and np.array_equal(g.numpy() * scale, mean.astype(np.float32))
dist.barrier()
print("ok", rank)
""" % root
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE))
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err.decode()[-3000:]
        assert b"ok" in out
