"""Boundary cache refresh and synchronised gradient on the GPU against the oracle: the exchange plan and
the row movers bit-exactly, several workers emulated on one device by running their kernels one after
the other (none of them waits for another) with the all-to-all written out as segment copies."""
import numpy as np
import pytest
import torch

from paper_2608_16305_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2608_16305_b200 import binding
    binding.load_library()
    return binding


def _dev(a, dt):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).cuda()


def _stream(seed, N, E, P):
    rng = np.random.default_rng(seed)
    w = 1.0 / np.arange(1, N + 1) ** 0.7
    w /= w.sum()
    src = rng.choice(N, size=E, p=w).astype(np.int32)
    dst = rng.choice(N, size=E, p=w).astype(np.int32)
    owner = rng.integers(0, P, size=N).astype(np.int32)
    return src, dst, owner


def _scan(B, src, dst, owner, P, batch, K):
    E, N = len(src), len(owner)
    nb = (E + batch - 1) // batch
    Q = (nb + K - 1) // K
    role = torch.empty((P, E), dtype=torch.uint8, device="cuda")
    n_sync = torch.empty((P, Q), dtype=torch.int32, device="cuda")
    sync = torch.empty((P, Q, N), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(B.backward_scan_scratch(E, batch, K, N, P), dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.backward_scan(_dev(src, np.int32), _dev(dst, np.int32), batch, K, _dev(owner, np.int32), P, role, n_sync, sync, scratch, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return sync, n_sync.cpu().numpy(), Q


def _oracle_sets(src, dst, owner, P, batch, K, Q):
    from oracle import scan as osc
    return [[osc.backward_scan(src, dst, owner, p, batch, K, q)[2] for p in range(P)] for q in range(Q)]


@pytest.mark.parametrize("seed,N,E,P,batch,K", [(1, 12, 60, 2, 5, 3), (2, 64, 1000, 4, 37, 4), (3, 2500, 6000, 8, 200, 6),
                                                (4, 1024, 900, 3, 300, 2), (5, 5000, 3001, 5, 1000, 1)])
def test_refresh_plan_bit_exact(B, seed, N, E, P, batch, K):
    """Receive and send lists of every worker and window against the oracle's plan on the oracle's own
    N_sync sets: node ranges below, at and above one sweep of the block, ragged last window."""
    from oracle import refresh as orf
    from paper_2608_16305_b200 import distributed as D
    src, dst, owner = _stream(seed, N, E, P)
    sync, n_sync, Q = _scan(B, src, dst, owner, P, batch, K)
    sets = _oracle_sets(src, dst, owner, P, batch, K, Q)
    owner_dev = _dev(owner, np.int32)
    plans = [D.RefreshPlan(sync, owner_dev, n_sync, P, me) for me in range(P)]
    some = 0
    for q in range(Q):
        send = orf.refresh_plan(sets[q], owner)
        for me, pl in enumerate(plans):
            rn, sn = pl.recv_nodes[q].cpu().numpy(), pl.send_nodes[q].cpu().numpy()
            for o in range(P):
                assert rn[pl.recv_off[q, o]:pl.recv_off[q, o + 1]].tolist() == send[o][me], (q, me, o)
                assert sn[pl.send_off[q, o]:pl.send_off[q, o + 1]].tolist() == send[me][o], (q, me, o)
                some += len(send[o][me])
            assert pl.recv_off[q, -1] == len(sets[q][me])
    assert some > 0


def test_refresh_plan_reports_short_capacity_and_owned_requests(B):
    N, P, Q = 300, 3, 2
    rng = np.random.default_rng(0)
    owner = rng.integers(0, P, N).astype(np.int32)
    sync = np.zeros((P, Q, N), np.uint8)
    for p in range(P):
        for q in range(Q):
            sync[p, q, (owner != p) & (rng.random(N) < 0.3)] = 1
    need = int(sync.sum(axis=(0, 2)).max())

    def run(flags, cap, me=0):
        out = [torch.full((Q, max(cap, 1)), -5, dtype=torch.int32, device="cuda") for _ in range(2)]
        off = [torch.zeros((Q, P + 1), dtype=torch.int32, device="cuda") for _ in range(2)]
        st = torch.full((1,), 9, dtype=torch.int32, device="cuda")
        B.refresh_plan(_dev(flags, np.uint8), _dev(owner, np.int32), P, Q, me, cap, out[0], off[0], out[1], off[1], st)
        torch.cuda.synchronize()
        return int(st.item()), out, off
    st, out, off = run(sync, need)
    assert st == 0
    st, out, off = run(sync, 5)
    assert st == 2                                            # too small: flagged, nothing written past the end
    assert off[0].cpu().numpy()[:, -1].tolist() == sync[0].sum(axis=1).tolist()   # the counts are still the true ones
    bad = sync.copy()
    mine = np.nonzero(owner == 1)[0][0]
    bad[1, 0, mine] = 1                                       # worker 1 asks for a node it owns
    st, out, off = run(bad, need + 1, me=1)
    assert st == 3
    assert mine not in out[0][0, :int(off[0][0, -1].item())].cpu().numpy().tolist()
    with pytest.raises(B.TgnnError):
        B.refresh_plan(_dev(sync, np.uint8), _dev(owner, np.int32), P, Q, P, need, out[0], off[0], out[1], off[1],
                       torch.zeros(1, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("d,N,n", [(100, 9000, 4001), (2, 50, 50), (256, 3000, 777), (32, 1000, 0), (172, 20000, 20000)])
def test_pack_and_unpack_rows_bit_exact(B, d, N, n):
    rng = np.random.default_rng(d + n)
    mem = rng.standard_normal((N, d)).astype(np.float32)
    lu = (rng.random(N) * 1e9 - 3e8)
    lu[::7] = -0.0
    lu[1::11] = np.nextafter(1e300, 2e300)                    # both halves of the fp64 matter
    nodes = rng.permutation(N)[:n].astype(np.int32)
    m, t = _dev(mem, np.float32), _dev(lu, np.float64)
    packed = torch.full((max(n, 1) * (d + 2) + 3,), 7.0, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    nd = _dev(nodes, np.int32) if n else None
    B.pack_rows(m, t, nd, packed, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    pk = packed.cpu().numpy()
    assert np.all(pk[n * (d + 2):] == 7.0)
    rows = pk[:n * (d + 2)].reshape(n, d + 2)
    assert np.array_equal(rows[:, :d], mem[nodes])
    assert np.array_equal(np.ascontiguousarray(rows[:, d:]).view(np.float64)[:, 0].view(np.uint64), lu[nodes].view(np.uint64))
    # unpack into another table: exactly the listed nodes change, to the packed values
    mem2 = rng.standard_normal((N, d)).astype(np.float32)
    lu2 = rng.random(N)
    m2, t2 = _dev(mem2, np.float32), _dev(lu2, np.float64)
    B.unpack_rows(m2, t2, nd, packed, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    want_m, want_t = mem2.copy(), lu2.copy()
    want_m[nodes], want_t[nodes] = mem[nodes], lu[nodes]
    assert np.array_equal(m2.cpu().numpy(), want_m)
    assert np.array_equal(t2.cpu().numpy().view(np.uint64), want_t.view(np.uint64))


def test_row_movers_flag_bad_node_ids_and_refuse_bad_shapes(B):
    N, d = 40, 6
    m = torch.ones((N, d), dtype=torch.float32, device="cuda")
    t = torch.ones(N, dtype=torch.float64, device="cuda")
    nodes = _dev([3, -1, 40, 7], np.int32)
    packed = torch.full((4 * (d + 2),), 5.0, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pack_rows(m, t, nodes, packed, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 4
    rows = packed.cpu().numpy().reshape(4, d + 2)
    assert np.all(rows[[1, 2]] == 0) and np.all(rows[[0, 3], :d] == 1)
    st.zero_()
    m2 = torch.zeros((N, d), dtype=torch.float32, device="cuda")
    B.unpack_rows(m2, t, nodes, packed, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 4
    assert m2.sum().item() == 2 * d                           # rows 3 and 7 only
    odd = torch.ones((N, 5), dtype=torch.float32, device="cuda")
    with pytest.raises(B.TgnnError):
        B.pack_rows(odd, t, nodes, packed, st)
    with pytest.raises(B.TgnnError):
        B.pack_rows(m, t, nodes, packed[:8], st)


def test_refresh_of_emulated_workers_matches_oracle(B):
    """P workers' tables on one device.  Every worker packs, the all-to-all is written out as the segment
    copies it stands for (segment r of worker o's send buffer -> segment o of worker r's receive buffer),
    every worker unpacks; the tables then equal the oracle's, bit for bit, window after window."""
    from oracle import refresh as orf
    from paper_2608_16305_b200 import distributed as D
    P, N, E, batch, K, d = 4, 3000, 9000, 250, 6, 100
    src, dst, owner = _stream(11, N, E, P)
    sync, n_sync, Q = _scan(B, src, dst, owner, P, batch, K)
    sets = _oracle_sets(src, dst, owner, P, batch, K, Q)
    owner_dev = _dev(owner, np.int32)
    rng = np.random.default_rng(2)
    mem = [rng.standard_normal((N, d)).astype(np.float32) for _ in range(P)]
    lu = [rng.random(N) * 1e6 for _ in range(P)]
    mem_dev = [_dev(m, np.float32) for m in mem]
    lu_dev = [_dev(t, np.float64) for t in lu]
    workers = [D.BoundaryRefresh(D.RefreshPlan(sync, owner_dev, n_sync, P, me), d) for me in range(P)]
    w = d + 2
    moved = 0
    for q in range(Q):
        for me, wk in enumerate(workers):
            wk.pack(q, mem_dev[me], lu_dev[me])
        for o, src_w in enumerate(workers):                       # the all-to-all, segment by segment
            so = src_w.plan.send_off[q]
            for r, dst_w in enumerate(workers):
                ro = dst_w.plan.recv_off[q]
                n = int(so[r + 1] - so[r])
                assert n == int(ro[o + 1] - ro[o])
                dst_w.recv_buf[ro[o] * w:(ro[o] + n) * w].copy_(src_w.send_buf[so[r] * w:(so[r] + n) * w])
                moved += n
        for me, wk in enumerate(workers):
            wk.unpack(q, mem_dev[me], lu_dev[me])
        torch.cuda.synchronize()
        mem, lu = orf.boundary_refresh(mem, lu, sets[q], owner)
        for me in range(P):
            assert int(workers[me].status.item()) == 0
            assert np.array_equal(mem_dev[me].cpu().numpy(), mem[me]), (q, me)
            assert np.array_equal(lu_dev[me].cpu().numpy(), lu[me]), (q, me)
        # between windows the workers' copies drift apart again
        for me in range(P):
            mem[me] = mem[me] + np.float32(0.25) * (me + 1)
            mem_dev[me] += 0.25 * (me + 1)
    assert moved > 0


def test_nccl_single_rank_moves_rows_and_reduces_the_gradient_buffer():
    """The collectives of the multi-worker form on a real NCCL communicator (one rank: the only size this
    machine offers): the all-to-all of packed rows between the library's pack and unpack kernels, the flag
    broadcast, and an all-reduce directly on the context's gradient buffer followed by the apply call."""
    import os
    import socket
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = r"""
import os, sys, numpy as np, torch, torch.distributed as dist
sys.path.insert(0, %r)
from paper_2608_16305_b200 import binding as B, distributed as D, trainer as T, workload as wl
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, init_method="tcp://127.0.0.1:" + os.environ["PORT"],
                        device_id=torch.device("cuda", 0))
N, d, n = 5000, 100, 1200
rng = np.random.default_rng(0)
mem = torch.from_numpy(rng.standard_normal((N, d)).astype(np.float32)).cuda()
lu = torch.from_numpy(rng.random(N) * 1e5).cuda()
perm = rng.permutation(N)
src_nodes, dst_nodes = perm[:n].astype(np.int32), perm[n:2 * n].astype(np.int32)
# a one-worker plan that sends n rows to itself: rows of src_nodes arrive as the new state of dst_nodes
plan = D.RefreshPlan.from_lists(torch.from_numpy(dst_nodes[None]).cuda(), np.array([[0, n]]),
                                torch.from_numpy(src_nodes[None]).cuda(), np.array([[0, n]]), 1, 0)
ref = D.BoundaryRefresh(plan, d)
want_m, want_t = mem.clone(), lu.clone()
want_m[dst_nodes.astype(np.int64)] = mem[src_nodes.astype(np.int64)]
want_t[dst_nodes.astype(np.int64)] = lu[src_nodes.astype(np.int64)]
assert D.broadcast_decision(1, torch.device("cuda", 0)) == 1
ref.run(0, mem, lu)
torch.cuda.synchronize()
assert int(ref.status.item()) == 0 and ref.rows_sent == n and ref.rows_received == n
assert torch.equal(mem, want_m) and torch.equal(lu, want_t)
# gradient buffer: a deferred step, an all-reduce on the library's own memory, then the apply call
cfg = wl.scaled(wl.CONFIGS["tiny"], num_events=2000)
dw = T.DeviceWorkload(wl.make_stream(cfg))
tr = T.Trainer(dw, wl.make_weights(cfg.d, cfg.d_e, cfg.seed, bias_scale=0.1), math_mode=B.TGNN_MATH_TF32)
tr.lib.set_grad_sync(True)
with torch.cuda.stream(tr.stream):
    for b in range(4):
        tr.step(b)
        g = tr.lib.grad_buffer()
        before = g.clone()
        dist.all_reduce(g, op=dist.ReduceOp.SUM)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(g, before) and float(g.abs().max()) > 0
        tr.lib.apply_gradient(1.0, tr.gradnorm)
    torch.cuda.synchronize()
assert int(tr.step_count.item()) == 4 and tr.lib.status() == 0
want = float(torch.linalg.vector_norm(tr.lib.grad_buffer().double()))
assert abs(float(tr.gradnorm.item()) - want) <= 1e-6 * want
dist.destroy_process_group()
print("ok")
""" % root
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    env = dict(os.environ, PORT=str(port), NCCL_NVLS_ENABLE="0")
    p = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, timeout=300)
    assert p.returncode == 0, p.stderr.decode()[-3000:]
    assert b"ok" in p.stdout
