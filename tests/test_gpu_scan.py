"""Backward dependency scan and mixed-batch construction on the GPU against the oracle (bit-exact)."""
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


def _gpu_scan(B, src, dst, owner, P, batch, K, want_sync=True):
    E, N = len(src), len(owner)
    nb = (E + batch - 1) // batch
    Q = (nb + K - 1) // K
    role = torch.full((P, E), 7, dtype=torch.uint8, device="cuda")
    n_sync = torch.full((P, Q), -1, dtype=torch.int32, device="cuda")
    sync = torch.full((P, Q, N), 7, dtype=torch.uint8, device="cuda") if want_sync else None
    scratch = torch.empty(B.backward_scan_scratch(E, batch, K, N, P), dtype=torch.int32, device="cuda")
    status = torch.full((1,), 9, dtype=torch.int32, device="cuda")
    B.backward_scan(_dev(src, np.int32), _dev(dst, np.int32), batch, K, _dev(owner, np.int32), P, role, n_sync, sync, scratch,
                    status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return role.cpu().numpy(), n_sync.cpu().numpy(), None if sync is None else sync.cpu().numpy()


def _check_against_oracle(B, src, dst, owner, P, batch, K):
    from oracle import scan as osc
    role, n_sync, sync = _gpu_scan(B, src, dst, owner, P, batch, K)
    role_ref, sets = osc.scan_stream(src, dst, owner, P, batch, K)
    assert np.array_equal(role, role_ref)
    for p in range(P):
        for q, F in enumerate(sets[p]):
            assert n_sync[p, q] == len(F), (p, q)
            assert set(np.nonzero(sync[p, q])[0].tolist()) == F, (p, q)
    return role


@pytest.mark.parametrize("seed,N,E,P,batch,K", [(1, 12, 60, 2, 5, 3), (2, 64, 1000, 4, 37, 4), (3, 500, 5000, 8, 200, 6),
                                                (4, 9, 700, 3, 300, 2), (5, 2000, 3001, 5, 1000, 1)])
def test_scan_random_streams_bit_exact(B, seed, N, E, P, batch, K):
    rng = np.random.default_rng(seed)
    w = 1.0 / np.arange(1, N + 1) ** 0.7
    w /= w.sum()
    src = rng.choice(N, size=E, p=w).astype(np.int32)
    dst = rng.choice(N, size=E, p=w).astype(np.int32)
    owner = rng.integers(0, P, size=N).astype(np.int32)
    _check_against_oracle(B, src, dst, owner, P, batch, K)


def test_scan_long_dependency_chain_and_single_worker(B):
    # a path 0 <- 1 <- 2 <- ... walked backward one event per sweep: the relaxation needs as many sweeps as events
    n = 300
    owner = np.ones(n + 2, np.int32)
    owner[0] = 0
    src = np.arange(n, 0, -1).astype(np.int32)          # chronological: (n, n-1), (n-1, n-2), ..., (1, 0)
    dst = (src - 1).astype(np.int32)
    src = np.concatenate([src, [0]]).astype(np.int32)   # last event: worker 0's target (0 -> 1); walking backward,
    dst = np.concatenate([dst, [1]]).astype(np.int32)   # (1,0) touches 1, (2,1) touches 1, (3,2) touches 2, ...
    role = _check_against_oracle(B, src, dst, owner, 2, n + 1, 1)
    assert (role[0, :n] == 2).all() and role[0, n] == 1
    # one worker owns every node: nothing is remote
    r1, ns, _ = _gpu_scan(B, src, dst, np.zeros(n + 2, np.int32), 1, 50, 3)
    assert (r1 == 1).all() and (ns == 0).all()


def test_scan_on_a_workload_stream_and_mixed_batches(B):
    from oracle import scan as osc
    cfg = wl.scaled(wl.CONFIGS["reddit"], num_events=12000)
    st = wl.make_stream(cfg)
    P, K = 4, 6
    owner = (np.arange(cfg.num_nodes) * 2654435761 % 2 ** 32 % P).astype(np.int32)    # a hash partition
    role = _check_against_oracle(B, st.src, st.dst, owner, P, cfg.batch, K)
    E, nb = cfg.num_events, cfg.num_batches
    src, dst, t, neg = _dev(st.src, np.int32), _dev(st.dst, np.int32), _dev(st.t, np.float64), _dev(st.neg, np.int32)
    for p in (0, 3):
        off, toff = torch.full((nb + 1,), -5, dtype=torch.int32, device="cuda"), torch.full((nb + 1,), -5, dtype=torch.int32, device="cuda")
        i32 = lambda: torch.full((E,), -9, dtype=torch.int32, device="cuda")
        mb = (i32(), i32(), torch.zeros(E, dtype=torch.float64, device="cuda"), i32(), torch.full((E,), 9, dtype=torch.uint8, device="cuda"))
        tg = (i32(), i32(), torch.zeros(E, dtype=torch.float64, device="cuda"), i32(), i32())
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.build_mixed(src, dst, t, neg, cfg.batch, _dev(role[p], np.uint8), off, toff, mb, tg, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        off, toff = off.cpu().numpy(), toff.cpu().numpy()
        mb, tg = [x.cpu().numpy() for x in mb], [x.cpu().numpy() for x in tg]
        for s in range(nb):
            lo, hi = s * cfg.batch, min(E, (s + 1) * cfg.batch)
            tar = [e for e in range(lo, hi) if role[p, e] == 1]
            aux = [e for e in range(lo, hi) if role[p, e] == 2]
            ids, mask = osc.mixed_batch(tar, aux)
            sl = slice(off[s], off[s + 1])
            assert np.array_equal(mb[3][sl], ids) and np.array_equal(mb[4][sl], mask), (p, s)
            assert np.array_equal(mb[0][sl], st.src[ids]) and np.array_equal(mb[1][sl], st.dst[ids])
            assert np.array_equal(mb[2][sl], st.t[ids])
            tl = slice(toff[s], toff[s + 1])
            assert np.array_equal(tg[4][tl], np.array(tar, dtype=np.int32)), (p, s)
            assert np.array_equal(tg[0][tl], st.src[tar]) and np.array_equal(tg[1][tl], st.dst[tar])
            assert np.array_equal(tg[2][tl], st.t[tar]) and np.array_equal(tg[3][tl], st.neg[tar])
        assert off[0] == 0 and toff[0] == 0 and off[-1] == (role[p] != 0).sum() and toff[-1] == (role[p] == 1).sum()
        assert (mb[3][off[-1]:] == -9).all() and (tg[4][toff[-1]:] == -9).all()        # nothing written past the end


def test_scan_errors_and_capacity(B):
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    u8 = torch.zeros(64, dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.TgnnError):
        B.backward_scan(z, z, 0, 2, z, 2, u8, z, None, z, st)          # batch < 1
    with pytest.raises(B.TgnnError):
        B.backward_scan(z, z, 4, 0, z, 2, u8, z, None, z, st)          # K < 1
    with pytest.raises(B.TgnnError):
        B.backward_scan_scratch(8, 4, 2, 0, 2)
    # a capacity that is too small is reported through the status word and nothing is written beyond it
    src = torch.arange(8, dtype=torch.int32, device="cuda") % 4
    role = torch.ones(8, dtype=torch.uint8, device="cuda")
    t = torch.arange(8, dtype=torch.float64, device="cuda")
    off, toff = torch.zeros(3, dtype=torch.int32, device="cuda"), torch.zeros(3, dtype=torch.int32, device="cuda")
    small = lambda dt: torch.full((5,), 77, dtype=dt, device="cuda")
    mb = (small(torch.int32), small(torch.int32), small(torch.float64), small(torch.int32), small(torch.uint8))
    tg = (small(torch.int32), small(torch.int32), small(torch.float64), None, small(torch.int32))
    B.build_mixed(src, src, t, None, 4, role, off, toff, mb, tg, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 2 and off.tolist() == [0, 4, 8]
    assert mb[3].tolist() == [0, 1, 2, 3, 4]
