"""Pins for the CPU oracle: each routine is checked against something other
than itself -- published vectors, brute force, closed forms, invariants the
paper states, library routines for the special cases that reduce to them,
and central finite differences for the gradient."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2608_16305_b200 import workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_cfg(orc, N=12, d=8, d_e=3, k=3, heads=2, **kw):
    return orc.make_config(N, d, d_e, k, heads, **kw)


def weights(cfg, seed=7, bias_scale=0.3):
    return wl.make_weights(cfg.d, cfg.d_e, seed, bias_scale=bias_scale)


# ------------------------------------------------------------ step (0) -----
def test_mixer_matches_published_splitmix64_vectors(oracle):
    vals = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64.txt")) if l.strip() and not l.startswith("#")]
    g = 0x9E3779B97F4A7C15
    for i, v in enumerate(vals, start=1):
        assert oracle.mix64((i * g) & (2 ** 64 - 1)) == v


def test_prune_targets_never_removed_and_light_batches_unchanged(oracle):
    rng = np.random.default_rng(1)
    n, N = 500, 200
    src = rng.integers(0, N, n)
    dst = rng.integers(0, N, n)
    eid = np.arange(n)
    aux = (rng.random(n) < 0.3).astype(np.uint8)
    # H = 0  =>  pruned batch == mixed batch (Eq. 11)
    keep, heavy = oracle.prune_mask(N, src, dst, eid, aux, force_heavy=0)
    assert heavy == 0 and keep.all()
    # H = 1, drop everything => exactly the pure-auxiliary set is removed (Eq. 10), targets stay
    keep, heavy = oracle.prune_mask(N, src, dst, eid, aux, force_heavy=1, drop_q32=0xFFFFFFFF)
    assert heavy == 1
    assert np.array_equal(keep, 1 - aux)
    # H = 1, half dropped: targets all kept, about half of the replay events go
    keep, _ = oracle.prune_mask(N, src, dst, eid, aux, force_heavy=1, drop_q32=1 << 31, seed=5, batch_idx=3)
    assert keep[aux == 0].all()
    # a different batch index gives a different subset (the hash is keyed by it)
    keep2, _ = oracle.prune_mask(N, src, dst, eid, aux, force_heavy=1, drop_q32=1 << 31, seed=5, batch_idx=4)
    assert not np.array_equal(keep, keep2)


def test_prune_drop_fraction_is_half(oracle):
    n = 40000
    src = np.zeros(n, np.int32)
    dst = np.ones(n, np.int32)
    keep, _ = oracle.prune_mask(4, src, dst, np.arange(n), np.ones(n, np.uint8), force_heavy=1, drop_q32=1 << 31, seed=9)
    frac = 1.0 - keep.mean()
    assert abs(frac - 0.5) < 4 * 0.5 / math.sqrt(n)


def test_prune_count_rule_against_recount(oracle):
    rng = np.random.default_rng(2)
    N = 300
    for trial in range(50):
        n = int(rng.integers(1, 400))
        s = 0.5 + 1.5 * rng.random()
        p = 1.0 / np.arange(1, N + 1) ** s
        p /= p.sum()
        src = rng.choice(N, n, p=p)
        dst = rng.choice(N, n, p=p)
        cnt = np.bincount(np.concatenate([src, dst]), minlength=N)
        touched = cnt[cnt > 0]
        expect = int(touched.max() > 4.0 * touched.mean())   # "max > 4 x mean" over touched nodes
        # avoid float ties in the comparison: skip exact equality cases
        if touched.max() * len(touched) == 4 * 2 * n:
            continue
        _, heavy = oracle.prune_mask(N, src, dst, np.arange(n), np.zeros(n, np.uint8))
        assert heavy == expect


def test_prune_handmade_uniform_and_hub(oracle):
    # uniform: 10 events over 20 distinct nodes -> max = mean = 1 -> light
    src, dst = np.arange(10), np.arange(10, 20)
    _, heavy = oracle.prune_mask(32, src, dst, np.arange(10), np.zeros(10, np.uint8))
    assert heavy == 0
    # hub: node 0 is the source of all 30 events, 30 distinct destinations:
    # counts {30, 1 x 30}, mean = 60/31 < 2, max = 30 > 4 x mean -> heavy
    src, dst = np.zeros(30, np.int32), np.arange(1, 31)
    _, heavy = oracle.prune_mask(32, src, dst, np.arange(30), np.zeros(30, np.uint8))
    assert heavy == 1


# ------------------------------------------------------------ step (1) -----
def test_neighbor_search_against_linear_scan(oracle):
    rng = np.random.default_rng(3)
    N, E, k = 9, 300, 4
    src = rng.integers(0, N, E).astype(np.int32)
    dst = rng.integers(0, N, E).astype(np.int32)
    t = np.cumsum(rng.integers(0, 2, E)).astype(np.float64)     # many ties by construction
    indptr, nbr, eid, ts = wl.build_tcsr(src, dst, t, N)
    nodes = np.concatenate([src, dst, rng.integers(0, N, 100).astype(np.int32)])
    times = np.concatenate([t, t, rng.uniform(-1, t[-1] + 2, 100)])
    nb, ne, nt, nc = oracle.sample_recent(indptr, nbr, eid, ts, nodes, times, k)
    for i in range(len(nodes)):
        # every earlier interaction of the node, ordered by (ts, eid), latest first
        hits = [(t[e], e, (dst[e] if r == 0 else src[e])) for e in range(E) for r in (0, 1)
                if (src[e] if r == 0 else dst[e]) == nodes[i] and t[e] < times[i]]
        hits.sort(key=lambda h: (h[0], h[1]))
        hits = hits[::-1][:k]
        assert nc[i] == len(hits)
        got = list(zip(nt[i, :nc[i]], ne[i, :nc[i]]))
        assert got == [(h[0], h[1]) for h in hits]
        # the neighbor of a self-loop entry is the node itself either way; otherwise it must match
        for s, h in enumerate(hits):
            e = h[1]
            assert nb[i, s] in (src[e], dst[e])
            assert {int(nb[i, s]), int(nodes[i])} == {int(src[e]), int(dst[e])}
        assert (nb[i, nc[i]:] == -1).all() and (ne[i, nc[i]:] == -1).all() and (nt[i, nc[i]:] == 0).all()


def test_first_event_of_a_node_has_no_neighbors(oracle):
    src = np.array([0, 1, 0], np.int32)
    dst = np.array([2, 3, 3], np.int32)
    t = np.array([1.0, 2.0, 3.0])
    g = wl.build_tcsr(src, dst, t, 4)
    _, _, _, nc = oracle.sample_recent(*g, [0, 2, 1, 3, 0, 3], [1.0, 1.0, 2.0, 2.0, 3.0, 3.0], 5)
    assert nc.tolist() == [0, 0, 0, 0, 1, 1]


# ----------------------------------------------------- time encoding -------
def test_time_encoding_closed_forms(oracle):
    cfg = small_cfg(oracle, d=4, phi_f32=False)
    b = np.array([0.0, 0.5, -1.0, 2.0])
    out = oracle.time_encode(cfg, np.array([1.0, 2.0, 3.0, 4.0]), b, [0.0])
    assert np.allclose(out[0], np.cos(b), atol=1e-15)            # dt = 0 -> cos(b)
    out = oracle.time_encode(cfg, np.zeros(4), b, [123.0])
    assert np.allclose(out[0], np.cos(b), atol=1e-15)            # w = 0 -> cos(b)
    out = oracle.time_encode(cfg, np.full(4, math.pi), np.zeros(4), [1.0, 2.0])
    assert np.allclose(out[0], -1.0) and np.allclose(out[1], 1.0)  # cos(pi) = -1, cos(2 pi) = 1


def test_time_encoding_fp32_argument(oracle):
    # in the model's precision the argument is one fp32 fma of fp32-rounded inputs
    cfg = small_cfg(oracle, d=2, phi_f32=True)
    w, b, dt = np.array([1.0, 0.37]), np.array([0.0, 0.2]), 123456.789
    out = oracle.time_encode(cfg, w, b, [dt])
    arg = np.float32(w.astype(np.float32)) * np.float32(dt) + b.astype(np.float32)   # exact in fp64
    ref = np.cos(np.float32(arg.astype(np.float64)).astype(np.float64))
    # w=1,b=0 has no fma rounding subtlety: cos(float32(dt)) exactly
    assert out[0, 0] == math.cos(float(np.float32(dt)))
    assert abs(out[0, 1] - ref[1]) < 1e-12


# ------------------------------------------------------------- GRU ---------
def _gru_setup(oracle, cfg, W):
    P = oracle.pack_params(cfg, W)
    N, d = cfg.num_nodes, cfg.d
    rng = np.random.default_rng(4)
    mem = rng.normal(size=(N, d))
    return P, mem


def test_gru_closed_forms(oracle):
    cfg = small_cfg(oracle, round_state_f32=False)
    d, dm = cfg.d, 3 * cfg.d + cfg.d_e
    W = {n: np.zeros(s) for n, s in wl.param_shapes(cfg.d, cfg.d_e).items()}
    P, mem = _gru_setup(oracle, cfg, W)
    msg = np.random.default_rng(0).normal(size=(2, dm))
    msg[0, :d] = mem[3]
    uniq, win, t = [3], [0], [5.0]
    # all-zero weights: r = z = 1/2, n = tanh(0) = 0  ->  h' = h / 2
    m2, lu2 = oracle.memory_update(cfg, P, msg, t, uniq, win, mem, np.zeros(cfg.num_nodes))
    assert np.allclose(m2[3], mem[3] / 2, atol=1e-15) and lu2[3] == 5.0
    assert np.array_equal(np.delete(m2, 3, 0), np.delete(mem, 3, 0))
    # update gate saturated open: h' = h
    W["gru_b_i"][d:2 * d] = 40.0
    m2, _ = oracle.memory_update(cfg, oracle.pack_params(cfg, W), msg, t, uniq, win, mem, np.zeros(cfg.num_nodes))
    assert np.allclose(m2[3], mem[3], atol=1e-12)
    # update gate shut, candidate bias c: h' = tanh(c)
    W["gru_b_i"][d:2 * d] = -40.0
    W["gru_b_i"][2 * d:] = 0.7
    m2, _ = oracle.memory_update(cfg, oracle.pack_params(cfg, W), msg, t, uniq, win, mem, np.zeros(cfg.num_nodes))
    assert np.allclose(m2[3], math.tanh(0.7), atol=1e-12)


def test_gru_matches_library_cell(oracle):
    cfg = small_cfg(oracle, round_state_f32=False)
    d, dm = cfg.d, 3 * cfg.d + cfg.d_e
    W = weights(cfg)
    P, mem = _gru_setup(oracle, cfg, W)
    rng = np.random.default_rng(5)
    U = 5
    uniq = np.array([1, 2, 5, 7, 11])
    msg = rng.normal(size=(2 * U, dm))
    win = np.array([9, 0, 4, 3, 6])
    for u in range(U):
        msg[win[u], :d] = mem[uniq[u]]
    m2, _ = oracle.memory_update(cfg, P, msg, np.arange(U, dtype=float), uniq, win, mem, np.zeros(cfg.num_nodes))
    cell = torch.nn.GRUCell(dm, d).double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(W["gru_w_i"].astype(np.float64)))
        cell.weight_hh.copy_(torch.from_numpy(W["gru_w_h"].astype(np.float64)))
        cell.bias_ih.copy_(torch.from_numpy(W["gru_b_i"].astype(np.float64)))
        cell.bias_hh.copy_(torch.from_numpy(W["gru_b_h"].astype(np.float64)))
        ref = cell(torch.from_numpy(msg[win]), torch.from_numpy(mem[uniq])).numpy()
    assert np.allclose(m2[uniq], ref, atol=1e-13)


def test_state_rounding_flag(oracle):
    cfg = small_cfg(oracle, round_state_f32=True)
    W = weights(cfg)
    P, mem = _gru_setup(oracle, cfg, W)
    dm = 3 * cfg.d + cfg.d_e
    msg = np.random.default_rng(6).normal(size=(2, dm))
    msg[1, :cfg.d] = mem[0]
    m2, _ = oracle.memory_update(cfg, P, msg, [1.0], [0], [1], mem, np.zeros(cfg.num_nodes))
    assert np.array_equal(m2[0], m2[0].astype(np.float32).astype(np.float64))


# ------------------------------------------------ messages / reduction -----
def _random_events(rng, N, n, t0=0.0):
    src = rng.integers(0, N, n).astype(np.int32)
    dst = rng.integers(0, N, n).astype(np.int32)
    t = t0 + np.cumsum(rng.random(n))
    return src, dst, t


def test_message_layout(oracle):
    cfg = small_cfg(oracle, phi_f32=False)
    d, de = cfg.d, cfg.d_e
    W = weights(cfg)
    P = oracle.pack_params(cfg, W)
    rng = np.random.default_rng(8)
    mem = rng.normal(size=(cfg.num_nodes, d))
    lu = rng.random(cfg.num_nodes) * 3
    ef = rng.normal(size=(40, de)).astype(np.float32)
    src, dst, t = np.array([2, 5], np.int32), np.array([7, 5], np.int32), np.array([4.0, 6.5])
    eid = np.array([17, 31], np.int32)
    msg, node = oracle.build_messages(cfg, P, mem, lu, ef, src, dst, t, eid, keep=[1, 1])
    assert node.tolist() == [2, 7, 5, 5]
    w, b = W["time_w"].astype(np.float64), W["time_b"].astype(np.float64)
    for j, (s, o, e, tt) in enumerate([(2, 7, 17, 4.0), (7, 2, 17, 4.0), (5, 5, 31, 6.5), (5, 5, 31, 6.5)]):
        assert np.array_equal(msg[j, :d], mem[s])                 # own memory first
        assert np.array_equal(msg[j, d:2 * d], mem[o])            # then the other endpoint
        assert np.array_equal(msg[j, 2 * d:2 * d + de], ef[e].astype(np.float64))
        assert np.allclose(msg[j, 2 * d + de:], np.cos(w * (tt - lu[s]) + b), atol=1e-14)
    msg, node = oracle.build_messages(cfg, P, mem, lu, ef, src, dst, t, eid, keep=[0, 1])
    assert node.tolist() == [-1, -1, 5, 5] and not msg[:2].any()


def test_bf16_features_are_decoded(oracle):
    cfg = small_cfg(oracle, feat_bf16=True, phi_f32=False)
    W = weights(cfg)
    P = oracle.pack_params(cfg, W)
    x = np.array([[1.0, -2.5, 0.15625]], np.float32)
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)      # these values are exact in bf16
    mem = np.zeros((cfg.num_nodes, cfg.d))
    msg, _ = oracle.build_messages(cfg, P, mem, np.zeros(cfg.num_nodes), bits, [0], [1], [1.0], [0])
    assert msg[0, 2 * cfg.d:2 * cfg.d + 3].tolist() == [1.0, -2.5, 0.15625]


def test_latest_reduction_is_last_writer_in_key_order(oracle):
    rng = np.random.default_rng(9)
    N = 15
    for trial in range(30):
        n = int(rng.integers(1, 60))
        src = rng.integers(0, N, n).astype(np.int32)
        dst = rng.integers(0, N, n).astype(np.int32)
        t = rng.integers(0, 6, n).astype(np.float64)           # heavy ties, unsorted
        eid = rng.permutation(100)[:n].astype(np.int32)
        keep = rng.random(n) < 0.8
        node = np.stack([src, dst], 1).reshape(-1)
        node[np.repeat(~keep, 2)] = -1
        uniq, win = oracle.reduce_latest(node, t, eid, N)
        order = sorted(range(2 * n), key=lambda j: (t[j >> 1], eid[j >> 1], j & 1))
        last = {}
        for j in order:                                        # sequential "last writer wins"
            if node[j] >= 0:
                last[int(node[j])] = j
        assert uniq.tolist() == sorted(last)
        assert win.tolist() == [last[u] for u in sorted(last)]


def test_batched_update_equals_sequential_replay_when_nodes_occur_once(oracle):
    # Eq. 1-2 applied event by event == one batched step when every node occurs once in the batch
    cfg = small_cfg(oracle, N=40, round_state_f32=False, phi_f32=False)
    W = weights(cfg)
    P = oracle.pack_params(cfg, W)
    rng = np.random.default_rng(10)
    mem0 = rng.normal(size=(cfg.num_nodes, cfg.d))
    lu0 = rng.random(cfg.num_nodes)
    perm = rng.permutation(cfg.num_nodes)[:24].astype(np.int32)
    src, dst = perm[:12], perm[12:]
    t = 2.0 + np.cumsum(rng.random(12))
    eid = np.arange(12, dtype=np.int32)
    ef = rng.normal(size=(12, cfg.d_e)).astype(np.float32)
    # batched
    msg, node = oracle.build_messages(cfg, P, mem0, lu0, ef, src, dst, t, eid)
    uniq, win = oracle.reduce_latest(node, t, eid, cfg.num_nodes)
    mem_b, lu_b = oracle.memory_update(cfg, P, msg, t, uniq, win, mem0, lu0)
    # sequential
    mem_s, lu_s = mem0.copy(), lu0.copy()
    for i in range(12):
        m1, n1 = oracle.build_messages(cfg, P, mem_s, lu_s, ef, src[i:i + 1], dst[i:i + 1], t[i:i + 1], eid[i:i + 1])
        u1, w1 = oracle.reduce_latest(n1, t[i:i + 1], eid[i:i + 1], cfg.num_nodes)
        mem_s, lu_s = oracle.memory_update(cfg, P, m1, t[i:i + 1], u1, w1, mem_s, lu_s)
    assert np.allclose(mem_b, mem_s, atol=1e-14) and np.array_equal(lu_b, lu_s)


# ---------------------------------------------------------- attention ------
def _embed_case(oracle, cfg, W, cnt, seed=11, perm=None):
    P = oracle.pack_params(cfg, W)
    rng = np.random.default_rng(seed)
    N, d, de, k = cfg.num_nodes, cfg.d, cfg.d_e, cfg.k
    mem = rng.normal(size=(N, d))
    ef = rng.normal(size=(50, de)).astype(np.float32)
    R = len(cnt)
    nodes = rng.integers(0, N, R).astype(np.int32)
    times = 50 + rng.random(R) * 10
    nb = rng.integers(0, N, (R, k)).astype(np.int32)
    ne = rng.integers(0, 50, (R, k)).astype(np.int32)
    nt = rng.random((R, k)) * 40
    cnt = np.asarray(cnt, np.int32)
    for i in range(R):
        nb[i, cnt[i]:] = -1
        ne[i, cnt[i]:] = -1
        nt[i, cnt[i]:] = 0
    if perm is not None:
        for i in range(R):
            p = perm[:cnt[i]] if len(perm) >= cnt[i] else None
            p = np.argsort(np.argsort(perm))[:cnt[i]] if p is None else np.array(sorted(range(cnt[i]), key=lambda s: perm[s]))
            nb[i, :cnt[i]], ne[i, :cnt[i]], nt[i, :cnt[i]] = nb[i, p], ne[i, p], nt[i, p]
    h = oracle.embed(cfg, P, mem, ef, nodes, times, nb, ne, nt, cnt)
    return dict(h=h, mem=mem, ef=ef, nodes=nodes, times=times, nb=nb, ne=ne, nt=nt, cnt=cnt, P=P)


def _z_rows(cfg, W, c, i):
    """[m_nbr || x_e || Phi(t - ts)] rows of root i (fp64 argument)."""
    w, b = W["time_w"].astype(np.float64), W["time_b"].astype(np.float64)
    rows = []
    for s in range(c["cnt"][i]):
        rows.append(np.concatenate([c["mem"][c["nb"][i, s]], c["ef"][c["ne"][i, s]].astype(np.float64),
                                    np.cos(w * (c["times"][i] - c["nt"][i, s]) + b)]))
    return np.array(rows)


def _merge(W, a, m):
    cat = np.concatenate([a, m])
    return np.maximum(W["w_o"].astype(np.float64) @ cat + W["b_o"].astype(np.float64), 0)


def test_attention_special_cases(oracle):
    cfg = small_cfg(oracle, phi_f32=False)
    W = weights(cfg)
    # make the output ReLU transparent enough to see the attention vector: large positive bias
    W["b_o"][:] = 50.0
    c = _embed_case(oracle, cfg, W, cnt=[1, 0, 3])
    Wv, bv = W["w_v"].astype(np.float64), W["b_v"].astype(np.float64)
    # cnt = 1: softmax over one slot is 1 -> a = V_1
    z = _z_rows(cfg, W, c, 0)
    assert np.allclose(c["h"][0], _merge(W, Wv @ z[0] + bv, c["mem"][c["nodes"][0]]), atol=1e-12)
    # cnt = 0: a = 0
    assert np.allclose(c["h"][1], _merge(W, np.zeros(cfg.d), c["mem"][c["nodes"][1]]), atol=1e-12)
    # W_k = 0: all logits equal -> a = mean of V_s
    W2 = dict(W)
    W2["w_k"] = np.zeros_like(W["w_k"])
    c2 = _embed_case(oracle, cfg, W2, cnt=[1, 0, 3])
    z = _z_rows(cfg, W2, c2, 2)
    vmean = (z @ Wv.T + bv).mean(0)
    assert np.allclose(c2["h"][2], _merge(W2, vmean, c2["mem"][c2["nodes"][2]]), atol=1e-12)


def test_attention_is_invariant_to_slot_order(oracle):
    cfg = small_cfg(oracle, phi_f32=False)
    W = weights(cfg)
    a = _embed_case(oracle, cfg, W, cnt=[3, 2, 3])
    b = _embed_case(oracle, cfg, W, cnt=[3, 2, 3], perm=[2, 0, 1])
    assert not np.array_equal(a["nb"], b["nb"])
    assert np.allclose(a["h"], b["h"], atol=1e-13)


def test_attention_core_matches_library_sdpa(oracle):
    cfg = small_cfg(oracle, d=8, heads=2, k=3, phi_f32=False)
    W = weights(cfg)
    W["b_o"][:] = 50.0
    c = _embed_case(oracle, cfg, W, cnt=[3, 3])
    d, H = cfg.d, cfg.heads
    w, b = W["time_w"].astype(np.float64), W["time_b"].astype(np.float64)
    for i in range(2):
        z = torch.from_numpy(_z_rows(cfg, W, c, i))
        zq = torch.from_numpy(np.concatenate([c["mem"][c["nodes"][i]], np.cos(b)]))
        Q = torch.from_numpy(W["w_q"]).double() @ zq + torch.from_numpy(W["b_q"]).double()
        K = z @ torch.from_numpy(W["w_k"]).double().T + torch.from_numpy(W["b_k"]).double()
        V = z @ torch.from_numpy(W["w_v"]).double().T + torch.from_numpy(W["b_v"]).double()
        q = Q.view(1, H, 1, d // H)
        kk = K.view(-1, H, d // H).permute(1, 0, 2).unsqueeze(0)
        vv = V.view(-1, H, d // H).permute(1, 0, 2).unsqueeze(0)
        a = torch.nn.functional.scaled_dot_product_attention(q, kk, vv).reshape(d).numpy()
        assert np.allclose(c["h"][i], _merge(W, a, c["mem"][c["nodes"][i]]), atol=1e-12)


# --------------------------------------------------------------- loss ------
def _full_case(oracle, cfg, W, seed=12, n_u=10, n_q=6, t_scale=1.0):
    rng = np.random.default_rng(seed)
    N, d, de, k = cfg.num_nodes, cfg.d, cfg.d_e, cfg.k
    E = 60
    src, dst, t = _random_events(rng, N, E)
    t *= t_scale
    g = wl.build_tcsr(src, dst, t, N)
    ef = rng.normal(size=(E, de)).astype(np.float32)
    mem = rng.normal(size=(N, d)) * 0.5
    lu = rng.random(N) * t[E // 2]
    u = slice(E - n_u - n_q, E - n_q)
    q = slice(E - n_q, E)
    upd = (src[u], dst[u], t[u], np.arange(E)[u].astype(np.int32), None)
    nodes = np.concatenate([src[q], dst[q], rng.integers(0, N, n_q).astype(np.int32)])
    times = np.concatenate([t[q]] * 3)
    nb = oracle.sample_recent(*g, nodes, times, k)
    return dict(P=oracle.pack_params(cfg, W), mem=mem, lu=lu, ef=ef, upd=upd, roots=(nodes, times) + nb, n_q=n_q)


def test_loss_closed_forms_and_masking(oracle):
    cfg = small_cfg(oracle, N=20, phi_f32=False, round_state_f32=False)
    W = weights(cfg)
    for n in ("w_1", "b_1", "w_2", "b_2"):
        W[n] = np.zeros_like(W[n])
    c = _full_case(oracle, cfg, W)
    r = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], None)
    assert abs(r.loss - 2 * math.log(2)) < 1e-14                 # zero head: score = 0 both ways
    W = weights(cfg)
    c = _full_case(oracle, cfg, W)
    r = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"],
                              np.zeros(c["n_q"], np.uint8))
    assert r.loss == 0.0 and r.gradnorm == 0.0 and not r.grads.any()   # Eq. 13, empty target set


def test_loss_is_masked_mean_of_library_bce(oracle):
    cfg = small_cfg(oracle, N=20, phi_f32=False, round_state_f32=False)
    W = weights(cfg)
    c = _full_case(oracle, cfg, W)
    mask = np.array([1, 0, 1, 1, 0, 1], np.uint8)
    r = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], mask, want_grads=False)
    h = torch.from_numpy(r.h)
    nq = c["n_q"]
    W1, b1 = torch.from_numpy(W["w_1"]).double(), torch.from_numpy(W["b_1"]).double()
    w2, b2 = torch.from_numpy(W["w_2"]).double(), torch.from_numpy(W["b_2"]).double()

    def score(a, b):
        return torch.relu(torch.cat([a, b], 1) @ W1.T + b1) @ w2 + b2

    pos, neg = score(h[:nq], h[nq:2 * nq]), score(h[:nq], h[2 * nq:])
    bce = torch.nn.functional.binary_cross_entropy_with_logits
    per = bce(pos, torch.ones_like(pos), reduction="none") + bce(neg, torch.zeros_like(neg), reduction="none")
    m = torch.from_numpy(mask.astype(np.float64))
    assert abs(r.loss - float((per * m).sum() / m.sum())) < 1e-13
    # masked-out events contribute nothing term by term: changing their negatives changes nothing
    full = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], mask)
    roots2 = list(c["roots"])
    roots2[0] = roots2[0].copy()
    roots2[0][2 * nq + 1] = (roots2[0][2 * nq + 1] + 3) % cfg.num_nodes       # event 1 is masked out
    nb = oracle.sample_recent(*wl.build_tcsr(np.zeros(1, np.int32), np.ones(1, np.int32), np.zeros(1), cfg.num_nodes),
                              roots2[0][2 * nq + 1:2 * nq + 2], roots2[1][2 * nq + 1:2 * nq + 2], cfg.k)
    for a, b in zip(roots2[2:], nb):
        a[2 * nq + 1] = b[0]
    alt = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], tuple(roots2), c["n_q"], mask)
    assert alt.loss == full.loss and np.allclose(alt.grads, full.grads, atol=1e-15)


# ----------------------------------------------------------- backward ------
@pytest.mark.parametrize("seed", [12, 13])
def test_gradient_against_central_differences(oracle, seed):
    cfg = small_cfg(oracle, N=14, d=6, d_e=3, k=3, heads=2, phi_f32=False, round_state_f32=False)
    W = weights(cfg, seed=seed)
    W["time_w"] = np.array([1.0, 0.5, 0.25, 0.1, 0.05, 0.01], np.float32)
    c = _full_case(oracle, cfg, W, seed=seed, t_scale=0.2)
    mask = np.array([1, 1, 0, 1, 1, 1], np.uint8)
    args = (c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], mask)
    base = oracle.loss_and_grads(cfg, c["P"], *args)
    assert len(base.uniq) > 3 and base.gradnorm > 0
    lay = oracle.param_layout(cfg)
    shapes = wl.param_shapes(cfg.d, cfg.d_e)
    eps = 1e-6
    rng = np.random.default_rng(0)
    for name in oracle.PARAM_NAMES:
        size = int(np.prod(shapes[name]))
        idx = np.arange(size) if size <= 40 else rng.choice(size, 40, replace=False)
        for j in idx:
            p = c["P"].copy()
            p[lay[name] + j] += eps
            lp = oracle.loss_and_grads(cfg, p, *args, want_grads=False).loss
            p[lay[name] + j] -= 2 * eps
            lm = oracle.loss_and_grads(cfg, p, *args, want_grads=False).loss
            fd = (lp - lm) / (2 * eps)
            g = base.grads[lay[name] + j]
            assert abs(fd - g) <= 2e-7 + 1e-5 * abs(g), (name, int(j), fd, g)
        # every tensor must actually receive gradient in this case (no silently dead path)
        assert np.abs(base.grads[lay[name]:lay[name] + size]).max() > 0, name
    assert abs(base.gradnorm - math.sqrt((base.grads ** 2).sum())) < 1e-14


def test_time_encoder_gradient_with_the_fp32_argument(oracle):
    """The backward pass of the message's time encoding when the argument is fp32 by definition: a hand
    case with one update event (a self-loop, so a single winner whose gate gradient is the update cell's
    bias gradient) and roots without neighbors at phase 0 (so the attention side contributes nothing to the
    encoder).  Then  dL/dw_c = -sin(arg_c) * dt32 * dx_c  and  dL/db_c = -sin(arg_c) * dx_c  with
    arg_c = w_c * dt32 formed in fp32, dt32 = fp32(16777217) = 16777216, and dx = W_i[:, Phi columns]^T dG
    computed here from the oracle's own bias gradient.  The fp64 reading (dt = 16777217) gives other sines
    and another factor, so a backward that forgot either rounding fails."""
    N, d, k = 5, 4, 3
    cfg = oracle.make_config(N, d, 0, k, 2, phi_f32=True, round_state_f32=False)
    W = wl.make_weights(d, 0, 3, bias_scale=0.3)
    W["time_w"] = np.array([1.0, 0.5, 0.25, 2.0 ** -20], np.float32)
    W["time_b"] = np.zeros(d, np.float32)
    P = oracle.pack_params(cfg, W)
    rng = np.random.default_rng(5)
    mem = rng.normal(size=(N, d)) * 0.5
    lu = np.zeros(N)
    t_ev = 16777217.0                                   # 2^24 + 1: not an fp32 number
    upd = (np.array([1], np.int32), np.array([1], np.int32), np.array([t_ev]), np.array([0], np.int32), None)
    nodes = np.array([1, 2, 3], np.int32)
    times = np.full(3, t_ev + 1.0)
    none = (np.full((3, k), -1, np.int32), np.full((3, k), -1, np.int32), np.zeros((3, k)), np.zeros(3, np.int32))
    r = oracle.loss_and_grads(cfg, P, mem, lu, None, upd, (nodes, times) + none, 1, None)
    assert list(r.uniq) == [1] and list(r.winner) == [1]            # role 1 wins the tie on (t, eid)
    lay = oracle.param_layout(cfg)
    dmsg = 3 * d
    dG = r.grads[lay["gru_b_i"]:lay["gru_b_i"] + 3 * d]             # single winner: the gate gradient itself
    Wi = np.asarray(W["gru_w_i"], np.float64).reshape(3 * d, dmsg)
    dx = Wi[:, 2 * d:].T @ dG
    assert np.abs(dx).min() > 0
    dt32 = float(np.float32(t_ev))
    assert dt32 == 16777216.0
    arg32 = (W["time_w"].astype(np.float32) * np.float32(dt32)).astype(np.float64)   # exact products, phase 0
    gw, gb = r.grads[lay["time_w"]:lay["time_w"] + d], r.grads[lay["time_b"]:lay["time_b"] + d]
    assert np.allclose(gb, -np.sin(arg32) * dx, rtol=1e-11, atol=1e-15)
    assert np.allclose(gw, -np.sin(arg32) * dt32 * dx, rtol=1e-11, atol=1e-9)
    # the fp64 reading of the same case differs in both factors
    arg64 = W["time_w"].astype(np.float64) * t_ev
    assert np.abs(np.sin(arg64) - np.sin(arg32)).max() > 0.1
    cfg64 = oracle.make_config(N, d, 0, k, 2, phi_f32=False, round_state_f32=False)
    r64 = oracle.loss_and_grads(cfg64, P, mem, lu, None, upd, (nodes, times) + none, 1, None)
    dx64 = Wi[:, 2 * d:].T @ r64.grads[lay["gru_b_i"]:lay["gru_b_i"] + 3 * d]
    assert np.allclose(r64.grads[lay["time_w"]:lay["time_w"] + d], -np.sin(arg64) * t_ev * dx64, rtol=1e-11, atol=1e-9)
    assert not np.allclose(r64.grads[lay["time_w"]:lay["time_w"] + d], gw, rtol=1e-3)


def test_relu_gate_hints_apply_only_inside_the_window(oracle):
    cfg = small_cfg(oracle, N=20, phi_f32=False, round_state_f32=False)
    W = weights(cfg)
    c = _full_case(oracle, cfg, W)
    args = (cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], None)
    base = oracle.loss_and_grads(*args)
    R, nq, d = len(c["roots"][0]), c["n_q"], cfg.d
    own_h = (base.h > 0).astype(np.uint8)
    zeros_h, zeros_hid = np.zeros((R, d), np.uint8), np.zeros((2 * nq, d), np.uint8)
    # a zero-width window ignores the hints entirely
    r = oracle.loss_and_grads(*args, h_gate=zeros_h, hid_gate=zeros_hid, gate_eps=0.0)
    assert r.loss == base.loss and np.array_equal(r.grads, base.grads)
    # a narrow window around zero touches no unit of this case: wrong hints change nothing
    r = oracle.loss_and_grads(*args, h_gate=1 - own_h, hid_gate=zeros_hid, gate_eps=1e-9)
    assert r.loss == base.loss and np.array_equal(r.grads, base.grads)
    # a window covering everything with all gates closed switches every unit off: h = 0, score = b_2
    r = oracle.loss_and_grads(*args, h_gate=zeros_h, hid_gate=zeros_hid, gate_eps=1.0)
    assert not r.h.any()
    b2 = float(W["b_2"][0])
    assert abs(r.loss - (math.log1p(math.exp(-b2)) + math.log1p(math.exp(b2)))) < 1e-12


# --------------------------------------------------------------- Adam ------
def test_adam_first_step_closed_form(oracle):
    cfg = small_cfg(oracle, lr=1e-3)
    g = np.array([0.5, -2.0, 1e-3, 0.0])
    p0 = np.array([1.0, 1.0, 1.0, 1.0])
    p, m, v, step = oracle.adam(cfg, g, p0, np.zeros(4), np.zeros(4), 0)
    # from zero moments the bias-corrected ratio is g / (|g| + eps)
    assert step == 1
    assert np.allclose(p - p0, -1e-3 * g / (np.abs(g) + 1e-8), atol=1e-15)
    assert np.allclose(m, 0.1 * g) and np.allclose(v, 0.001 * g * g)
    opt_p = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.Adam([opt_p], lr=1e-3, betas=(0.9, 0.999), eps=1e-8)
    pp, mm, vv, st = p0, np.zeros(4), np.zeros(4), 0
    for it in range(3):                                     # and three steps against the library optimizer
        gi = g * (it + 1)
        opt_p.grad = torch.from_numpy(gi.copy())
        opt.step()
        pp, mm, vv, st = oracle.adam(cfg, gi, pp, mm, vv, st)
    assert np.allclose(pp, opt_p.detach().numpy(), atol=1e-12)


# ------------------------------------------------------ whole-step glue ----
def test_step_sequencing_uses_post_update_memory_and_lag_one(oracle):
    cfg = small_cfg(oracle, N=20, phi_f32=False, round_state_f32=False)
    W = weights(cfg)
    c = _full_case(oracle, cfg, W)
    r = oracle.loss_and_grads(cfg, c["P"], c["mem"], c["lu"], c["ef"], c["upd"], c["roots"], c["n_q"], None, want_grads=False)
    # the same result from the piecewise routines: messages -> reduce -> GRU -> embed on the *updated* table
    msg, node = oracle.build_messages(cfg, c["P"], c["mem"], c["lu"], c["ef"], *c["upd"][:4])
    uniq, win = oracle.reduce_latest(node, c["upd"][2], c["upd"][3], cfg.num_nodes)
    mem2, lu2 = oracle.memory_update(cfg, c["P"], msg, c["upd"][2], uniq, win, c["mem"], c["lu"])
    h = oracle.embed(cfg, c["P"], mem2, c["ef"], *c["roots"])
    assert np.array_equal(uniq, r.uniq) and np.array_equal(win, r.winner)
    assert np.allclose(mem2, r.memory_post, atol=1e-15) and np.array_equal(lu2, r.last_update_post)
    assert np.allclose(h, r.h, atol=1e-14)
    h_stale = oracle.embed(cfg, c["P"], c["mem"], c["ef"], *c["roots"])
    assert not np.allclose(h_stale, r.h)
