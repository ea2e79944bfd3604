"""Pins for the JODIE-variant oracle: library cells, closed forms, brute-force replay, finite differences."""
import numpy as np
import pytest
import torch

from oracle import jodie as oj
from oracle import oracle as orc


def _cfg(N=40, d=8, de=6, phi_f32=False, round_state=False):
    return orc.make_config(N, d, de, 4, 2, phi_f32=phi_f32, round_state_f32=round_state)


def _weights(rng, d, de, scale=0.5):
    W = {n: rng.uniform(-scale, scale, size=s) for n, s in oj.param_shapes(d, de).items()}
    W["time_w"] = 10.0 ** (-2.0 * np.arange(d) / max(d - 1, 1))
    return W


def _case(rng, cfg, n_u=30, nq=12, t0=5.0):
    N, d, de = cfg.num_nodes, cfg.d, cfg.d_e
    E = 200
    efeat = rng.normal(size=(E, de)).astype(np.float32)
    mem = rng.normal(scale=0.5, size=(N, d))
    lu = rng.uniform(0.0, t0, size=N)
    u_src, u_dst = rng.integers(0, N // 2, n_u), rng.integers(0, N, n_u)
    u_t = np.sort(rng.uniform(t0, t0 + 3.0, n_u))
    u_eid = np.arange(n_u) + 7
    keep = (rng.uniform(size=n_u) < 0.85).astype(np.uint8)
    tgt = (rng.integers(0, N // 2, nq), rng.integers(0, N, nq), rng.integers(0, N, nq), np.sort(rng.uniform(t0 + 3.0, t0 + 4.0, nq)))
    return efeat, mem, lu, (u_src, u_dst, u_t, u_eid, keep), tgt


def test_recurrent_cell_is_the_library_cell():
    rng = np.random.default_rng(0)
    d, dmsg = 8, 30
    W = {"rnn_w_i": rng.normal(size=(d, dmsg)), "rnn_w_h": rng.normal(size=(d, d)), "rnn_b_i": rng.normal(size=d),
         "rnn_b_h": rng.normal(size=d)}
    X, H = rng.normal(size=(5, dmsg)), rng.normal(size=(5, d))
    cell = torch.nn.RNNCell(dmsg, d, nonlinearity="tanh").double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(W["rnn_w_i"])); cell.weight_hh.copy_(torch.from_numpy(W["rnn_w_h"]))
        cell.bias_ih.copy_(torch.from_numpy(W["rnn_b_i"])); cell.bias_hh.copy_(torch.from_numpy(W["rnn_b_h"]))
        ref = cell(torch.from_numpy(X), torch.from_numpy(H)).numpy()
    assert np.abs(oj.rnn_rows(W, X, H) - ref).max() < 1e-14
    Z = {k: np.zeros_like(v) for k, v in W.items()}
    assert np.all(oj.rnn_rows(Z, X, H) == 0.0)                                   # zero cell: tanh(0)


def test_time_projection_closed_forms():
    m = np.array([[1.0, -2.0, 0.5]])
    z = np.zeros(3)
    assert np.array_equal(oj.time_projection(m, np.array([7.0]), z, z), m)       # no drift: the memory itself
    assert np.array_equal(oj.time_projection(m, np.array([0.0]), np.ones(3), np.array([0.5, 0.0, 1.0])), m * [1.5, 1.0, 2.0])
    assert np.array_equal(oj.time_projection(m, np.array([2.0]), np.array([0.25, -0.5, 1.0]), z), m * [1.5, 0.0, 3.0])


@pytest.mark.parametrize("phi_f32", [False, True])
def test_time_arguments_reproduce_the_pinned_encoding(phi_f32):
    rng = np.random.default_rng(1)
    cfg = _cfg(d=16, phi_f32=phi_f32)
    w = (10.0 ** (-9.0 * np.arange(16) / 15)).astype(np.float32).astype(np.float64)
    b = rng.uniform(-1, 1, 16).astype(np.float32).astype(np.float64)
    dt = np.concatenate([rng.uniform(-50, 5e5, 300), [0.0, 1e-3, 123456.789]])
    arg, dtv = oj.time_args(phi_f32, w, b, dt)
    ref = orc.time_encode(cfg, w, b, dt)
    assert np.abs(np.cos(arg) - ref).max() <= (1e-6 if phi_f32 else 1e-12)
    if phi_f32:   # the argument is an fp32 number and almost always the same one (a differing rounding moves cos by ~1e-2 at 5e5)
        assert np.array_equal(arg, arg.astype(np.float32).astype(np.float64))
        assert np.mean(np.cos(arg) == ref) > 0.999
        assert np.array_equal(dtv, dt.astype(np.float32).astype(np.float64))


def test_winner_messages_match_the_attention_models_message_builder():
    rng = np.random.default_rng(2)
    cfg = _cfg(phi_f32=True)
    d, de = cfg.d, cfg.d_e
    efeat, mem, lu, upd, _ = _case(rng, cfg)
    W = _weights(rng, d, de)
    W = {k: v.astype(np.float32).astype(np.float64) for k, v in W.items()}
    uniq, winner, X, H, _, _, win_t = oj.winner_messages(cfg, W, mem, lu, efeat, upd)
    lay = orc.param_layout(cfg)
    flat = np.zeros(lay["total"])
    flat[lay["time_w"]:lay["time_w"] + d] = W["time_w"]
    flat[lay["time_b"]:lay["time_b"] + d] = W["time_b"]
    msg, node = orc.build_messages(cfg, flat, mem, lu, efeat, *upd[:4], keep=upd[4])
    assert np.array_equal(node[winner], uniq)
    assert np.abs(X - msg[winner]).max() <= 1e-6 and np.mean(X == msg[winner]) > 0.99
    assert np.array_equal(H, mem[uniq]) and np.array_equal(win_t, upd[2][winner >> 1])


def test_memory_update_equals_event_by_event_replay_when_nodes_occur_once():
    rng = np.random.default_rng(3)
    cfg = _cfg(N=64)
    d, de = cfg.d, cfg.d_e
    efeat, mem, lu, _, tgt = _case(rng, cfg)
    perm = rng.permutation(64)
    n_u = 20
    u_src, u_dst = perm[:n_u], perm[n_u:2 * n_u]                                  # every node occurs once
    u_t = np.sort(rng.uniform(6.0, 9.0, n_u))
    upd = (u_src, u_dst, u_t, np.arange(n_u), None)
    W = _weights(rng, d, de)
    res = oj.step(cfg, oj.pack(d, de, W), mem, lu, efeat, upd, tgt)
    m2, l2 = mem.copy(), lu.copy()
    for i in range(n_u):                                                           # Eq. 1-2, one event at a time
        u, v, t = u_src[i], u_dst[i], u_t[i]
        x = efeat[i].astype(np.float64)
        new = {}
        for a, b in ((u, v), (v, u)):
            phi = np.cos(W["time_w"] * (t - lu[a]) + W["time_b"])
            msg = np.concatenate([mem[a], mem[b], x, phi])
            new[a] = np.tanh(W["rnn_w_i"] @ msg + W["rnn_b_i"] + W["rnn_w_h"] @ mem[a] + W["rnn_b_h"])
        for a in new:
            m2[a], l2[a] = new[a], t
    assert np.abs(res.memory_post - m2).max() < 1e-13 and np.array_equal(res.last_update_post, l2)


def test_loss_special_cases_and_constant_rows():
    rng = np.random.default_rng(4)
    cfg = _cfg()
    d, de = cfg.d, cfg.d_e
    efeat, mem, lu, upd, tgt = _case(rng, cfg)
    W = _weights(rng, d, de)
    W0 = dict(W, w_2=np.zeros(d), b_2=np.zeros(1))
    assert abs(oj.step(cfg, oj.pack(d, de, W0), mem, lu, efeat, upd, tgt).loss - 2 * np.log(2)) < 1e-14
    r = oj.step(cfg, oj.pack(d, de, W), mem, lu, efeat, upd, tgt, loss_mask=np.zeros(len(tgt[0]), np.uint8))
    assert r.loss == 0.0 and not r.grads.any()                                     # Eq. 13: empty mask
    # masked-out events contribute nothing
    mask = (rng.uniform(size=len(tgt[0])) < 0.5).astype(np.uint8)
    mask[0] = 1
    ra = oj.step(cfg, oj.pack(d, de, W), mem, lu, efeat, upd, tgt, loss_mask=mask)
    sel = mask.astype(bool)
    rb = oj.step(cfg, oj.pack(d, de, W), mem, lu, efeat, upd, tuple(a[sel] for a in tgt))
    assert abs(ra.loss - rb.loss) < 1e-14 and np.abs(ra.grads - rb.grads).max() < 1e-14
    # no update events: the table is untouched and the update cell and the time encoder get no gradient
    z = np.zeros(0, np.int64)
    rn = oj.step(cfg, oj.pack(d, de, W), mem, lu, efeat, (z, z, np.zeros(0), z, None), tgt)
    lay = oj.param_layout(d, de)
    assert np.array_equal(rn.memory_post, mem) and not rn.grads[:lay["proj_w"]].any() and rn.grads[lay["proj_w"]:].any()
    # with no drift parameters the embedding is the memory row itself
    Wz = dict(W, proj_w=np.zeros(d), proj_b=np.zeros(d))
    rz = oj.step(cfg, oj.pack(d, de, Wz), mem, lu, efeat, upd, tgt)
    nodes = np.concatenate(tgt[:3])
    assert np.array_equal(rz.h, rz.memory_post[nodes])


def test_backward_by_central_differences():
    rng = np.random.default_rng(5)
    cfg = _cfg(N=24, d=8, de=4)
    d, de = cfg.d, cfg.d_e
    efeat, mem, lu, upd, tgt = _case(rng, cfg, n_u=40, nq=16)
    W = _weights(rng, d, de)
    W["time_w"] = rng.uniform(0.05, 0.5, d)
    W["time_b"] = rng.uniform(-1, 1, d)
    p = oj.pack(d, de, W)
    mask = (rng.uniform(size=16) < 0.8).astype(np.uint8)
    base = oj.step(cfg, p, mem, lu, efeat, upd, tgt, loss_mask=mask)
    lay, sh = oj.param_layout(d, de), oj.param_shapes(d, de)
    eps = 1e-6
    for name in oj.PARAM_NAMES:
        n = int(np.prod(sh[name]))
        g = base.grads[lay[name]:lay[name] + n]
        assert np.abs(g).max() > 0, name                                           # every tensor takes part
        for j in rng.choice(n, size=min(n, 6), replace=False):
            pp, pm = p.copy(), p.copy()
            pp[lay[name] + j] += eps
            pm[lay[name] + j] -= eps
            fd = (oj.step(cfg, pp, mem, lu, efeat, upd, tgt, loss_mask=mask).loss -
                  oj.step(cfg, pm, mem, lu, efeat, upd, tgt, loss_mask=mask).loss) / (2 * eps)
            assert abs(fd - g[j]) <= 1e-6 * max(1.0, abs(g[j])) + 2e-8, (name, j, fd, g[j])
    assert abs(base.gradnorm - np.linalg.norm(base.grads)) < 1e-15
