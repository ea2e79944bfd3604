"""Oracle for the JODIE-style variant of the training step (the paper's second model).

TEST INFRASTRUCTURE: only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module.  It shares no code with the library.

The paper names JODIE only as a memory-based model whose user and item states are
updated recurrently along the interactions (experimental setup, "Models"); like the
attention model, its internals are the textbook form, here in the memory-module
framing of the work the paper builds on:

  messages     identical to the attention model: [m_self || m_other || x || Phi(t - last_update[self])],
               latest message per node wins                                            (Eq. 1)
  update       plain recurrent cell  m' = tanh(W_i msg + b_i + W_h m + b_h)           (Eq. 2)
  embedding    time projection       h(n, t) = m_n * (1 + dt * w_p + b_p),  dt = fp32(t - last_update[n])
               on the post-update table; no neighbor sampling, no attention
  head, loss   the same two-layer link-prediction head and masked loss                 (Eq. 13)
  backward     exact gradient; as in the attention model only the rows written in this step
               depend on the update cell's parameters and, through Phi, on (w, b)
  optimiser    Adam (the attention model's oracle routine is reused by the tests)

Plain numpy in fp64: one matrix product per projection, elementwise formulas written out.
fp32 by definition, as in the attention model's oracle: the argument of Phi and dt of the
projection (when cfg.phi_f32), and the memory rows written back (when cfg.round_state_f32).
Steps (0)-(3) are the attention model's: the latest-message reduction is the pinned routine of
oracle.py, called as a library step.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

from . import oracle as orc

PARAM_NAMES = ("time_w", "time_b", "rnn_w_i", "rnn_w_h", "rnn_b_i", "rnn_b_h", "proj_w", "proj_b", "w_1", "b_1", "w_2", "b_2")


def param_shapes(d: int, d_e: int) -> Dict[str, tuple]:
    dmsg = 3 * d + d_e
    return {"time_w": (d,), "time_b": (d,), "rnn_w_i": (d, dmsg), "rnn_w_h": (d, d), "rnn_b_i": (d,), "rnn_b_h": (d,),
            "proj_w": (d,), "proj_b": (d,), "w_1": (d, 2 * d), "b_1": (d,), "w_2": (d,), "b_2": (1,)}


def param_layout(d: int, d_e: int) -> Dict[str, int]:
    off, o = {}, 0
    for n, s in param_shapes(d, d_e).items():
        off[n] = o
        o += int(np.prod(s))
    off["total"] = o
    return off


def pack(d: int, d_e: int, weights: Dict[str, np.ndarray]) -> np.ndarray:
    lay = param_layout(d, d_e)
    flat = np.zeros(lay["total"], np.float64)
    for n in PARAM_NAMES:
        w = np.asarray(weights[n], np.float64).ravel()
        flat[lay[n]:lay[n] + w.size] = w
    return flat


def unpack(d: int, d_e: int, flat: np.ndarray) -> Dict[str, np.ndarray]:
    lay, sh = param_layout(d, d_e), param_shapes(d, d_e)
    return {n: np.asarray(flat[lay[n]:lay[n] + int(np.prod(sh[n]))], np.float64).reshape(sh[n]) for n in PARAM_NAMES}


def _f32(x):
    return np.asarray(x, np.float64).astype(np.float32).astype(np.float64)


def time_args(phi_f32: bool, w: np.ndarray, b: np.ndarray, dt: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Argument of Phi and the dt that multiplies w in it.  fp32 mode: dt rounded to fp32 first, then one
    fused multiply-add rounded to fp32 (formed in extended precision, rounded once)."""
    dt = np.asarray(dt, np.float64)
    if not phi_f32:
        return dt[:, None] * w[None, :] + b[None, :], dt
    dtf = _f32(dt)
    ext = np.longdouble(dtf)[:, None] * np.longdouble(_f32(w))[None, :] + np.longdouble(_f32(b))[None, :]
    return ext.astype(np.float32).astype(np.float64), dtf


def decode_features(efeat: Optional[np.ndarray], eid: np.ndarray, d_e: int) -> np.ndarray:
    if d_e == 0 or efeat is None:
        return np.zeros((len(eid), d_e), np.float64)
    rows = efeat[np.asarray(eid, np.int64)]
    if rows.dtype == np.uint16:                                    # bf16 bit patterns
        rows = (rows.astype(np.uint32) << 16).view(np.float32)
    return rows.astype(np.float64)


def rnn_rows(W: Dict[str, np.ndarray], X: np.ndarray, H: np.ndarray) -> np.ndarray:
    """m' = tanh(W_i x + b_i + W_h h + b_h), row by row."""
    return np.tanh(X @ W["rnn_w_i"].T + W["rnn_b_i"] + H @ W["rnn_w_h"].T + W["rnn_b_h"])


def time_projection(m: np.ndarray, dt: np.ndarray, w_p: np.ndarray, b_p: np.ndarray) -> np.ndarray:
    """h = m * (1 + dt w_p + b_p)."""
    return m * (1.0 + dt[:, None] * w_p[None, :] + b_p[None, :])


def winner_messages(cfg: orc.OrcConfig, W: Dict[str, np.ndarray], mem: np.ndarray, lu: np.ndarray, efeat, upd):
    """Steps (2)-(3): the message row of the latest event of every touched node.

    Returns (uniq, winner, X [U, 3d + d_e], H [U, d] = the nodes' own rows, Phi's arguments [U, d], the dt inside
    them [U], the winners' timestamps [U])."""
    d, de, N = cfg.d, cfg.d_e, cfg.num_nodes
    u_src, u_dst, u_t, u_eid, keep = upd
    u_src, u_dst, u_eid = np.asarray(u_src, np.int64), np.asarray(u_dst, np.int64), np.asarray(u_eid, np.int64)
    u_t = np.asarray(u_t, np.float64)
    n_u = len(u_src)
    if n_u == 0:
        z = np.zeros(0, np.int32)
        return z, z, np.zeros((0, 3 * d + de)), np.zeros((0, d)), np.zeros((0, d)), np.zeros(0), np.zeros(0)
    kept = np.ones(n_u, bool) if keep is None else np.asarray(keep).astype(bool)
    msg_node = np.full(2 * n_u, -1, np.int32)
    msg_node[0::2] = np.where(kept, u_src, -1)       # message 2i -> source (role 0), 2i+1 -> destination (role 1)
    msg_node[1::2] = np.where(kept, u_dst, -1)
    uniq, winner = orc.reduce_latest(msg_node, u_t, u_eid.astype(np.int32), N)
    ev, role = winner >> 1, winner & 1
    self_n = np.where(role == 0, u_src[ev], u_dst[ev])
    other_n = np.where(role == 0, u_dst[ev], u_src[ev])
    assert np.array_equal(self_n, uniq)
    x_arg, x_dt = time_args(bool(cfg.phi_f32), W["time_w"], W["time_b"], u_t[ev] - lu[self_n])
    X = np.concatenate([mem[self_n], mem[other_n], decode_features(efeat, u_eid[ev], de), np.cos(x_arg)], axis=1)
    return uniq, winner, X, mem[self_n], x_arg, x_dt, u_t[ev]


@dataclass
class JodieResult:
    loss: float
    gradnorm: float
    grads: np.ndarray            # flat, PARAM_NAMES order
    memory_post: np.ndarray
    last_update_post: np.ndarray
    h: np.ndarray
    uniq: np.ndarray
    winner: np.ndarray


def step(cfg: orc.OrcConfig, params: np.ndarray, memory: np.ndarray, last_update: np.ndarray, efeat,
         upd, targets, loss_mask=None, hid_gate: Optional[np.ndarray] = None, gate_eps: float = 0.0) -> JodieResult:
    """Forward and exact backward of one step from the pre-step state.

    upd = (src, dst, t, eid, keep or None): the previous kept mixed batch; targets = (src, dst, neg, t)."""
    d, de, N = cfg.d, cfg.d_e, cfg.num_nodes
    W = unpack(d, de, params)
    mem = np.asarray(memory, np.float64)
    lu = np.asarray(last_update, np.float64)
    phi32 = bool(cfg.phi_f32)

    # ---- steps (2)-(4): messages on the pre-step table, latest per node, recurrent cell, write-back ----
    uniq, winner, X, H, x_arg, x_dt, win_t = winner_messages(cfg, W, mem, lu, efeat, upd)
    U = len(uniq)
    m_new = rnn_rows(W, X, H)
    mem_post, lu_post = mem.copy(), lu.copy()
    mem_post[uniq] = _f32(m_new) if cfg.round_state_f32 else m_new
    lu_post[uniq] = win_t
    slot = np.full(N, -1, np.int64)
    slot[uniq] = np.arange(U)

    # ---- step (5): time-projected embedding of the roots on the post-update table ----
    t_src, t_dst, t_neg, t_t = targets
    nq = len(t_src)
    nodes = np.concatenate([t_src, t_dst, t_neg]).astype(np.int64)
    times = np.concatenate([t_t] * 3).astype(np.float64)
    r_dt = times - lu_post[nodes]
    r_dt = _f32(r_dt) if phi32 else r_dt
    m_r = mem_post[nodes]
    h = time_projection(m_r, r_dt, W["proj_w"], W["proj_b"])

    # ---- step (6): head and masked loss (Eq. 13) ----
    M = np.ones(nq) if loss_mask is None else (np.asarray(loss_mask) != 0).astype(np.float64)
    msum = M.sum()
    cat = np.concatenate([np.concatenate([h[:nq], h[nq:2 * nq]], axis=1),          # positive pairs
                          np.concatenate([h[:nq], h[2 * nq:]], axis=1)], axis=0)   # negative pairs
    pre1 = cat @ W["w_1"].T + W["b_1"]
    gate = pre1 > 0.0
    if hid_gate is not None and gate_eps > 0.0 and pre1.size:
        near = np.abs(pre1) <= gate_eps * np.abs(pre1).max()
        gate = np.where(near, np.asarray(hid_gate).astype(bool), gate)
    hid = np.where(gate, pre1, 0.0)
    score = hid @ W["w_2"] + W["b_2"][0]
    sp, sn = score[:nq], score[nq:]
    softplus = lambda z: np.logaddexp(0.0, z)
    wj = M / msum if msum > 0 else np.zeros(nq)
    loss = float(np.sum(wj * (softplus(-sp) + softplus(sn))))

    # ---- backward ----
    G = {n: np.zeros_like(W[n]) for n in PARAM_NAMES}
    sig = lambda z: 1.0 / (1.0 + np.exp(-z))
    dscore = np.concatenate([-wj * sig(-sp), wj * sig(sn)])
    G["b_2"][0] = dscore.sum()
    G["w_2"] = hid.T @ dscore
    dpre1 = np.where(gate, dscore[:, None] * W["w_2"][None, :], 0.0)
    G["w_1"] = dpre1.T @ cat
    G["b_1"] = dpre1.sum(axis=0)
    dcat = dpre1 @ W["w_1"]
    dh = np.zeros_like(h)
    dh[:nq] = dcat[:nq, :d] + dcat[nq:, :d]
    dh[nq:2 * nq] = dcat[:nq, d:]
    dh[2 * nq:] = dcat[nq:, d:]
    G["proj_w"] = np.sum(dh * m_r * r_dt[:, None], axis=0)
    G["proj_b"] = np.sum(dh * m_r, axis=0)
    dm_r = dh * (1.0 + r_dt[:, None] * W["proj_w"][None, :] + W["proj_b"][None, :])
    dM = np.zeros((U, d))
    touched = slot[nodes] >= 0                      # only rows written in this step carry gradient further
    np.add.at(dM, slot[nodes][touched], dm_r[touched])
    dpre = dM * (1.0 - m_new * m_new)
    G["rnn_w_i"] = dpre.T @ X
    G["rnn_w_h"] = dpre.T @ H
    G["rnn_b_i"] = dpre.sum(axis=0)
    G["rnn_b_h"] = dpre.sum(axis=0)
    dphi = dpre @ W["rnn_w_i"][:, 2 * d + de:]     # gradient w.r.t. the message's time encoding
    t_term = -np.sin(x_arg) * dphi
    G["time_w"] = np.sum(t_term * x_dt[:, None], axis=0) if U else np.zeros(d)
    G["time_b"] = t_term.sum(axis=0) if U else np.zeros(d)
    grads = pack(d, de, G)
    return JodieResult(loss, float(np.sqrt(np.sum(grads * grads))), grads, mem_post, lu_post, h, uniq, winner)
