"""TEST INFRASTRUCTURE -- ctypes front end of the CPU oracle (tgnn_oracle.cpp).

Only tests, the smoke check and the benchmark's cpu-baseline leg may import
this module; the product path never does.  It compiles the C++ file with g++
on first use and exposes each oracle routine on numpy arrays, plus
`OracleState.step`, which sequences one training step in the order of the
paper's Algorithm 2 (prune -> execute -> masked loss -> backprop and gradient
norm -> parameter update).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tgnn_oracle.cpp")
_LIB = os.path.join(_HERE, "libtgnn_oracle.so")

PARAM_NAMES = ("time_w", "time_b", "gru_w_i", "gru_w_h", "gru_b_i", "gru_b_h", "w_q", "b_q", "w_k", "w_v",
               "b_k", "b_v", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2")


class OrcConfig(C.Structure):
    _fields_ = [("num_nodes", C.c_int64), ("d", C.c_int32), ("d_e", C.c_int32), ("k", C.c_int32),
                ("heads", C.c_int32), ("feat_bf16", C.c_int32), ("phi_f32", C.c_int32),
                ("round_state_f32", C.c_int32), ("reserved", C.c_int32),
                ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double)]


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_param_count.restype = C.c_int64
        _lib.orc_mix64.restype = C.c_uint64
        _lib.orc_mix64.argtypes = [C.c_uint64]
        _lib.orc_hash32.restype = C.c_uint32
        _lib.orc_hash32.argtypes = [C.c_uint64, C.c_int64, C.c_int32]
    return _lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def make_config(num_nodes, d, d_e, k, heads, feat_bf16=False, phi_f32=True, round_state_f32=True,
                lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8) -> OrcConfig:
    assert d % heads == 0 and k <= 64
    return OrcConfig(num_nodes, d, d_e, k, heads, int(feat_bf16), int(phi_f32), int(round_state_f32), 0,
                     lr, beta1, beta2, eps)


def param_layout(cfg: OrcConfig) -> Dict[str, int]:
    out = np.zeros(19, dtype=np.int64)
    lib().orc_param_layout(C.byref(cfg), _p(out))
    lay = {n: int(out[i]) for i, n in enumerate(PARAM_NAMES)}
    lay["total"] = int(out[18])
    return lay


def pack_params(cfg: OrcConfig, weights: Dict[str, np.ndarray]) -> np.ndarray:
    lay = param_layout(cfg)
    flat = np.zeros(lay["total"], dtype=np.float64)
    for n in PARAM_NAMES:
        w = np.asarray(weights[n], dtype=np.float64).ravel()
        flat[lay[n]:lay[n] + w.size] = w
    return flat


def unpack_params(cfg: OrcConfig, flat: np.ndarray, shapes: Dict[str, tuple]) -> Dict[str, np.ndarray]:
    lay = param_layout(cfg)
    return {n: flat[lay[n]:lay[n] + int(np.prod(shapes[n]))].reshape(shapes[n]) for n in PARAM_NAMES}


def mix64(z: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(z)))


def hash32(seed: int, batch_idx: int, eid: int) -> int:
    return int(lib().orc_hash32(C.c_uint64(seed), C.c_int64(batch_idx), C.c_int32(eid)))


def prune_mask(num_nodes, src, dst, eid, is_aux, force_heavy=-1, drop_q32=1 << 31, seed=0, batch_idx=0):
    src, dst, eid, is_aux = _i32(src), _i32(dst), _i32(eid), _u8(is_aux)
    n = len(src)
    keep = np.zeros(n, dtype=np.uint8)
    heavy = np.zeros(1, dtype=np.int32)
    lib().orc_prune_mask(C.c_int64(num_nodes), _p(src), _p(dst), _p(eid), _p(is_aux), C.c_int(n),
                         C.c_int(force_heavy), C.c_uint32(drop_q32), C.c_uint64(seed), C.c_int64(batch_idx),
                         _p(keep), _p(heavy))
    return keep, int(heavy[0])


def sample_recent(indptr, nbr, eid, ts, nodes, times, k):
    nodes, times = _i32(nodes), _f64(times)
    n = len(nodes)
    nbr_o = np.zeros((n, k), np.int32)
    eid_o = np.zeros((n, k), np.int32)
    ts_o = np.zeros((n, k), np.float64)
    cnt_o = np.zeros(n, np.int32)
    lib().orc_sample_recent(_p(np.ascontiguousarray(indptr, np.int64)), _p(_i32(nbr)), _p(_i32(eid)), _p(_f64(ts)),
                            _p(nodes), _p(times), C.c_int(n), C.c_int(k), _p(nbr_o), _p(eid_o), _p(ts_o), _p(cnt_o))
    return nbr_o, eid_o, ts_o, cnt_o


def time_encode(cfg: OrcConfig, w, b, dt):
    w, b, dt = _f64(w), _f64(b), _f64(dt)
    out = np.zeros((len(dt), cfg.d), np.float64)
    lib().orc_time_encode(C.byref(cfg), _p(w), _p(b), _p(dt), C.c_int(len(dt)), _p(out))
    return out


def _feat(cfg: OrcConfig, efeat):
    if efeat is None:
        return np.zeros((1, max(cfg.d_e, 1)), np.uint16 if cfg.feat_bf16 else np.float32)
    want = np.uint16 if cfg.feat_bf16 else np.float32
    assert efeat.dtype == want, (efeat.dtype, want)
    return np.ascontiguousarray(efeat)


def build_messages(cfg, params, memory, last_update, efeat, src, dst, t, eid, keep=None):
    src, dst, t, eid = _i32(src), _i32(dst), _f64(t), _i32(eid)
    n = len(src)
    d_msg = 3 * cfg.d + cfg.d_e
    msg = np.zeros((2 * n, d_msg), np.float64)
    node = np.zeros(2 * n, np.int32)
    ef = _feat(cfg, efeat)
    kp = _u8(keep) if keep is not None else None
    lib().orc_build_messages(C.byref(cfg), _p(_f64(params)), _p(_f64(memory)), _p(_f64(last_update)), _p(ef),
                             _p(src), _p(dst), _p(t), _p(eid), _p(kp), C.c_int(n), _p(msg), _p(node))
    return msg, node


def reduce_latest(msg_node, t, eid, num_nodes):
    msg_node, t, eid = _i32(msg_node), _f64(t), _i32(eid)
    n_msg = len(msg_node)
    uniq = np.zeros(max(n_msg, 1), np.int32)
    win = np.zeros(max(n_msg, 1), np.int32)
    nu = np.zeros(1, np.int32)
    lib().orc_reduce_latest(_p(msg_node), _p(t), _p(eid), C.c_int(n_msg), C.c_int64(num_nodes), _p(uniq), _p(win), _p(nu))
    return uniq[:nu[0]].copy(), win[:nu[0]].copy()


def memory_update(cfg, params, msg, t, uniq, winner, memory, last_update):
    """Returns updated copies (memory [N,d] float64, last_update [N])."""
    mem = _f64(memory).copy()
    lu = _f64(last_update).copy()
    uniq, winner = _i32(uniq), _i32(winner)
    lib().orc_memory_update(C.byref(cfg), _p(_f64(params)), _p(_f64(msg)), _p(_f64(t)), _p(uniq), _p(winner),
                            C.c_int(len(uniq)), _p(mem), _p(lu))
    return mem, lu


def embed(cfg, params, memory, efeat, nodes, times, nbr, eid, ts, cnt):
    nodes, times = _i32(nodes), _f64(times)
    n = len(nodes)
    h = np.zeros((n, cfg.d), np.float64)
    lib().orc_embed(C.byref(cfg), _p(_f64(params)), _p(_f64(memory)), _p(_feat(cfg, efeat)), _p(nodes), _p(times),
                    C.c_int(n), _p(_i32(nbr)), _p(_i32(eid)), _p(_f64(ts)), _p(_i32(cnt)), _p(h))
    return h


@dataclass
class StepResult:
    loss: float
    gradnorm: float
    grads: Optional[np.ndarray]
    memory_post: np.ndarray
    last_update_post: np.ndarray
    h: np.ndarray
    uniq: np.ndarray
    winner: np.ndarray
    gate_overrides: tuple = (0, 0)   # units whose ReLU branch a hint decided against the fp64 sign (output layer, head)


def loss_and_grads(cfg, params, memory, last_update, efeat, upd, roots, n_q, loss_mask, want_grads=True,
                   h_gate=None, hid_gate=None, gate_eps=0.0) -> StepResult:
    """upd = (src, dst, t, eid, keep|None) of the update events; roots = (nodes, times, nbr, eid, ts, cnt).
    h_gate / hid_gate: ReLU branch decisions of a lower-precision run, used only for units whose
    pre-activation lies within gate_eps * max|pre-activation| of zero (either branch is valid there)."""
    u_src, u_dst, u_t, u_eid = _i32(upd[0]), _i32(upd[1]), _f64(upd[2]), _i32(upd[3])
    u_keep = _u8(upd[4]) if upd[4] is not None else None
    n_u = len(u_src)
    r_node, r_time = _i32(roots[0]), _f64(roots[1])
    nb_node, nb_eid, nb_ts, nb_cnt = _i32(roots[2]), _i32(roots[3]), _f64(roots[4]), _i32(roots[5])
    n_r = len(r_node)
    N, d = cfg.num_nodes, cfg.d
    P = int(lib().orc_param_count(C.byref(cfg)))
    loss = np.zeros(1)
    gn = np.zeros(1)
    grads = np.zeros(P) if want_grads else None
    mem_post = np.zeros((N, d))
    lu_post = np.zeros(N)
    h = np.zeros((n_r, d))
    uniq = np.zeros(max(2 * n_u, 1), np.int32)
    win = np.zeros(max(2 * n_u, 1), np.int32)
    nu = np.zeros(1, np.int32)
    lm = _u8(loss_mask) if loss_mask is not None else None
    lib().orc_loss_and_grads(C.byref(cfg), _p(_f64(params)), _p(_f64(memory)), _p(_f64(last_update)),
                             _p(_feat(cfg, efeat)), _p(u_src), _p(u_dst), _p(u_t), _p(u_eid), _p(u_keep), C.c_int(n_u),
                             _p(r_node), _p(r_time), C.c_int(n_r), _p(nb_node), _p(nb_eid), _p(nb_ts), _p(nb_cnt),
                             C.c_int(n_q), _p(lm), _p(_u8(h_gate) if h_gate is not None else None),
                             _p(_u8(hid_gate) if hid_gate is not None else None), C.c_double(gate_eps),
                             C.c_int(int(want_grads)), _p(loss), _p(grads), _p(gn),
                             _p(mem_post), _p(lu_post), _p(h), _p(uniq), _p(win), _p(nu))
    ov = np.zeros(2, np.int64)
    lib().orc_last_gate_overrides(_p(ov))
    return StepResult(float(loss[0]), float(gn[0]), grads, mem_post, lu_post, h, uniq[:nu[0]].copy(), win[:nu[0]].copy(),
                      (int(ov[0]), int(ov[1])))


def adam(cfg, grads, params, m, v, step):
    """Returns updated copies (params, m, v, step)."""
    p, m2, v2 = _f64(params).copy(), _f64(m).copy(), _f64(v).copy()
    st = np.array([step], dtype=np.int64)
    lib().orc_adam(C.byref(cfg), C.c_int64(len(p)), _p(_f64(grads)), _p(p), _p(m2), _p(v2), _p(st))
    return p, m2, v2, int(st[0])


class OracleState:
    """Model state plus `step`, one chronological training step (lag-one order:
    the previous kept mixed batch updates memory, then the current batch's
    target events are embedded and scored)."""

    def __init__(self, cfg: OrcConfig, params: np.ndarray):
        self.cfg = cfg
        N, d = cfg.num_nodes, cfg.d
        self.memory = np.zeros((N, d), np.float64)
        self.last_update = np.zeros(N, np.float64)
        self.params = _f64(params).copy()
        self.adam_m = np.zeros_like(self.params)
        self.adam_v = np.zeros_like(self.params)
        self.step_count = 0

    def step(self, graph, efeat, upd, tgt_src, tgt_dst, tgt_neg, tgt_t, loss_mask=None, apply_adam=True) -> StepResult:
        """graph = (indptr, nbr, eid, ts); upd = previous kept batch (src,dst,t,eid,keep|None) or None."""
        cfg = self.cfg
        n_q = len(tgt_src)
        nodes = np.concatenate([_i32(tgt_src), _i32(tgt_dst), _i32(tgt_neg)])
        times = np.concatenate([_f64(tgt_t)] * 3)
        nb, ne, nt, nc = sample_recent(*graph, nodes, times, cfg.k)
        if upd is None:
            z = np.zeros(0, np.int32)
            upd = (z, z, np.zeros(0), z, None)
        res = loss_and_grads(cfg, self.params, self.memory, self.last_update, efeat, upd,
                             (nodes, times, nb, ne, nt, nc), n_q, loss_mask, want_grads=True)
        self.memory, self.last_update = res.memory_post, res.last_update_post
        if apply_adam:
            self.params, self.adam_m, self.adam_v, self.step_count = adam(
                cfg, res.grads, self.params, self.adam_m, self.adam_v, self.step_count)
        return res
