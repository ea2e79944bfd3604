"""Thin ctypes binding of libtgnn_b200.so: same names as the C ABI, argument
marshalling only.  torch is used for device memory and streams; every step of
the path runs in the library's CUDA kernels.  There is no CPU fallback: loading
fails loudly when the shared library is missing."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtgnn_b200.so")

TGNN_OK, TGNN_EINVAL, TGNN_ESHAPE, TGNN_ECAPACITY, TGNN_ESTATE, TGNN_ECUDA, TGNN_ETIMEOUT, TGNN_EBOUNDS = (
    0, -1, -2, -3, -4, -5, -6, -7)
TGNN_F32, TGNN_BF16 = 0, 1
TGNN_MATH_FP32, TGNN_MATH_TF32, TGNN_MATH_TF32_FAST, TGNN_MATH_F16X3 = 0, 1, 2, 3

PARAM_NAMES = ("time_w", "time_b", "gru_w_i", "gru_w_h", "gru_b_i", "gru_b_h", "w_q", "b_q", "w_k", "w_v",
               "b_k", "b_v", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2")
# the time-projection model: plain recurrent cell in the update-cell slots, no attention block, w_p | b_p
PARAM_NAMES_JODIE = ("time_w", "time_b", "rnn_w_i", "rnn_w_h", "rnn_b_i", "rnn_b_h", "proj_w", "proj_b",
                     "w_1", "b_1", "w_2", "b_2")
_JODIE_SLOT = {"time_w": 0, "time_b": 1, "rnn_w_i": 2, "rnn_w_h": 3, "rnn_b_i": 4, "rnn_b_h": 5, "proj_w": 18, "proj_b": 19,
               "w_1": 14, "b_1": 15, "w_2": 16, "b_2": 17}
TGNN_MODEL_TGN, TGNN_MODEL_JODIE = 0, 1

EXPORTS = ("tgnn_create", "tgnn_destroy", "tgnn_last_error", "tgnn_param_count", "tgnn_param_layout",
           "tgnn_set_graph", "tgnn_set_edge_features", "tgnn_set_state", "tgnn_prune_mask", "tgnn_sample_recent",
           "tgnn_build_messages", "tgnn_reduce_latest", "tgnn_memory_update", "tgnn_embed", "tgnn_backward_step",
           "tgnn_train_step", "tgnn_train_step_host", "tgnn_debug_get_grads", "tgnn_status", "tgnn_kernel_launches", "tgnn_profile_begin",
           "tgnn_profile_report", "tgnn_reduce_latest_static", "tgnn_debug_gemm", "tgnn_debug_get_gates", "tgnn_set_graph_replay", "tgnn_profile_timeline", "tgnn_step_mixed_host",
           "tgnn_controller_create", "tgnn_controller_destroy", "tgnn_controller_begin_batch",
           "tgnn_controller_end_batch", "tgnn_controller_state", "tgnn_backward_scan_scratch", "tgnn_backward_scan",
           "tgnn_build_mixed", "tgnn_set_grad_sync", "tgnn_grad_buffer", "tgnn_apply_gradient", "tgnn_refresh_plan",
           "tgnn_pack_rows", "tgnn_unpack_rows", "tgnn_debug_get_embeddings", "tgnn_debug_gemm_split",
           "tgnn_clear_status")
TGNN_STATIC_MAX_NODES = 65536


class TgnnConfig(C.Structure):
    _fields_ = [("num_nodes", C.c_int64), ("d", C.c_int32), ("d_e", C.c_int32), ("k", C.c_int32),
                ("heads", C.c_int32), ("feat_dtype", C.c_int32), ("max_events", C.c_int32),
                ("max_roots", C.c_int32), ("math_mode", C.c_int32),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("model", C.c_int32), ("embed_aux", C.c_int32)]


class TgnnError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"tgnn error {code}: {msg}")
        self.code = code


_lib = None


def load_library():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_16305_b200.build` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        vp, i32, i64, u32, u64 = C.c_void_p, C.c_int, C.c_int64, C.c_uint32, C.c_uint64
        lib.tgnn_create.argtypes = [C.POINTER(TgnnConfig), C.POINTER(vp)]
        lib.tgnn_destroy.argtypes = [vp]
        lib.tgnn_last_error.argtypes = [vp]
        lib.tgnn_last_error.restype = C.c_char_p
        lib.tgnn_param_count.argtypes = [C.POINTER(TgnnConfig)]
        lib.tgnn_param_count.restype = i64
        lib.tgnn_param_layout.argtypes = [C.POINTER(TgnnConfig), vp]
        lib.tgnn_set_graph.argtypes = [vp, vp, vp, vp, vp, i64]
        lib.tgnn_set_edge_features.argtypes = [vp, vp, i32, i64, i32]
        lib.tgnn_set_state.argtypes = [vp] * 7
        lib.tgnn_prune_mask.argtypes = [vp, vp, vp, vp, vp, i32, i32, u32, u64, i64, vp, vp, vp]
        lib.tgnn_sample_recent.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
        lib.tgnn_build_messages.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        lib.tgnn_reduce_latest.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp]
        lib.tgnn_memory_update.argtypes = [vp, vp, vp, vp, vp, vp]
        lib.tgnn_embed.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        lib.tgnn_backward_step.argtypes = [vp, i32, vp, vp, vp, vp]
        lib.tgnn_train_step.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp]
        lib.tgnn_train_step_host.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp]
        lib.tgnn_debug_get_grads.argtypes = [vp, vp, vp]
        lib.tgnn_status.argtypes = [vp, vp, vp]
        lib.tgnn_kernel_launches.argtypes = [vp]
        lib.tgnn_kernel_launches.restype = i64
        lib.tgnn_profile_begin.argtypes = [vp]
        lib.tgnn_profile_report.argtypes = [vp, vp, i64]
        lib.tgnn_profile_timeline.argtypes = [vp, vp, i64]
        lib.tgnn_debug_gemm.argtypes = [vp, vp, i64, i64, vp, i64, i64, vp, i64, i32, i32, i32, vp, vp, vp, vp, i32, i32, i32, i32,
                                        vp]
        lib.tgnn_debug_get_gates.argtypes = [vp, vp, vp, vp]
        lib.tgnn_debug_get_embeddings.argtypes = [vp, vp, vp]
        lib.tgnn_clear_status.argtypes = [vp, vp]
        lib.tgnn_debug_gemm_split.argtypes = [vp, vp, i64, i64, vp, i64, i64, vp, i64, i32, i32, i32, vp, i32, i32, i32, vp, i64,
                                              i32, u32, vp]
        lib.tgnn_step_mixed_host.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, i32, u32, u64, i64, vp, vp, vp]
        lib.tgnn_set_graph_replay.argtypes = [vp, i32]
        lib.tgnn_reduce_latest_static.argtypes = [vp, vp, vp, i32, i64, vp, vp, vp, vp, vp, i32]
        f64 = C.c_double
        lib.tgnn_controller_create.argtypes = [f64, f64, f64, f64, i32, C.POINTER(vp)]
        lib.tgnn_controller_destroy.argtypes = [vp]
        lib.tgnn_controller_begin_batch.argtypes = [vp, i64, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
        lib.tgnn_controller_end_batch.argtypes = [vp, f64, f64]
        lib.tgnn_controller_state.argtypes = [vp, C.POINTER(f64)]
        lib.tgnn_backward_scan_scratch.argtypes = [i64, i32, i32, i64, i32]
        lib.tgnn_backward_scan_scratch.restype = i64
        lib.tgnn_backward_scan.argtypes = [vp, vp, i64, i32, i32, vp, i64, i32, vp, vp, vp, vp, vp, vp, vp, i64]
        lib.tgnn_build_mixed.argtypes = [vp, vp, vp, vp, i64, i32, vp, vp, vp, i64, i64] + [vp] * 11 + [vp, vp, i64]
        lib.tgnn_set_grad_sync.argtypes = [vp, i32]
        lib.tgnn_grad_buffer.argtypes = [vp, C.POINTER(vp), C.POINTER(i64)]
        lib.tgnn_apply_gradient.argtypes = [vp, C.c_float, vp, vp]
        lib.tgnn_refresh_plan.argtypes = [vp, vp, i64, i32, i32, i32, i64, vp, vp, vp, vp, vp, vp, vp, i64]
        lib.tgnn_pack_rows.argtypes = [vp, vp, i64, i32, vp, i32, vp, vp, vp, vp, i64]
        lib.tgnn_unpack_rows.argtypes = [vp, vp, i64, i32, vp, i32, vp, vp, vp, vp, i64]
        _lib = lib
    return _lib


_TORCH_DT = {"i32": torch.int32, "i64": torch.int64, "f32": torch.float32, "f64": torch.float64, "u8": torch.uint8,
             "bf16": torch.bfloat16}


def _dp(t: Optional[torch.Tensor], dt: str, name: str):
    """Device pointer of a contiguous CUDA tensor of the expected dtype (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda or t.dtype != _TORCH_DT[dt] or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dt}, got {t.dtype} on {t.device}")
    return t.data_ptr()


def _hp(t: Optional[torch.Tensor], dt: str, name: str):
    if t is None:
        return None
    if t.is_cuda or t.dtype != _TORCH_DT[dt] or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous host tensor of dtype {dt}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_config(num_nodes, d, d_e, k, heads, feat_dtype=TGNN_F32, max_events=1024, max_roots=3072,
                math_mode=TGNN_MATH_FP32, lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, model=TGNN_MODEL_TGN,
                embed_aux=0) -> TgnnConfig:
    return TgnnConfig(num_nodes, d, d_e, k, heads, feat_dtype, max_events, max_roots, math_mode, lr, beta1, beta2, eps,
                      model, int(embed_aux))


def param_names(cfg: TgnnConfig):
    """Names of the model's parameter tensors in memory order."""
    return PARAM_NAMES_JODIE if cfg.model == TGNN_MODEL_JODIE else PARAM_NAMES


def param_layout(cfg: TgnnConfig) -> Dict[str, int]:
    out = np.zeros(21, dtype=np.int64)
    rc = load_library().tgnn_param_layout(C.byref(cfg), out.ctypes.data)
    if rc != TGNN_OK:
        raise TgnnError(rc, "invalid configuration")
    if cfg.model == TGNN_MODEL_JODIE:
        lay = {n: int(out[_JODIE_SLOT[n]]) for n in PARAM_NAMES_JODIE}
    else:
        lay = {n: int(out[i]) for i, n in enumerate(PARAM_NAMES)}
    lay["total"] = int(out[20])
    return lay


def pack_params(cfg: TgnnConfig, weights: Dict[str, np.ndarray]) -> np.ndarray:
    lay = param_layout(cfg)
    flat = np.zeros(lay["total"], dtype=np.float32)
    for n in param_names(cfg):
        w = np.asarray(weights[n], dtype=np.float32).ravel()
        flat[lay[n]:lay[n] + w.size] = w
    return flat


def reduce_latest_static(msg_node, t, eid, num_nodes, uniq_out, winner_out, n_uniq_out) -> int:
    """tgnn_reduce_latest_static: step (3) for hosts that may not allocate device memory, so no
    context is involved -- the scratch tables are an array inside the library (at most
    TGNN_STATIC_MAX_NODES nodes).  Raises TgnnError with the library's message on failure.
    Calls share that array: do not let two of them overlap on one GPU."""
    err = C.create_string_buffer(512)
    rc = load_library().tgnn_reduce_latest_static(
        _dp(msg_node, "i32", "msg_node"), _dp(t, "f64", "t"), _dp(eid, "i32", "eid"), msg_node.numel(), num_nodes,
        _dp(uniq_out, "i32", "uniq_out"), _dp(winner_out, "i32", "winner_out"), _dp(n_uniq_out, "i32", "n_uniq_out"),
        _stream(), C.addressof(err), len(err))
    if rc != TGNN_OK:
        raise TgnnError(rc, err.value.decode())
    return rc


def backward_scan_scratch(num_events: int, batch: int, K: int, num_nodes: int, P: int) -> int:
    """int32 elements tgnn_backward_scan needs as scratch."""
    n = load_library().tgnn_backward_scan_scratch(num_events, batch, K, num_nodes, P)
    if n < 0:
        raise TgnnError(TGNN_EINVAL, "tgnn_backward_scan_scratch: size out of range")
    return n


def backward_scan(src, dst, batch: int, K: int, owner, P: int, role_out, n_sync_out, sync_out, scratch, status_out) -> int:
    """tgnn_backward_scan: Algorithm 1 for every worker and window (device tensors; sync_out may be None)."""
    err = C.create_string_buffer(512)
    rc = load_library().tgnn_backward_scan(
        _dp(src, "i32", "src"), _dp(dst, "i32", "dst"), src.numel(), batch, K, _dp(owner, "i32", "owner"), owner.numel(), P,
        _dp(role_out, "u8", "role_out"), _dp(n_sync_out, "i32", "n_sync_out"), _dp(sync_out, "u8", "sync_out"),
        _dp(scratch, "i32", "scratch"), _dp(status_out, "i32", "status_out"), _stream(), C.addressof(err), len(err))
    if rc != TGNN_OK:
        raise TgnnError(rc, err.value.decode())
    return rc


def build_mixed(src, dst, t, neg, batch: int, role, mb_off_out, tgt_off_out, mb, tgt, status_out) -> int:
    """tgnn_build_mixed: one worker's mixed batches (Eq. 5).  mb = (src, dst, t, eid, aux) output tensors,
    tgt = (src, dst, t, neg or None, eid) output tensors."""
    err = C.create_string_buffer(512)
    rc = load_library().tgnn_build_mixed(
        _dp(src, "i32", "src"), _dp(dst, "i32", "dst"), _dp(t, "f64", "t"), _dp(neg, "i32", "neg"), src.numel(), batch,
        _dp(role, "u8", "role"), _dp(mb_off_out, "i32", "mb_off_out"), _dp(tgt_off_out, "i32", "tgt_off_out"),
        mb[0].numel(), tgt[0].numel(),
        _dp(mb[0], "i32", "mb_src"), _dp(mb[1], "i32", "mb_dst"), _dp(mb[2], "f64", "mb_t"), _dp(mb[3], "i32", "mb_eid"),
        _dp(mb[4], "u8", "mb_aux"), _dp(tgt[0], "i32", "tgt_src"), _dp(tgt[1], "i32", "tgt_dst"), _dp(tgt[2], "f64", "tgt_t"),
        _dp(tgt[3], "i32", "tgt_neg"), _dp(tgt[4], "i32", "tgt_eid"), _dp(status_out, "i32", "status_out"),
        _stream(), C.addressof(err), len(err))
    if rc != TGNN_OK:
        raise TgnnError(rc, err.value.decode())
    return rc


def refresh_plan(sync, owner, P: int, Q: int, me: int, cap: int, recv_nodes, recv_off, send_nodes, send_off, status_out) -> int:
    """tgnn_refresh_plan: worker `me`'s receive and send lists for every window (device tensors)."""
    err = C.create_string_buffer(512)
    rc = load_library().tgnn_refresh_plan(
        _dp(sync, "u8", "sync"), _dp(owner, "i32", "owner"), owner.numel(), P, Q, me, cap,
        _dp(recv_nodes, "i32", "recv_nodes"), _dp(recv_off, "i32", "recv_off"), _dp(send_nodes, "i32", "send_nodes"),
        _dp(send_off, "i32", "send_off"), _dp(status_out, "i32", "status_out"), _stream(), C.addressof(err), len(err))
    if rc != TGNN_OK:
        raise TgnnError(rc, err.value.decode())
    return rc


def _rows(fn, memory, last_update, nodes, packed, status) -> int:
    err = C.create_string_buffer(512)
    n = 0 if nodes is None else nodes.numel()
    if n and packed.numel() < n * (memory.shape[1] + 2):
        raise TgnnError(TGNN_EINVAL, "packed buffer too small")
    rc = fn(_dp(memory, "f32", "memory"), _dp(last_update, "f64", "last_update"), memory.shape[0], memory.shape[1],
            _dp(nodes, "i32", "nodes"), n, _dp(packed, "f32", "packed"), _dp(status, "i32", "status"), _stream(),
            C.addressof(err), len(err))
    if rc != TGNN_OK:
        raise TgnnError(rc, err.value.decode())
    return rc


def pack_rows(memory, last_update, nodes, packed, status) -> int:
    """tgnn_pack_rows: packed[i] = (memory row, last-update time) of nodes[i], d + 2 floats per row."""
    return _rows(load_library().tgnn_pack_rows, memory, last_update, nodes, packed, status)


def unpack_rows(memory, last_update, nodes, packed, status) -> int:
    """tgnn_unpack_rows: the state of nodes[i] becomes packed[i]."""
    return _rows(load_library().tgnn_unpack_rows, memory, last_update, nodes, packed, status)


class Controller:
    """The adaptive runtime controller (host-side; mirrors the tgnn_controller_* entry points)."""

    def __init__(self, alpha: float, beta: float, tau_g: float, tau_c: float, K: int):
        self.lib = load_library()
        self.K = int(K)
        self._h = C.c_void_p()
        rc = self.lib.tgnn_controller_create(alpha, beta, tau_g, tau_c, K, C.byref(self._h))
        if rc != TGNN_OK:
            raise TgnnError(rc, "tgnn_controller_create: parameter out of range")

    def close(self):
        if self._h:
            self.lib.tgnn_controller_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def begin_batch(self, r: int):
        """(boundary, S_r or -1, H_r) for batch r."""
        b, s, h = C.c_int(), C.c_int(), C.c_int()
        rc = self.lib.tgnn_controller_begin_batch(self._h, r, C.byref(b), C.byref(s), C.byref(h))
        if rc != TGNN_OK:
            raise TgnnError(rc, "tgnn_controller_begin_batch: invalid argument")
        return b.value, s.value, h.value

    def end_batch(self, g_r: float, c_r: float):
        rc = self.lib.tgnn_controller_end_batch(self._h, g_r, c_r)
        if rc != TGNN_OK:
            raise TgnnError(rc, "tgnn_controller_end_batch: invalid argument")

    def state(self):
        out = (C.c_double * 4)()
        rc = self.lib.tgnn_controller_state(self._h, out)
        if rc != TGNN_OK:
            raise TgnnError(rc, "tgnn_controller_state: invalid argument")
        return tuple(out)


class Tgnn:
    """One library context.  Methods mirror the C entry points one to one."""

    def __init__(self, cfg: TgnnConfig):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.lib = load_library()
        self.cfg = cfg
        self._h = C.c_void_p()
        rc = self.lib.tgnn_create(C.byref(cfg), C.byref(self._h))
        if rc != TGNN_OK:
            raise TgnnError(rc, "tgnn_create failed (invalid configuration, not an sm_100 device, or out of memory)")
        self._keep = {}     # tensors the library borrows: keep them alive

    def close(self):
        if self._h:
            self.lib.tgnn_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc: int):
        if rc != TGNN_OK:
            raise TgnnError(rc, self.lib.tgnn_last_error(self._h).decode())

    def call_raw(self, name: str, *args) -> int:
        """Calls an entry point and returns its code without raising (error-path tests)."""
        return getattr(self.lib, name)(self._h, *args)

    def last_error(self) -> str:
        return self.lib.tgnn_last_error(self._h).decode()

    def kernel_launches(self) -> int:
        return int(self.lib.tgnn_kernel_launches(self._h))

    # ---- set-up ----
    def set_graph(self, indptr, nbr, eid, ts):
        self._keep["graph"] = (indptr, nbr, eid, ts)
        self._ck(self.lib.tgnn_set_graph(self._h, _dp(indptr, "i64", "indptr"), _dp(nbr, "i32", "nbr"),
                                         _dp(eid, "i32", "eid"), _dp(ts, "f64", "ts"), nbr.numel()))

    def set_edge_features(self, efeat: Optional[torch.Tensor], num_events: int):
        self._keep["efeat"] = efeat
        dt = "bf16" if self.cfg.feat_dtype == TGNN_BF16 else "f32"
        self._ck(self.lib.tgnn_set_edge_features(self._h, _dp(efeat, dt, "efeat") if self.cfg.d_e else None,
                                                 self.cfg.feat_dtype, num_events, self.cfg.d_e))

    def set_state(self, memory, last_update, params, adam_m, adam_v, step):
        self._keep["state"] = (memory, last_update, params, adam_m, adam_v, step)
        self._ck(self.lib.tgnn_set_state(self._h, _dp(memory, "f32", "memory"), _dp(last_update, "f64", "last_update"),
                                         _dp(params, "f32", "params"), _dp(adam_m, "f32", "adam_m"),
                                         _dp(adam_v, "f32", "adam_v"), _dp(step, "i64", "step")))

    # ---- the step ----
    def prune_mask(self, src, dst, eid, is_aux, keep_out, heavy_out, force_heavy=-1, drop_q32=1 << 31, seed=0,
                   batch_idx=0):
        self._ck(self.lib.tgnn_prune_mask(self._h, _dp(src, "i32", "src"), _dp(dst, "i32", "dst"), _dp(eid, "i32", "eid"),
                                          _dp(is_aux, "u8", "is_aux"), src.numel(), force_heavy, drop_q32, seed,
                                          batch_idx, _dp(keep_out, "u8", "keep_out"), _dp(heavy_out, "i32", "heavy_out"),
                                          _stream()))

    def sample_recent(self, nodes, times, nbr_out, eid_out, ts_out, cnt_out):
        self._ck(self.lib.tgnn_sample_recent(self._h, _dp(nodes, "i32", "nodes"), _dp(times, "f64", "times"),
                                             nodes.numel(), _dp(nbr_out, "i32", "nbr_out"), _dp(eid_out, "i32", "eid_out"),
                                             _dp(ts_out, "f64", "ts_out"), _dp(cnt_out, "i32", "cnt_out"), _stream()))

    def build_messages(self, src, dst, t, eid, keep, msg_out, msg_node_out):
        self._keep["upd"] = (src, dst, t, eid, keep)
        self._ck(self.lib.tgnn_build_messages(self._h, _dp(src, "i32", "src"), _dp(dst, "i32", "dst"), _dp(t, "f64", "t"),
                                              _dp(eid, "i32", "eid"), _dp(keep, "u8", "keep"), src.numel(),
                                              _dp(msg_out, "f32", "msg_out"), _dp(msg_node_out, "i32", "msg_node_out"),
                                              _stream()))

    def reduce_latest(self, msg_node, t, eid, uniq_out, winner_out, n_uniq_out):
        self._ck(self.lib.tgnn_reduce_latest(self._h, _dp(msg_node, "i32", "msg_node"), _dp(t, "f64", "t"),
                                             _dp(eid, "i32", "eid"), msg_node.numel(), _dp(uniq_out, "i32", "uniq_out"),
                                             _dp(winner_out, "i32", "winner_out"), _dp(n_uniq_out, "i32", "n_uniq_out"),
                                             _stream()))

    def memory_update(self, msg, uniq, winner, n_uniq):
        self._keep["upd_idx"] = (msg, uniq, winner, n_uniq)
        self._ck(self.lib.tgnn_memory_update(self._h, _dp(msg, "f32", "msg"), _dp(uniq, "i32", "uniq"),
                                             _dp(winner, "i32", "winner"), _dp(n_uniq, "i32", "n_uniq"), _stream()))

    def embed(self, nodes, times, nbr, eid, ts, cnt, h_out):
        self._keep["embed"] = (nodes, times, nbr, eid, ts, cnt, h_out)
        self._ck(self.lib.tgnn_embed(self._h, _dp(nodes, "i32", "nodes"), _dp(times, "f64", "times"), nodes.numel(),
                                     _dp(nbr, "i32", "nbr"), _dp(eid, "i32", "eid"), _dp(ts, "f64", "ts"),
                                     _dp(cnt, "i32", "cnt"), _dp(h_out, "f32", "h_out"), _stream()))

    def backward_step(self, n_q, loss_mask, loss_out, gradnorm_out):
        self._ck(self.lib.tgnn_backward_step(self._h, n_q, _dp(loss_mask, "u8", "loss_mask"),
                                             _dp(loss_out, "f32", "loss_out"), _dp(gradnorm_out, "f32", "gradnorm_out"),
                                             _stream()))

    def train_step(self, u_src, u_dst, u_t, u_eid, u_keep, q_src, q_dst, q_neg, q_t, loss_mask, loss_out, gradnorm_out):
        n_u = 0 if u_src is None else u_src.numel()
        self._ck(self.lib.tgnn_train_step(self._h, _dp(u_src, "i32", "u_src"), _dp(u_dst, "i32", "u_dst"),
                                          _dp(u_t, "f64", "u_t"), _dp(u_eid, "i32", "u_eid"), _dp(u_keep, "u8", "u_keep"),
                                          n_u, _dp(q_src, "i32", "q_src"), _dp(q_dst, "i32", "q_dst"),
                                          _dp(q_neg, "i32", "q_neg"), _dp(q_t, "f64", "q_t"), q_src.numel(),
                                          _dp(loss_mask, "u8", "loss_mask"), _dp(loss_out, "f32", "loss_out"),
                                          _dp(gradnorm_out, "f32", "gradnorm_out"), _stream()))

    def train_step_host(self, u_src, u_dst, u_t, u_eid, u_keep, q_src, q_dst, q_neg, q_t, loss_mask, loss_host,
                        gradnorm_host):
        n_u = 0 if u_src is None else u_src.numel()
        self._ck(self.lib.tgnn_train_step_host(self._h, _hp(u_src, "i32", "u_src"), _hp(u_dst, "i32", "u_dst"),
                                               _hp(u_t, "f64", "u_t"), _hp(u_eid, "i32", "u_eid"),
                                               _hp(u_keep, "u8", "u_keep"), n_u, _hp(q_src, "i32", "q_src"),
                                               _hp(q_dst, "i32", "q_dst"), _hp(q_neg, "i32", "q_neg"),
                                               _hp(q_t, "f64", "q_t"), q_src.numel(), _hp(loss_mask, "u8", "loss_mask"),
                                               _hp(loss_host, "f32", "loss_host"), _hp(gradnorm_host, "f32", "gradnorm_host"),
                                               _stream()))

    def step_mixed_host(self, src, dst, t, eid, is_aux, neg, loss_host, gradnorm_host, force_heavy=-1,
                        drop_q32=1 << 31, seed=0, batch_idx=0):
        self._ck(self.lib.tgnn_step_mixed_host(self._h, _hp(src, "i32", "src"), _hp(dst, "i32", "dst"), _hp(t, "f64", "t"),
                                               _hp(eid, "i32", "eid"), _hp(is_aux, "u8", "is_aux"), src.numel(),
                                               _hp(neg, "i32", "neg"), force_heavy, drop_q32, seed, batch_idx,
                                               _hp(loss_host, "f32", "loss_host"),
                                               _hp(gradnorm_host, "f32", "gradnorm_host"), _stream()))

    def set_graph_replay(self, enable: bool):
        self._ck(self.lib.tgnn_set_graph_replay(self._h, int(enable)))

    def set_grad_sync(self, defer: bool):
        """Steps stop after the gradient (to be reduced across workers); apply_gradient finishes them."""
        self._ck(self.lib.tgnn_set_grad_sync(self._h, int(defer)))

    def grad_buffer(self) -> torch.Tensor:
        """The context's gradient buffer as a float32 CUDA tensor (a view; valid while the context lives)."""
        ptr, n = C.c_void_p(), C.c_int64()
        self._ck(self.lib.tgnn_grad_buffer(self._h, C.byref(ptr), C.byref(n)))

        class _Mem:   # the CUDA array interface: torch wraps the pointer without copying
            __cuda_array_interface__ = {"shape": (n.value,), "typestr": "<f4", "data": (ptr.value, False), "version": 2}
        return torch.as_tensor(_Mem(), device=torch.device("cuda", torch.cuda.current_device()))

    def apply_gradient(self, scale: float, gradnorm_out):
        self._ck(self.lib.tgnn_apply_gradient(self._h, float(scale), _dp(gradnorm_out, "f32", "gradnorm_out"), _stream()))

    # ---- debug ----
    def debug_get_grads(self, grads_out):
        self._ck(self.lib.tgnn_debug_get_grads(self._h, _dp(grads_out, "f32", "grads_out"), _stream()))

    def debug_gemm(self, A, a_rs, a_cs, Bm, b_rs, b_cs, Cm, ldc, M, N, K, dev_M=None, dev_K=None, bias=None,
                   rowsum_out=None, relu=False, accumulate=False, split_k=1, precise=False):
        self._ck(self.lib.tgnn_debug_gemm(self._h, _dp(A, "f32", "A"), a_rs, a_cs, _dp(Bm, "f32", "B"), b_rs, b_cs,
                                          _dp(Cm, "f32", "C"), ldc, M, N, K, _dp(dev_M, "i32", "dev_M"),
                                          _dp(dev_K, "i32", "dev_K"), _dp(bias, "f32", "bias"),
                                          _dp(rowsum_out, "f32", "rowsum_out"), int(relu), int(accumulate), split_k,
                                          int(precise), _stream()))

    def profile_timeline(self):
        """[(kernel name, start_us, duration_us)] in issue order since profile_begin; switches profiling off."""
        buf = C.create_string_buffer(1 << 20)
        self._ck(self.lib.tgnn_profile_timeline(self._h, C.addressof(buf), len(buf)))
        out = []
        for line in buf.value.decode().splitlines():
            name, t0, dt = line.rsplit(" ", 2)
            out.append((name, float(t0), float(dt)))
        return out

    def debug_gemm_split(self, A, a_rs, a_cs, Bm, b_rs, b_cs, Cm, ldc, M, N, K, scratch, bias=None, relu=False,
                         accumulate=False, split_k=1, debug_withhold=0, spin_limit=0, check=True):
        """The split-bf16 projection kernel on fp32 operands (split inside `scratch`, a uint8 CUDA tensor)."""
        rc = self.lib.tgnn_debug_gemm_split(self._h, _dp(A, "f32", "A"), a_rs, a_cs, _dp(Bm, "f32", "B"), b_rs, b_cs,
                                            _dp(Cm, "f32", "C"), ldc, M, N, K, _dp(bias, "f32", "bias"), int(relu),
                                            int(accumulate), split_k, _dp(scratch, "u8", "scratch"), scratch.numel(),
                                            debug_withhold, spin_limit, _stream())
        if check:
            self._ck(rc)
        return rc

    def debug_get_embeddings(self, h_out):
        self._ck(self.lib.tgnn_debug_get_embeddings(self._h, _dp(h_out, "f32", "h_out"), _stream()))

    def debug_get_gates(self, h_gate_out, hid_gate_out):
        self._ck(self.lib.tgnn_debug_get_gates(self._h, _dp(h_gate_out, "u8", "h_gate_out"),
                                               _dp(hid_gate_out, "u8", "hid_gate_out"), _stream()))

    def profile_begin(self):
        self._ck(self.lib.tgnn_profile_begin(self._h))

    def profile_report(self) -> Dict[str, tuple]:
        """{kernel name: (launches, total_ms)} since profile_begin; switches profiling off."""
        buf = C.create_string_buffer(1 << 16)
        self._ck(self.lib.tgnn_profile_report(self._h, C.addressof(buf), len(buf)))
        out = {}
        for line in buf.value.decode().splitlines():
            name, cnt, ms = line.rsplit(" ", 2)
            out[name] = (int(cnt), float(ms))
        return out

    def clear_status(self):
        self._ck(self.lib.tgnn_clear_status(self._h, _stream()))

    def status(self) -> int:
        out = C.c_int32(0)
        self._ck(self.lib.tgnn_status(self._h, C.addressof(out), _stream()))
        return int(out.value)
