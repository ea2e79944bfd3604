"""Device-resident workload and the per-batch driver around the C ABI.

`DeviceWorkload` uploads a synthetic stream (events, T-CSR, edge features,
mixed batches) once; `Trainer.step(b)` then issues the calls of one
chronological training step in the lag-one order:

    prune mask of mixed batch b          (step 0; kept for when b is replayed)
    memory update from kept batch b-1    (steps 2-4)
    sample / embed / loss / backward / Adam on the targets of batch b (steps 1,5,6)

All arithmetic happens inside the library; this file only slices tensors.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding as B
from . import workload as wl


class DeviceWorkload:
    """The event stream, its neighbor index and its mixed batches on the device.

    embed_aux: every event of a mixed batch is embedded and scored, auxiliary events under loss weight 0
    (the target mask of Eq. 12 applied in Eq. 13), instead of the target events only; the negative of an
    event is the stream's negative for its event id either way."""

    def __init__(self, stream: wl.EventStream, device="cuda", batches: Optional[range] = None,
                 efeat: Optional[torch.Tensor] = None, embed_aux: bool = False):
        cfg = stream.cfg
        self.cfg = cfg
        self.embed_aux = bool(embed_aux)
        self.stream = stream
        dev = torch.device(device)
        self.device = dev
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.src, self.dst, self.t, self.neg = t(stream.src), t(stream.dst), t(stream.t), t(stream.neg)
        self.indptr, self.nbr, self.eid, self.ts = t(stream.indptr), t(stream.nbr), t(stream.eid), t(stream.ts)
        if efeat is not None:
            self.efeat = efeat
        elif cfg.d_e == 0:
            self.efeat = None
        elif cfg.feat_dtype == "f32":
            self.efeat = t(stream.efeat())
        else:
            self.efeat = torch.from_numpy(stream.efeat().view(np.int16)).to(dev).view(torch.bfloat16)
        # mixed batches, concatenated; batch b occupies [off[b], off[b+1])
        self.batches = batches if batches is not None else range(cfg.num_batches)
        mbs = [wl.mixed_batch(stream, b) for b in self.batches]
        self.mb_host: List[wl.MixedBatch] = mbs
        off = np.zeros(len(mbs) + 1, dtype=np.int64)
        np.cumsum([m.n for m in mbs], out=off[1:])
        self.mb_off = off
        cat = lambda f, dt: t(np.concatenate([getattr(m, f) for m in mbs]).astype(dt)) if mbs else None
        self.mb_src, self.mb_dst = cat("src", np.int32), cat("dst", np.int32)
        self.mb_t, self.mb_eid, self.mb_aux = cat("t", np.float64), cat("eid", np.int32), cat("is_aux", np.uint8)
        self.mb_keep = torch.ones_like(self.mb_aux) if mbs else None
        self.heavy = torch.zeros(len(mbs), dtype=torch.int32, device=dev)
        self.max_mixed = cfg.max_mixed      # capacities the library context is created with
        self.max_targets = cfg.max_mixed if self.embed_aux else cfg.batch
        self._scored_arrays()

    def _scored_arrays(self):
        """Negatives and loss mask per mixed-batch event (used when every event is scored)."""
        if self.embed_aux and self.mb_aux is not None:
            self.mb_neg = self.neg[self.mb_eid.long()].contiguous()
            self.mb_lmask = (1 - self.mb_aux).contiguous()

    def mb_slice(self, b: int):
        i = b - self.batches.start
        return slice(int(self.mb_off[i]), int(self.mb_off[i + 1]))

    def target_slice(self, b: int):
        return slice(b * self.cfg.batch, min((b + 1) * self.cfg.batch, self.cfg.num_events))

    def targets(self, b: int):
        """Device tensors (src, dst, neg, t) of the scored events of batch b: its target events, or every
        event of the mixed batch under embed_aux."""
        if self.embed_aux:
            m = self.mb_slice(b)
            return self.mb_src[m], self.mb_dst[m], self.mb_neg[m], self.mb_t[m]
        return self._targets(b)

    def _targets(self, b: int):
        q = self.target_slice(b)
        return self.src[q], self.dst[q], self.neg[q], self.t[q]

    def loss_mask(self, b: int):
        """Target mask (Eq. 12) over the scored events of batch b; None when all of them are targets."""
        return self.mb_lmask[self.mb_slice(b)] if self.embed_aux else None

    def targets_host(self, b: int):
        if self.embed_aux:
            mb = self.mb_host[b - self.batches.start]
            return mb.src, mb.dst, self.stream.neg[mb.eid], mb.t
        return self._targets_host(b)

    def _targets_host(self, b: int):
        q = self.target_slice(b)
        s = self.stream
        return s.src[q], s.dst[q], s.neg[q], s.t[q]

    def loss_mask_host(self, b: int):
        return (1 - self.mb_host[b - self.batches.start].is_aux).astype(np.uint8) if self.embed_aux else None


class PartitionedWorkload(DeviceWorkload):
    """Worker p's view of the stream under a node partition: its mixed batches come from the
    backward dependency scan (Algorithm 1) instead of the resampled replay sets, its targets are the
    source-owned events of each global batch.  The scan and the batch construction run on the device."""

    def __init__(self, stream: wl.EventStream, owner: np.ndarray, P: int, p: int, K: int, device="cuda",
                 efeat: Optional[torch.Tensor] = None, embed_aux: bool = False, keep_sync: bool = False):
        super().__init__(stream, device=device, batches=range(0, 0), efeat=efeat, embed_aux=embed_aux)
        cfg = self.cfg
        dev = self.device
        E, nb = cfg.num_events, cfg.num_batches
        Q = (nb + K - 1) // K
        self.owner = torch.from_numpy(np.ascontiguousarray(owner, dtype=np.int32)).to(dev)
        self.P, self.p, self.K = P, p, K
        self.role = torch.empty((P, E), dtype=torch.uint8, device=dev)
        self.n_sync = torch.empty((P, Q), dtype=torch.int32, device=dev)
        # N_sync membership flags of every (worker, window): the input of the boundary refresh plan
        self.sync = torch.empty((P, Q, cfg.num_nodes), dtype=torch.uint8, device=dev) if keep_sync else None
        scratch = torch.empty(B.backward_scan_scratch(E, cfg.batch, K, cfg.num_nodes, P), dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.backward_scan(self.src, self.dst, cfg.batch, K, self.owner, P, self.role, self.n_sync, self.sync, scratch, status)
        off = torch.empty(nb + 1, dtype=torch.int32, device=dev)
        toff = torch.empty(nb + 1, dtype=torch.int32, device=dev)
        i32 = lambda: torch.empty(E, dtype=torch.int32, device=dev)
        mb = (i32(), i32(), torch.empty(E, dtype=torch.float64, device=dev), i32(), torch.empty(E, dtype=torch.uint8, device=dev))
        tg = (i32(), i32(), torch.empty(E, dtype=torch.float64, device=dev), i32(), i32())
        status2 = torch.zeros(1, dtype=torch.int32, device=dev)
        B.build_mixed(self.src, self.dst, self.t, self.neg, cfg.batch, self.role[p], off, toff, mb, tg, status2)
        torch.cuda.synchronize(dev)
        if int(status.item()) or int(status2.item()):
            raise RuntimeError("backward scan / mixed-batch construction reported a device-side error")
        self.mb_off = off.cpu().numpy().astype(np.int64)
        self.tgt_off = toff.cpu().numpy().astype(np.int64)
        n_m, n_t = int(self.mb_off[-1]), int(self.tgt_off[-1])
        self.mb_src, self.mb_dst, self.mb_t, self.mb_eid, self.mb_aux = (x[:n_m].clone() for x in mb)
        self.tgt_src, self.tgt_dst, self.tgt_t, self.tgt_neg, self.tgt_eid = (x[:n_t].clone() for x in tg)
        self.mb_keep = torch.ones_like(self.mb_aux)
        self.batches = range(0, nb)
        self.heavy = torch.zeros(nb, dtype=torch.int32, device=dev)
        self.max_mixed = max(1, int(np.diff(self.mb_off).max()))
        self.max_targets = self.max_mixed if self.embed_aux else max(1, int(np.diff(self.tgt_off).max()))
        self._scored_arrays()
        h = [x.cpu().numpy() for x in (self.mb_src, self.mb_dst, self.mb_t, self.mb_eid, self.mb_aux)]
        self.mb_host = [wl.MixedBatch(b, *(a[self.mb_off[b]:self.mb_off[b + 1]] for a in h)) for b in range(nb)]
        self._tgt_host = [x.cpu().numpy() for x in (self.tgt_src, self.tgt_dst, self.tgt_neg, self.tgt_t)]

    def refresh_plan(self):
        """This worker's boundary refresh plan for every window (needs keep_sync=True)."""
        from . import distributed as D
        if self.sync is None:
            raise RuntimeError("the workload was built without the N_sync flags (keep_sync=True)")
        return D.RefreshPlan(self.sync, self.owner, self.n_sync.cpu().numpy(), self.P, self.p)

    def _tslice(self, b: int):
        return slice(int(self.tgt_off[b]), int(self.tgt_off[b + 1]))

    def _targets(self, b: int):
        q = self._tslice(b)
        return self.tgt_src[q], self.tgt_dst[q], self.tgt_neg[q], self.tgt_t[q]

    def _targets_host(self, b: int):
        q = self._tslice(b)
        return tuple(a[q] for a in self._tgt_host)


class Trainer:
    def __init__(self, dw: DeviceWorkload, weights, math_mode=B.TGNN_MATH_FP32, lr=1e-4, model: str = "tgn"):
        cfg = dw.cfg
        self.dw = dw
        self.tcfg = B.make_config(cfg.num_nodes, cfg.d, cfg.d_e, cfg.k, cfg.heads,
                                  feat_dtype=B.TGNN_BF16 if cfg.feat_dtype == "bf16" else B.TGNN_F32,
                                  max_events=dw.max_mixed, max_roots=3 * dw.max_targets, math_mode=math_mode, lr=lr,
                                  model=B.TGNN_MODEL_JODIE if model == "jodie" else B.TGNN_MODEL_TGN,
                                  embed_aux=dw.embed_aux)
        self.lib = B.Tgnn(self.tcfg)
        dev = dw.device
        P = B.param_layout(self.tcfg)["total"]
        self.memory = torch.zeros((cfg.num_nodes, cfg.d), dtype=torch.float32, device=dev)
        self.last_update = torch.zeros(cfg.num_nodes, dtype=torch.float64, device=dev)
        self.params = torch.from_numpy(B.pack_params(self.tcfg, weights)).to(dev)
        self.adam_m = torch.zeros(P, dtype=torch.float32, device=dev)
        self.adam_v = torch.zeros(P, dtype=torch.float32, device=dev)
        self.step_count = torch.zeros(1, dtype=torch.int64, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.gradnorm = torch.zeros(1, dtype=torch.float32, device=dev)
        self.lib.set_graph(dw.indptr, dw.nbr, dw.eid, dw.ts)
        self.lib.set_edge_features(dw.efeat, cfg.num_events)
        self.lib.set_state(self.memory, self.last_update, self.params, self.adam_m, self.adam_v, self.step_count)
        self.prune_seed = cfg.seed
        self.drop_q32 = 1 << 31
        # The library replays a step as a CUDA graph, which it records by stream capture; the legacy
        # default stream cannot capture, so when the caller is on it the step runs on this stream,
        # ordered after / before the caller's stream with events.
        self.stream = torch.cuda.Stream(device=dev, priority=-1)
        # The prune mask of batch b is consumed only when b is replayed as the update batch of step b+1,
        # so it runs on a stream of its own beside step b and is waited for at the start of step b+1.
        self.prune_stream = torch.cuda.Stream(device=dev)

    def _run(self, fn):
        cur = torch.cuda.current_stream()
        if cur != torch.cuda.default_stream():
            return fn()
        self.stream.wait_stream(cur)
        with torch.cuda.stream(self.stream):
            out = fn()
        cur.wait_stream(self.stream)
        return out

    def prune(self, b: int, force_heavy: Optional[int] = None, drop_q32: Optional[int] = None):
        """Keep mask of mixed batch b.  Default: the workload's own rule (count trigger, hashed half);
        force_heavy / drop_q32 override it (the adaptive controller passes its H and "all")."""
        dw = self.dw
        s = dw.mb_slice(b)
        i = b - dw.batches.start
        if force_heavy is None:
            force_heavy = -1 if dw.cfg.prune else 0
        self.lib.prune_mask(dw.mb_src[s], dw.mb_dst[s], dw.mb_eid[s], dw.mb_aux[s], dw.mb_keep[s], dw.heavy[i:i + 1],
                            force_heavy=force_heavy, drop_q32=self.drop_q32 if drop_q32 is None else drop_q32,
                            seed=self.prune_seed, batch_idx=b)

    def host_batch(self, b: int):
        """Pinned host copies of mixed batch b and of its targets' negatives (what a data loader would hand over)."""
        dw = self.dw
        mb = dw.mb_host[b - dw.batches.start]
        pin = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).pin_memory()
        return dict(src=pin(mb.src, np.int32), dst=pin(mb.dst, np.int32), t=pin(mb.t, np.float64),
                    eid=pin(mb.eid, np.int32), aux=pin(mb.is_aux, np.uint8), neg=pin(dw.targets_host(b)[2], np.int32))

    def step_host(self, b: int, hb, loss_host, gradnorm_host):
        """One training step fed from host memory: a single call of the streaming entry point per mixed batch."""
        cfg = self.dw.cfg
        return self._run(lambda: self.lib.step_mixed_host(
            hb["src"], hb["dst"], hb["t"], hb["eid"], hb["aux"], hb["neg"], loss_host, gradnorm_host,
            force_heavy=-1 if cfg.prune else 0, drop_q32=self.drop_q32, seed=self.prune_seed, batch_idx=b))

    def step(self, b: int, with_update: bool = True, force_heavy: Optional[int] = None,
             drop_q32: Optional[int] = None):
        """One training step on batch b (device-resident inputs)."""
        return self._run(lambda: self._step(b, with_update, force_heavy, drop_q32))

    def step_adaptive(self, b: int, ctl: "B.Controller", batch_time: Optional[float] = None):
        """One step under the adaptive runtime controller (Algorithm 2).

        Before the step the controller decides S_r (logged only: one GPU has no remote cache to
        refresh) and H_r; under H_r = 1 every pure replay event of mixed batch b is pruned
        (Eq. 10-11).  After it, the gradient norm and the step's device time (CUDA events, ms;
        or `batch_time` when the caller supplies its own measurement) feed the controller's
        averages.  Reads two scalars back, so it synchronises once per step.
        """
        r = b - self.dw.batches.start
        boundary, sync, heavy = ctl.begin_batch(r)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def run():
            e0.record()
            self._step(b, True, heavy, 0xFFFFFFFF)
            e1.record()
        self._run(run)
        e1.synchronize()
        c = float(e0.elapsed_time(e1)) if batch_time is None else float(batch_time)
        g = float(self.gradnorm.item())
        ctl.end_batch(g, c)
        return dict(r=r, boundary=boundary, sync=sync, heavy=heavy, g=g, c=c)

    def step_distributed(self, b: int, ctl: "B.Controller", refresh=None, group=None, reduce_gradient=None,
                         batch_time: Optional[float] = None):
        """One step of one worker among several (Algorithm 2 with its exchanges).

        At a candidate boundary the coordinator's decision S_r is broadcast and, if 1, the boundary
        refresh of the window that starts here runs on the tables as they stand (the lag-one update of
        the previous batch is applied after it, by this worker's own mixed batch).  The step then stops
        after the gradient; the workers' gradients are summed (`reduce_gradient(buffer)`, default an
        all-reduce over `group`), and norm and Adam run on their mean, so g_r is the same number on every
        worker.  Requires lib.set_grad_sync(True).
        """
        from . import distributed as D
        import torch.distributed as dist
        r = b - self.dw.batches.start
        boundary, sync, heavy = ctl.begin_batch(r)
        multi = dist.is_available() and dist.is_initialized()
        if boundary and refresh is not None:
            if multi:
                sync = D.broadcast_decision(sync, self.dw.device, group)
            if sync:
                self._run(lambda: refresh.run(r // ctl.K, self.memory, self.last_update))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        world = dist.get_world_size(group) if multi else 1

        def run():
            e0.record()
            self._step(b, True, heavy, 0xFFFFFFFF)
            e1.record()                                     # the worker's own batch time excludes the wait for the others
            g = self.lib.grad_buffer()
            if reduce_gradient is not None:
                world_ = reduce_gradient(g)
            else:
                if world > 1:
                    dist.all_reduce(g, op=dist.ReduceOp.SUM, group=group)
                world_ = world
            self.lib.apply_gradient(1.0 / world_, self.gradnorm)
        self._run(run)
        e1.synchronize()
        c = float(e0.elapsed_time(e1)) if batch_time is None else float(batch_time)
        g = float(self.gradnorm.item())
        ctl.end_batch(g, c)
        return dict(r=r, boundary=boundary, sync=sync, heavy=heavy, g=g, c=c)

    def _step(self, b: int, with_update: bool, force_heavy: Optional[int] = None, drop_q32: Optional[int] = None):
        dw = self.dw
        cur = torch.cuda.current_stream()
        cur.wait_stream(self.prune_stream)          # keep mask of batch b-1 is complete
        self.prune_stream.wait_stream(cur)          # inputs uploaded on this stream are visible
        with torch.cuda.stream(self.prune_stream):
            self.prune(b, force_heavy, drop_q32)
        tsrc, tdst, tneg, tt = dw.targets(b)
        if with_update and b > dw.batches.start:
            u = dw.mb_slice(b - 1)
            upd = (dw.mb_src[u], dw.mb_dst[u], dw.mb_t[u], dw.mb_eid[u], dw.mb_keep[u])
        else:
            upd = (None, None, None, None, None)
        self.lib.train_step(*upd, tsrc, tdst, tneg, tt, dw.loss_mask(b), self.loss, self.gradnorm)
