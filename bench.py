#!/usr/bin/env python
"""Benchmark of one chronological TGN-style training step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of the synthetic
"large" workload, the largest configuration that fits one GPU (17,000 nodes,
50,000,000 events, 186-d bf16 edge features resident in HBM, d = 100, k = 10,
2 heads, batch 4,000, 20 % replay events with pruning; `--workload` selects
the smaller ones): prune mask of the mixed batch, memory
update from the previous batch (messages, latest-event reduction, GRU), neighbor
search, attention embedding, masked loss, backward and Adam.  The metric is
target events per second (replay events are not counted, as in the paper's
throughput definition).  Inputs are resident in HBM for `value`; `e2e` repeats
the measurement through the host-buffer entry point with the per-step copies
inside the timed region.  Every step is timed with its own CUDA event pair on
the launching stream and L2 is flushed between steps (outside the events).

With N > 1 every rank runs an independent replica on its own GPU (under a
launcher, or spawned by this script when `--gpus N` is given without one): the
step has no independent units to shard, so there is no collective on the data
path; timing is the max over ranks.

Both arms run the same consecutive batches from the middle of the stream.
`--impl reference` times the CPU oracle on a bounded sample of them.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_16305_b200 import workload as wl  # noqa: E402

METRIC = "train events/s on 1 B200 (fwd+bwd, memory+embed)"
SPLIT_KERNELS = ("kv_proj", "dZ", "dW_kv")       # products that run on the split-fp16 kernel in the f16x3 mode
UNIT = "events/s"
WORKLOAD = "large"
SM_COUNT, FP32_LANES_PER_SM = 148, 128


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def aggregate_over_ranks(ms_local: float, units_local: int, device):
    """(max over ranks of the time, sum over ranks of the units); identity without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, interval_ms: int = 20):
        self.index, self.rows, self.proc, self.interval_ms = index, [], None, interval_ms
        self.t0 = self.t1 = None          # host times of the timed region (mark_begin / mark_end)

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.interval_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in line.split(",")]))

    def mark_begin(self):
        self.t0 = time.perf_counter()

    def mark_end(self):
        self.t1 = time.perf_counter()

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        # samples taken while the timed region ran (the sampler itself starts before the warm-up steps, so
        # that the tool is already reporting when the region begins)
        inside = [r for ts, r in self.rows if self.t0 is None or (ts >= self.t0 and (self.t1 is None or ts <= self.t1 + 0.05))]
        for r in inside:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_work(cfg: wl.WorkloadConfig, n_u: int, n_q: int, U: int):
    """Algorithmic bytes and flops of one step (what the method must move / compute).  Flops are the
    products of the step written out one by one: forward = the two update-cell products, the key/value, query
    and output projections, the attention's two contractions per head, the head's hidden layer and score;
    backward = one weight-gradient product per forward projection (same size as it), the input gradients that
    are needed (toward the head's inputs, the output and query projections' inputs, and only the memory and
    time-encoding columns of the attention inputs and of the winners' messages), and twice the attention's
    contractions.  About 1.1-1.2 x the forward count."""
    d, de, k = cfg.d, cfg.d_e, cfg.k
    f = 4 if cfg.feat_dtype == "f32" else 2
    R, NB = 3 * n_q, 3 * n_q * k
    P = sum(int(np.prod(s)) for s in wl.param_shapes(d, de).values())
    by = (R * 16 + NB * 16) + (2 * n_u * (2 * d * 4 + 8) + n_u * de * f) + U * (2 * d * 4 + 8) \
        + NB * (4 * d + de * f + 16) + 2 * R * 4 * d + NB * (4 * d + de * f) + R * 4 * d + 28 * P
    w = kernel_work(cfg, n_q, U)
    fwd = sum(w[n][1] for n in ("gru_gi", "gru_gh", "kv_proj", "q_proj", "out_proj")) + 4 * d * R * k \
        + 2.0 * (2 * n_q) * (2 * d * d + d)
    bwd = sum(w[n][1] for n in ("dW_i", "dW_h", "dW_kv", "dW_q", "dW_o", "dW_1", "dcat1", "dcat_o", "dzq", "dZ", "dX_phi")) \
        + 8 * d * R * k + 2.0 * (2 * n_q) * d
    return by, fwd, bwd


def kernel_work(cfg, n_q: int, U: int):
    """Algorithmic work of one launch of each kernel that can lead the step's time, by the library's profiler
    name: ("tensor", flops) for the dense products, ("hbm", bytes) for the gathers and reductions."""
    d, de, k = cfg.d, cfg.d_e, cfg.k
    f = 4 if cfg.feat_dtype == "f32" else 2
    R, NB, Q2 = 3 * n_q, 3 * n_q * k, 2 * n_q
    mm = lambda m, n, kk: ("tensor", 2.0 * m * n * kk)
    w = {
        "gru_gi": mm(U, 3 * d, cfg.d_msg), "gru_gh": mm(U, 3 * d, d), "kv_proj": mm(NB, 2 * d, cfg.d_kv),
        "q_proj": mm(R, d, 2 * d), "out_proj": mm(R, d, 2 * d), "head_hidden": mm(Q2, d, 2 * d),
        "dW_i": mm(3 * d, cfg.d_msg, U), "dW_h": mm(3 * d, d, U), "dW_kv": mm(2 * d, cfg.d_kv, NB),
        "dW_q": mm(d, 2 * d, R), "dW_o": mm(d, 2 * d, R), "dW_1": mm(d, 2 * d, Q2),
        "dcat1": mm(Q2, 2 * d, d), "dcat_o": mm(R, 2 * d, d), "dzq": mm(R, 2 * d, d),
        "dZ": mm(NB, 2 * d, 2 * d), "dX_phi": mm(U, d, 3 * d),
        # rows in, rows out
        "gather_z_static": ("hbm", NB * (de * f + 16) + NB * 4 * (de + d + 1)),
        "gather_z_memory": ("hbm", NB * (4 + 2 * 4 * d) + R * 2 * 4 * d),
        "attention_fwd": ("hbm", NB * 2 * d * 4 + R * (3 * d * 4 + 2 * k * 4)),
        "attention_bwd": ("hbm", NB * 2 * d * 4 * 2 + R * 4 * d * 3),
        "scatter_dmem": ("hbm", NB * (4 * d + 4) + R * 4 * d),
        "time_grad_z": ("hbm", NB * (4 * d + 4)),
        "head_fused": ("hbm", n_q * 3 * 4 * d * 2 + Q2 * (3 * d * 4 + d)),
        "sample_recent": ("hbm", R * 16 + NB * 16),
        "gradnorm_adam": ("hbm", 28 * sum(int(np.prod(s)) for s in wl.param_shapes(d, de).values())),
    }
    w["weight_grads"] = ("tensor", sum(w[n][1] for n in ("dW_kv", "dW_q", "dW_o", "dW_1", "dW_i", "dW_h")))
    return w


def algorithmic_work_jodie(cfg: wl.WorkloadConfig, n_u: int, n_q: int, U: int):
    """The same accounting for the time-projection model: no neighbor search, no attention."""
    d, de = cfg.d, cfg.d_e
    f = 4 if cfg.feat_dtype == "f32" else 2
    R = 3 * n_q
    P = sum(int(np.prod(s)) for s in wl.param_shapes(d, de, "jodie").values())
    by = (2 * n_u * (2 * d * 4 + 8) + n_u * de * f) + U * (2 * d * 4 + 8) + 2 * R * (4 * d + 8) + 28 * P
    fwd = 2 * d * (cfg.d_msg + d) * U + 2 * R * d + 2 * (2 * n_q) * 2 * d * d
    return by, fwd, 2.0 * fwd


def bench_batches(cfg, n_steps: int):
    """(first, span): both arms run batches first, first + 1, ... of the stream, `span` of them before the
    sequence starts over (with the state reset): consecutive batches from the middle of the epoch, where the
    neighbor lists are full; the whole epoch when it is shorter than the run."""
    nb = cfg.num_batches - 1                       # full batches only
    span = min(nb - 1, n_steps)
    first = max(1, min(nb // 2, nb - span))
    return first, span


def run_ours(args, rank, world, device):
    from paper_2608_16305_b200 import binding as B
    from paper_2608_16305_b200 import trainer as T
    cfg = wl.CONFIGS[args.workload]
    stream = wl.make_stream(cfg)
    efeat = wl.edge_feature_table_torch(cfg, device)
    first, span = bench_batches(cfg, args.steps + args.warmup)
    dw = T.DeviceWorkload(stream, device=device, efeat=efeat, batches=range(first - 1, first + span),
                          embed_aux=args.embed_aux)
    weights = wl.make_weights(cfg.d, cfg.d_e, cfg.seed, model=args.model)
    math_mode = {"fp32": B.TGNN_MATH_FP32, "tf32": B.TGNN_MATH_TF32, "tf32fast": B.TGNN_MATH_TF32_FAST,
                 "f16x3": B.TGNN_MATH_F16X3}[args.math]
    tr = T.Trainer(dw, weights, math_mode=math_mode, model=args.model)
    if args.no_graph:
        tr.lib.set_graph_replay(False)
    torch.cuda.synchronize()
    with torch.cuda.stream(tr.stream):     # a capturable stream: the library replays the step as a CUDA graph
        _run_ours_on_stream(args, rank, world, device, cfg, stream, dw, weights, tr)


def _run_ours_on_stream(args, rank, world, device, cfg, stream, dw, weights, tr):
    from paper_2608_16305_b200 import binding as B
    first, span = bench_batches(cfg, args.steps + args.warmup)
    K, W = args.steps, args.warmup
    # Cache hygiene between timed steps.  Workloads whose step streams far more than the 126 MB L2 through it (the
    # batch-4000 ones: > 1 GB of attention inputs, key/value rows and their gradients per step) evict everything
    # by themselves, and the only lines that survive a step are the small state every real training loop keeps
    # warm (parameters, the memory table); the small workloads get a 512 MB write between steps instead.
    step_bytes = 3 * cfg.batch * cfg.k * (cfg.d_kv * 4 * 2 + 2 * cfg.d * 4 * 4)
    use_flush = (step_bytes < 4 * (126 << 20)) if args.flush == "auto" else args.flush == "on"
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device) if use_flush else None   # > 126 MB L2
    peaks = measured_peaks()

    def batch_of(i):
        return first + i % span

    def reset_epoch():
        tr.memory.zero_()
        tr.last_update.zero_()

    def run_steps(first, count, fn, timed):
        evs = []
        for i in range(first, first + count):
            b = batch_of(i)
            if b == first:
                reset_epoch()
            if flush is not None:
                flush.fill_(i & 0xff)
            if timed:
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn(b)
                z.record()
                evs.append((a, z))
            else:
                fn(b)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(z) for a, z in evs)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    dev_step = lambda b: tr.step(b)

    # ---- device-resident inputs ----
    with ClockSampler(torch.cuda.current_device()) as clk:    # started before the warm-up: reporting by the time the region begins
        run_steps(0, W, dev_step, False)
        barrier()
        l0 = tr.lib.kernel_launches()
        clk.mark_begin()
        ms_dev = run_steps(W, K, dev_step, True)
        clk.mark_end()
    launches = tr.lib.kernel_launches() - l0
    barrier()
    clocks = clk.summary()
    loss_end = float(tr.loss.item())
    # events the timed steps processed: the targets plus the auxiliary replay events their prune masks kept
    keep_cum = torch.cat([torch.zeros(1, dtype=torch.int64, device=device), dw.mb_keep.to(torch.int64).cumsum(0)]).cpu().numpy()
    processed = sum(int(keep_cum[dw.mb_slice(batch_of(i)).stop] - keep_cum[dw.mb_slice(batch_of(i)).start]) for i in range(W, W + K))

    # ---- host buffers: one streaming call per mixed batch (packed H2D of the batch, D2H of loss and gradient norm) ----
    host = {}
    for i in range(W + K, W + K + W + K):
        bb = batch_of(i)
        if bb not in host:
            host[bb] = tr.host_batch(bb)
    # Loss and gradient norm come back every step into one of two pinned slots; the host reads a step's pair once
    # the NEXT step has been enqueued (its own event has long fired by then), so packing batch b+1 on the host
    # overlaps step b on the device -- a training loop that logs its loss one step late.
    loss_h = [torch.zeros(1).pin_memory() for _ in range(2)]
    gn_h = [torch.zeros(1).pin_memory() for _ in range(2)]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    h2d = d2h = 0
    n_host = 0
    last_read = [0.0, 0.0]

    def host_step(b):
        nonlocal h2d, d2h, n_host
        hb = host[b]
        if b == first:
            tr.lib.set_state(tr.memory, tr.last_update, tr.params, tr.adam_m, tr.adam_v, tr.step_count)  # restart the stream
        slot = n_host & 1
        tr.step_host(b, hb, loss_h[slot], gn_h[slot])
        done[slot].record()
        if n_host > 0:                                   # the previous step's result, read on the host
            done[1 - slot].synchronize()
            last_read[0], last_read[1] = float(loss_h[1 - slot][0]), float(gn_h[1 - slot][0])
        n_host += 1
        n, nq = hb["src"].numel(), hb["neg"].numel()
        h2d += 21 * n + 20 * nq + (nq if args.embed_aux else 0)    # + the target mask when every event is scored
        d2h += 8

    reset_epoch()
    tr.lib.set_state(tr.memory, tr.last_update, tr.params, tr.adam_m, tr.adam_v, tr.step_count)
    run_steps(W + K, W, host_step, False)
    barrier()
    h2d = d2h = 0
    ms_host = run_steps(W + K + W, K, host_step, True)
    barrier()
    h2d_step, d2h_step = h2d / K, d2h / K

    # ---- optional: the same steps under the adaptive runtime controller (Algorithm 2) ----
    adaptive = None
    if args.adaptive:
        ctl = B.Controller(alpha=0.1, beta=0.1, tau_g=1.6, tau_c=0.5, K=6)
        logs = []
        reset_epoch()
        ad_step = lambda b: logs.append(tr.step_adaptive(b, ctl))
        run_steps(0, W, ad_step, False)
        logs.clear()
        ms_ad = run_steps(W, K, ad_step, True)
        adaptive = {"value": K * cfg.batch / (ms_ad * 1e-3), "unit": UNIT, "ms_per_step": ms_ad / K,
                    "heavy_batches": sum(l["heavy"] for l in logs),
                    "boundaries": sum(l["boundary"] for l in logs),
                    "refresh_skipped": sum(1 for l in logs if l["sync"] == 0),
                    "constants": "K=6, tau_g=1.6, tau_c=0.5 (the paper's), alpha=beta=0.1 (unstated there)",
                    "how": "Trainer.step_adaptive: controller decisions on the host, one synchronisation per step "
                           "to read the gradient norm and the step's device time"}

    # ---- optional: the offline preprocessing pass (Algorithm 1 + Eq. 5) on this workload's stream ----
    preprocess = preprocess_pass(cfg, stream, dw, device) if args.preprocess else None

    # ---- per-kernel times of the same K steps (separate pass: the event pairs perturb a latency-bound step) ----
    reset_epoch()
    run_steps(0, W, dev_step, False)
    tr.lib.profile_begin()
    run_steps(W, K, dev_step, False)
    prof = tr.lib.profile_report()
    tot = sum(v[1] for v in prof.values()) or 1.0
    top = sorted(prof.items(), key=lambda kv: -kv[1][1])

    # throughput counts target events only; with every event scored the roots are the whole mixed batch
    ms_dev_max, units = aggregate_over_ranks(ms_dev, K * cfg.batch, device)
    ms_host_max, _ = aggregate_over_ranks(ms_host, K * cfg.batch, device)
    _, processed_all = aggregate_over_ranks(ms_dev, processed, device)
    n_q = cfg.max_mixed if args.embed_aux else cfg.batch
    if rank != 0:
        return
    # roofline of the dominant kernel: the one with the largest share of the per-kernel pass, measured by its own
    # algorithmic work (flops of the product, or bytes of the rows it must move) over its average launch time
    jodie = args.model == "jodie"
    U_est = min(2 * cfg.max_mixed, cfg.num_nodes) // 2
    work = {"gru_gi": ("tensor", 2.0 * U_est * cfg.d_msg * cfg.d)} if jodie else kernel_work(cfg, n_q, U_est)
    fp32_clk_ghz = (clocks["sm_max_mhz"] or 1965.0) / 1000.0

    def roof(name):
        cnt, ms_tot = prof.get(name, (0, 0.0))
        if name not in work or cnt == 0:
            return None
        kind, amount = work[name]
        dur_s = (ms_tot / cnt) * 1e-3
        if kind == "hbm":
            peak, unit, note, bound = peaks["hbm_gbs"], "GB/s", f"{peaks['source']} copy bandwidth", "hbm"
            ach = amount / dur_s / 1e9
        elif args.math == "f16x3" and name in SPLIT_KERNELS:
            # fp16 operands (two per value, three passes): the 16-bit tensor peak, fp16 = bf16 nominally
            peak, unit, bound = peaks["bf16_tflops"], "TFLOP/s", "tensor"
            note = f"{peaks['source']} bf16 burst (fp16 runs at the same nominal rate)"
            ach = amount / dur_s / 1e12
        elif args.math != "fp32":
            peak, unit, bound = peaks["bf16_tflops"] * 0.5, "TFLOP/s", "tensor"
            note = f"0.5 x {peaks['source']} bf16 burst (TF32 nominal ratio)"
            ach = amount / dur_s / 1e12
        else:
            peak, unit, bound = SM_COUNT * FP32_LANES_PER_SM * 2 * fp32_clk_ghz / 1000.0, "TFLOP/s", "alu"
            note = "148 SMs x 128 fp32 lanes x 2 flop x max SM clock"
            ach = amount / dur_s / 1e12
        return {"kernel": name, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "peak_source": note, ("flops_per_launch" if kind == "tensor" else "algorithmic_bytes_per_launch"): amount,
                "avg_launch_us": dur_s * 1e6, "launches": cnt}

    dom = next((n for n, _ in top if n in work), "kv_proj")
    rl = roof(dom) or {"kernel": dom, "bound": None, "achieved": None, "peak": None, "unit": None, "frac": None}
    # DRAM bytes of one launch come from an ncu capture, not from this run: null here, the committed summary is named
    rl["traffic"] = None
    rl["traffic_source"] = "profiles/ (ncu summary of this kernel: dram__bytes_read.sum + dram__bytes_write.sum per launch)"
    others = {n: roof(n) for n, _ in top[:8] if n != dom and n in work}
    by, f_fwd, f_bwd = (algorithmic_work_jodie if jodie else algorithmic_work)(cfg, cfg.max_mixed, n_q, U_est)
    out = {
        "metric": METRIC, "value": units / (ms_dev_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_dev_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"fp32": "f32", "f16x3": "f16 (two per fp32 value, 3 passes) + tf32 (3 passes), fp32 accumulate"}.get(args.math, "tf32"),
        "data": "synthetic",
        # targets + auxiliary replay events that passed pruning (the metric itself counts targets only, as the paper does)
        "processed_events_per_s": processed_all / (ms_dev_max * 1e-3),
        "config": {"workload": f"{cfg.name}: {cfg.num_nodes} nodes" + (f" ({cfg.num_src}+{cfg.num_nodes - cfg.num_src} bipartite)" if cfg.num_src else "")
                               + f", {cfg.num_events} events, d_e={cfg.d_e} {cfg.feat_dtype}, d={cfg.d}, k={cfg.k}, {cfg.heads} heads, "
                               f"batch {cfg.batch}, replay {cfg.replay_frac:g}" + (" with pruning" if cfg.prune else ""),
                   "model": "JODIE-style (recurrent cell + time projection)" if jodie else "TGN-style (GRU + temporal attention)",
                   "scored_events": "every event of the mixed batch, auxiliary events under loss weight 0" if args.embed_aux
                                    else "target events only",
                   "math_mode": args.math,
                   "l2": "512 MB buffer written between timed steps (outside the event pairs)" if use_flush else
                         f"inputs larger than L2: every step streams about {step_bytes / 1e6:.0f} MB of attention inputs, key/value rows and "
                         "gradients through the 126 MB L2; no extra flush",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "launch": "kernel by kernel" if args.no_graph else "CUDA graph replay of the step (captured by the library)",
                   "inputs": "resident in HBM"},
        "e2e": {"value": units / (ms_host_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d_step,
                "d2h_bytes_per_step": d2h_step, "ms_per_step": ms_host_max / K,
                "how": "tgnn_step_mixed_host: one call per mixed batch from host arrays (packed copy into one of two pinned blocks), loss and gradient norm copied back every step and read on the host one step later (the host packs batch b+1 while step b runs)"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": dict(rl, **{
            # the default mode splits every operand into a head and a tail: three tensor-core passes per
            # algorithmic product (not counted in "achieved"; shown for the pipe's real load)
            "tensor_passes": 3 if args.math in ("tf32", "f16x3") else 1,
            "other_kernels": {n: {k: r[k] for k in ("bound", "achieved", "unit", "frac", "avg_launch_us")} for n, r in others.items() if r},
            "step_algorithmic_bytes": by, "step_algorithmic_flops": f_fwd + f_bwd,
            "step_hbm_frac": (by / (ms_dev_max / K * 1e-3)) / (peaks["hbm_gbs"] * 1e9),
            "step_tensor_frac": ((f_fwd + f_bwd) / (ms_dev_max / K * 1e-3) / 1e12) / (peaks["bf16_tflops"] * (1.0 if args.math == "f16x3" else 0.5)),
            "kernel_share": {k: round(v[1] / tot, 4) for k, v in top[:12]},
            "kernel_ms_total": round(tot, 3)}),
        "loss_last": loss_end,
    }
    if adaptive is not None:
        out["adaptive"] = adaptive
    if preprocess is not None:
        out["preprocess"] = preprocess
    # the host baseline times the default costing (target events only)
    out["cpu_baseline"] = (cpu_baseline(cfg, stream, weights, budget_s=args.cpu_budget, model=args.model, b0=first + W)
                           if args.cpu_budget > 0 and not args.embed_aux else None)
    print(json.dumps(out))


def run_partitioned(args, rank, world, device):
    """The multi-worker form of the step, one worker per GPU: worker `rank` of a `world`-way node partition
    trains on its scanned mixed batches (Algorithm 1, Eq. 5) under the adaptive controller (Algorithm 2), with
    the boundary cache refresh as an all-to-all of packed rows and the gradient all-reduced before Adam.
    Throughput counts the original events of the global batches processed (each is some worker's target)."""
    import torch.distributed as dist
    from paper_2608_16305_b200 import binding as B
    from paper_2608_16305_b200 import distributed as D
    from paper_2608_16305_b200 import trainer as T
    cfg = wl.CONFIGS[args.workload]
    stream = wl.make_stream(cfg)
    efeat = wl.edge_feature_table_torch(cfg, device)
    K_sync = 6
    owner = (np.arange(cfg.num_nodes, dtype=np.int64) * 2654435761 % 2 ** 32 % world).astype(np.int32)
    t0 = time.time()
    dw = T.PartitionedWorkload(stream, owner, world, rank, K_sync, device=device, efeat=efeat, keep_sync=True)
    refresh = D.BoundaryRefresh(dw.refresh_plan(), cfg.d)
    torch.cuda.synchronize()
    prep_s = time.time() - t0
    weights = wl.make_weights(cfg.d, cfg.d_e, cfg.seed, model=args.model)
    math_mode = {"fp32": B.TGNN_MATH_FP32, "tf32": B.TGNN_MATH_TF32, "tf32fast": B.TGNN_MATH_TF32_FAST,
                 "f16x3": B.TGNN_MATH_F16X3}[args.math]
    tr = T.Trainer(dw, weights, math_mode=math_mode, model=args.model)
    tr.lib.set_grad_sync(True)
    ctl = B.Controller(alpha=0.1, beta=0.1, tau_g=1.6, tau_c=0.5, K=K_sync)
    nb = len(dw.batches) - 1
    K, W = args.steps, args.warmup
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    logs = []

    def run_steps(first, count):
        ms = 0.0
        for i in range(first, first + count):
            b = i % nb
            if b == 0:
                tr.memory.zero_()
                tr.last_update.zero_()
            flush.fill_(i & 0xff)
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            logs.append(tr.step_distributed(b, ctl, refresh=refresh))
            z.record()
            z.synchronize()
            ms += a.elapsed_time(z)
        return ms

    def barrier():
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(tr.stream):
        run_steps(0, W)
        barrier()
        logs.clear()
        l0 = tr.lib.kernel_launches()
        with ClockSampler(torch.cuda.current_device()) as clk:
            ms = run_steps(W, K)
        launches = tr.lib.kernel_launches() - l0
        barrier()
    ms_max, units = aggregate_over_ranks(ms, K * cfg.batch if rank == 0 else 0, device)
    if int(refresh.status.item()) or tr.lib.status():
        raise SystemExit("device status set during the partitioned run")
    if rank != 0:
        return
    print(json.dumps({
        "metric": METRIC, "value": units / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
        "dtype": "f32" if args.math == "fp32" else "tf32", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.num_nodes} nodes, {cfg.num_events} events, batch {cfg.batch} (global), "
                               f"{world}-way hashed node partition, source-owned targets, K = {K_sync}",
                   "parallelism": f"{world} partitioned worker(s): scanned mixed batches, boundary refresh (all-to-all of "
                                  "packed rows), gradient all-reduce, adaptive controller",
                   "math_mode": args.math, "l2": "512 MB buffer written between timed steps",
                   "inputs": "resident in HBM", "preprocess_s": round(prep_s, 3)},
        "e2e": None, "gpu_launches": int(launches), "clocks": clk.summary(),
        "worker0": {"mixed_events_per_step": float(np.diff(dw.mb_off).mean()), "targets_per_step": float(np.diff(dw.tgt_off).mean()),
                    "boundaries": sum(l["boundary"] for l in logs), "refreshes": sum(1 for l in logs if l["boundary"] and l["sync"]),
                    "rows_received": refresh.rows_received, "rows_sent": refresh.rows_sent,
                    "heavy_batches": sum(l["heavy"] for l in logs)},
        "loss_last": float(tr.loss.item()),
    }))


def preprocess_pass(cfg, stream, dw, device, P=8, K=6, reps=5):
    """Backward dependency scan for all P workers and windows, then worker 0's mixed batches; the oracle's
    scan is timed on a bounded number of (worker, window) pairs."""
    from paper_2608_16305_b200 import binding as B
    from oracle import scan as osc
    E, nb, N = cfg.num_events, cfg.num_batches, cfg.num_nodes
    Q = (nb + K - 1) // K
    owner_h = (np.arange(N, dtype=np.int64) * 2654435761 % 2 ** 32 % P).astype(np.int32)
    owner = torch.from_numpy(owner_h).to(device)
    role = torch.empty((P, E), dtype=torch.uint8, device=device)
    n_sync = torch.empty((P, Q), dtype=torch.int32, device=device)
    scratch = torch.empty(B.backward_scan_scratch(E, cfg.batch, K, N, P), dtype=torch.int32, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    off = torch.empty(nb + 1, dtype=torch.int32, device=device)
    toff = torch.empty(nb + 1, dtype=torch.int32, device=device)
    i32 = lambda: torch.empty(E, dtype=torch.int32, device=device)
    f64 = lambda: torch.empty(E, dtype=torch.float64, device=device)
    mb = (i32(), i32(), f64(), i32(), torch.empty(E, dtype=torch.uint8, device=device))
    tg = (i32(), i32(), f64(), i32(), i32())
    ev = lambda: torch.cuda.Event(enable_timing=True)
    ms_scan, ms_build = [], []
    for _ in range(reps + 2):
        a, b_, c = ev(), ev(), ev()
        a.record()
        B.backward_scan(dw.src, dw.dst, cfg.batch, K, owner, P, role, n_sync, None, scratch, status)
        b_.record()
        B.build_mixed(dw.src, dw.dst, dw.t, dw.neg, cfg.batch, role[0], off, toff, mb, tg, status)
        c.record()
        torch.cuda.synchronize()
        ms_scan.append(a.elapsed_time(b_))
        ms_build.append(b_.elapsed_time(c))
    ms_scan, ms_build = float(np.median(ms_scan[2:])), float(np.median(ms_build[2:]))
    aux_frac = float((role == 2).sum().item()) / float(max((role == 1).sum().item(), 1))
    t0, pairs = time.perf_counter(), 0
    for q in range(Q):
        osc.backward_scan(stream.src, stream.dst, owner_h, q % P, cfg.batch, K, q)
        pairs += 1
        if time.perf_counter() - t0 > 5.0:
            break
    cpu_s = time.perf_counter() - t0
    refresh = refresh_pass(cfg, dw, device, owner, P, K, Q, reps)
    return {"workers": P, "K": K, "windows": Q, "scan_ms": ms_scan, "build_mixed_ms": ms_build, "refresh": refresh,
            "scan_events_per_s": P * E / (ms_scan * 1e-3), "aux_per_target": aux_frac,
            "n_sync_mean": float(n_sync.float().mean().item()),
            "cpu_oracle_events_per_s": pairs * K * cfg.batch / cpu_s, "cpu_oracle_sample": f"{pairs} (worker, window) scans",
            "how": "tgnn_backward_scan over all workers and windows (hash partition), tgnn_build_mixed for worker 0; "
                   "CUDA events, median of %d" % reps}


def refresh_pass(cfg, dw, device, owner, P, K, Q, reps):
    """The boundary refresh's device work: worker 0's exchange plan for every window, and the two row movers,
    on a window of this workload and on a table larger than L2 (where their HBM rate means something)."""
    from paper_2608_16305_b200 import binding as B
    from paper_2608_16305_b200 import distributed as D
    N, d = cfg.num_nodes, cfg.d
    E = cfg.num_events
    role = torch.empty((P, E), dtype=torch.uint8, device=device)
    n_sync = torch.empty((P, Q), dtype=torch.int32, device=device)
    sync = torch.empty((P, Q, N), dtype=torch.uint8, device=device)
    scratch = torch.empty(B.backward_scan_scratch(E, cfg.batch, K, N, P), dtype=torch.int32, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    B.backward_scan(dw.src, dw.dst, cfg.batch, K, owner, P, role, n_sync, sync, scratch, status)
    n_sync_h = n_sync.cpu().numpy()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    plan, ms_plan = None, []
    for _ in range(reps + 2):
        a, z = ev(), ev()
        a.record()
        plan = D.RefreshPlan(sync, owner, n_sync_h, P, 0)
        z.record()
        torch.cuda.synchronize()
        ms_plan.append(a.elapsed_time(z))
    # a window of this workload: what worker 0 sends and receives at its busiest boundary
    q = int(np.argmax(plan.recv_off[:, -1] + plan.send_off[:, -1]))
    mem = torch.randn((N, d), dtype=torch.float32, device=device)
    lu = torch.rand(N, dtype=torch.float64, device=device)
    ref = D.BoundaryRefresh(plan, d)
    # a table larger than L2: 2 M rows, a random three quarters of them moved
    Nbig = 2_000_000
    big = torch.randn((Nbig, d), dtype=torch.float32, device=device)
    big_t = torch.rand(Nbig, dtype=torch.float64, device=device)
    nodes = torch.randperm(Nbig, device=device)[:Nbig * 3 // 4].to(torch.int32).contiguous()
    packed = torch.empty(nodes.numel() * (d + 2), dtype=torch.float32, device=device)
    st = torch.zeros(1, dtype=torch.int32, device=device)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    t = {"pack_window": [], "unpack_window": [], "pack_big": [], "unpack_big": []}
    for i in range(reps + 2):
        flush.fill_(i)
        e = [ev() for _ in range(3)]
        e[0].record()
        ref.pack(q, mem, lu)
        e[1].record()
        ref.unpack(q, mem, lu)
        e[2].record()
        torch.cuda.synchronize()
        t["pack_window"].append(e[0].elapsed_time(e[1]))
        t["unpack_window"].append(e[1].elapsed_time(e[2]))
        flush.fill_(i + 1)
        e = [ev() for _ in range(2)]
        e[0].record()
        B.pack_rows(big, big_t, nodes, packed, st)
        e[1].record()
        torch.cuda.synchronize()
        t["pack_big"].append(e[0].elapsed_time(e[1]))
        flush.fill_(i + 2)
        e = [ev() for _ in range(2)]
        e[0].record()
        B.unpack_rows(big, big_t, nodes, packed, st)
        e[1].record()
        torch.cuda.synchronize()
        t["unpack_big"].append(e[0].elapsed_time(e[1]))
    med = {k: float(np.median(v[2:])) for k, v in t.items()}
    row_bytes = 2 * (4 * d + 8) + 4               # state read + state written + the node id
    big_bytes = nodes.numel() * row_bytes
    peaks = measured_peaks()
    assert int(st.item()) == 0 and int(ref.status.item()) == 0
    return {"plan_ms_all_windows": float(np.median(ms_plan[2:])), "window": q,
            "window_rows_sent": int(plan.send_off[q, -1]), "window_rows_received": int(plan.recv_off[q, -1]),
            "pack_window_us": med["pack_window"] * 1e3, "unpack_window_us": med["unpack_window"] * 1e3,
            "bytes_per_row": row_bytes, "big_rows": int(nodes.numel()),
            "pack_big_gbs": big_bytes / (med["pack_big"] * 1e-3) / 1e9, "unpack_big_gbs": big_bytes / (med["unpack_big"] * 1e-3) / 1e9,
            "hbm_peak_gbs": peaks["hbm_gbs"], "pack_big_frac": big_bytes / (med["pack_big"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "unpack_big_frac": big_bytes / (med["unpack_big"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "how": "tgnn_refresh_plan for worker 0 over all windows; tgnn_pack_rows / tgnn_unpack_rows on worker 0's busiest "
                   "window and on 1.5 M random rows of a 2 M-row table (L2 flushed before each), CUDA events, median"}


def cpu_baseline(cfg, stream, weights, budget_s=20.0, steps=None, model="tgn", b0=None):
    """The oracle as it stands, one thread, on consecutive batches starting at b0 (the first batch the GPU
    arm times; default: the middle of the epoch)."""
    from oracle import oracle as orc
    ocfg = orc.make_config(cfg.num_nodes, cfg.d, cfg.d_e, cfg.k, cfg.heads, feat_bf16=cfg.feat_dtype == "bf16")
    ef = stream.efeat() if (cfg.d_e and cfg.num_events * cfg.d_e <= 500_000_000) else None
    if model == "jodie":
        return cpu_baseline_jodie(cfg, stream, weights, ocfg, ef, budget_s, steps, b0)
    state = orc.OracleState(ocfg, orc.pack_params(ocfg, weights))
    graph = (stream.indptr, stream.nbr, stream.eid, stream.ts)
    b0 = cfg.num_batches // 2 if b0 is None else b0
    # a feature table too large for a host copy: the oracle is handed the rows a step touches, regenerated
    # from the seed (bit-identical by construction) with the event ids renumbered in order; building that
    # view is input preparation and is not timed
    compact = cfg.num_events * cfg.d_e > 500_000_000
    prev, done, spent = None, 0, 0.0
    mbp = wl.mixed_batch(stream, b0 - 1)
    prev = (mbp.src, mbp.dst, mbp.t, mbp.eid, None)
    while (steps is None and spent < budget_s and done < 64) or (steps is not None and done < steps):
        b = b0 + done
        mb = wl.mixed_batch(stream, b)
        q = slice(b * cfg.batch, (b + 1) * cfg.batch)
        t0 = time.perf_counter()
        keep, _ = orc.prune_mask(cfg.num_nodes, mb.src, mb.dst, mb.eid, mb.is_aux, force_heavy=-1 if cfg.prune else 0,
                                 seed=cfg.seed, batch_idx=b)
        if not compact:
            state.step(graph, ef, prev, stream.src[q], stream.dst[q], stream.neg[q], stream.t[q])
            spent += time.perf_counter() - t0
        else:
            nodes = np.concatenate([stream.src[q], stream.dst[q], stream.neg[q]]).astype(np.int32)
            times = np.concatenate([stream.t[q]] * 3)
            nb = orc.sample_recent(*graph, nodes, times, cfg.k)
            spent += time.perf_counter() - t0
            ids = np.unique(np.concatenate([np.asarray(prev[3], np.int64), nb[1][nb[1] >= 0].astype(np.int64)]))
            rows = wl.edge_feature_rows(cfg.seed, ids, cfg.d_e, cfg.feat_dtype)
            remap = lambda e: np.where(np.asarray(e) >= 0, np.searchsorted(ids, np.maximum(e, 0)), -1).astype(np.int32)
            upd = (prev[0], prev[1], prev[2], remap(prev[3]), prev[4])
            t0 = time.perf_counter()
            res = orc.loss_and_grads(ocfg, state.params, state.memory, state.last_update, rows, upd,
                                     (nodes, times, nb[0], remap(nb[1]), nb[2], nb[3]), cfg.batch, None)
            state.memory, state.last_update = res.memory_post, res.last_update_post
            state.params, state.adam_m, state.adam_v, state.step_count = orc.adam(
                ocfg, res.grads, state.params, state.adam_m, state.adam_v, state.step_count)
            spent += time.perf_counter() - t0
        prev = (mb.src, mb.dst, mb.t, mb.eid, keep)
        done += 1
    return {"value": done * cfg.batch / spent, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": spent,
            "sample": f"{done} consecutive steps (batches {b0}..{b0 + done - 1}) of the {cfg.name} workload, "
                      f"single thread, host has {os.cpu_count()} cores"}


def cpu_baseline_jodie(cfg, stream, weights, ocfg, ef, budget_s, steps, b0=None):
    """The time-projection model's oracle (numpy, one process; its matrix products may use several threads)."""
    if ef is None and cfg.d_e:
        return None                      # feature table too large for a host copy: not sampled for this model
    from oracle import jodie as oj
    from oracle import oracle as orc
    p = oj.pack(cfg.d, cfg.d_e, weights)
    m, v, st = np.zeros_like(p), np.zeros_like(p), 0
    mem, lu = np.zeros((cfg.num_nodes, cfg.d)), np.zeros(cfg.num_nodes)
    b0 = cfg.num_batches // 2 if b0 is None else b0
    mbp = wl.mixed_batch(stream, b0 - 1)
    prev, done, spent = (mbp.src, mbp.dst, mbp.t, mbp.eid, None), 0, 0.0
    while (steps is None and spent < budget_s and done < 64) or (steps is not None and done < steps):
        b = b0 + done
        mb = wl.mixed_batch(stream, b)
        q = slice(b * cfg.batch, (b + 1) * cfg.batch)
        t0 = time.perf_counter()
        keep, _ = orc.prune_mask(cfg.num_nodes, mb.src, mb.dst, mb.eid, mb.is_aux, force_heavy=-1 if cfg.prune else 0,
                                 seed=cfg.seed, batch_idx=b)
        res = oj.step(ocfg, p, mem, lu, ef, prev, (stream.src[q], stream.dst[q], stream.neg[q], stream.t[q]))
        p, m, v, st = orc.adam(ocfg, res.grads, p, m, v, st)
        mem, lu = res.memory_post, res.last_update_post
        spent += time.perf_counter() - t0
        prev = (mb.src, mb.dst, mb.t, mb.eid, keep)
        done += 1
    return {"value": done * cfg.batch / spent, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "seconds": spent,
            "sample": f"{done} consecutive steps (batches {b0}..{b0 + done - 1}) of the {cfg.name} workload, numpy "
                      f"(BLAS threads as configured on the host, {os.cpu_count()} cores)"}


def run_reference(args, rank, world):
    """The CPU oracle as it stands on the GPU arm's workload and batches; each benchmark step is sampled by
    one oracle step, at most `n` of them, so that the run ends within minutes."""
    if rank != 0:
        return
    cfg = wl.CONFIGS[args.workload]
    stream = wl.make_stream(cfg)
    weights = wl.make_weights(cfg.d, cfg.d_e, cfg.seed, model=args.model)
    K, W = args.steps, args.warmup
    first, _ = bench_batches(cfg, K + W)
    per_step_s = 10.0 if cfg.batch >= 2000 else 1.5     # rough cost of one oracle step: bounds the sample
    n = max(1, min(K, int(60.0 / per_step_s)))
    res = cpu_baseline(cfg, stream, weights, steps=n, model=args.model, b0=first + W)
    ms = res["seconds"] * 1e3 / n
    desc = (f"{cfg.name}: {cfg.num_nodes} nodes, {cfg.num_events} events, d_e={cfg.d_e} {cfg.feat_dtype}, d={cfg.d}, "
            f"k={cfg.k}, {cfg.heads} heads, batch {cfg.batch}, replay {cfg.replay_frac:g}" + (" with pruning" if cfg.prune else ""))
    out = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": K,
           "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic",
           "config": {"workload": desc, "sample": f"{n} oracle steps standing for {K} steps"},
           "cpu_baseline": {"value": res["value"], "unit": UNIT, "kind": "oracle", "cores": res["cores"], "sample": res["sample"]},
           "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--math", default=os.environ.get("TGNN_BENCH_MATH", "f16x3"), choices=["fp32", "tf32", "tf32fast", "f16x3"],
                    help="f16x3 (default): the three products over the neighbor rows on split-fp16 operands, the small ones on "
                         "split-TF32; tf32: split-TF32 everywhere; fp32: FMA tiles")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(wl.CONFIGS),
                    help="default: large, the largest single-GPU configuration (the headline line); the others are parity-test cases")
    ap.add_argument("--model", default="tgn", choices=["tgn", "jodie"],
                    help="tgn: GRU + temporal attention (the benchmark's model); jodie: recurrent cell + time projection")
    ap.add_argument("--preprocess", action="store_true",
                    help="also time the backward dependency scan and mixed-batch construction (adds a 'preprocess' object)")
    ap.add_argument("--adaptive", action="store_true",
                    help="also time the steps under the adaptive runtime controller (adds an 'adaptive' object)")
    ap.add_argument("--embed-aux", action="store_true",
                    help="embed and score every event of the mixed batch (auxiliary events under loss weight 0) "
                         "instead of the target events only: the costing in which replay events pay the forward pass")
    ap.add_argument("--partitioned", action="store_true",
                    help="run the multi-worker form instead of independent replicas: one node-partitioned worker per "
                         "GPU with boundary refresh and gradient all-reduce (strong scaling over the same stream)")
    ap.add_argument("--flush", default="auto", choices=["auto", "on", "off"],
                    help="write a 512 MB buffer between timed steps; auto: only for workloads whose own step does not already "
                         "stream several times the L2 size")
    ap.add_argument("--no-graph", action="store_true", help="launch kernel by kernel instead of replaying a CUDA graph")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.gpus > 1 and "RANK" not in os.environ:
        # no launcher around us: start the N replica ranks ourselves (one process per GPU, rendezvous on localhost)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback); use --impl reference for the CPU oracle")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    group = world > 1 or (args.partitioned and "RANK" in os.environ)     # a launcher's single rank also gets its group
    if group:
        torch.distributed.init_process_group("nccl", device_id=device)
    try:
        (run_partitioned if args.partitioned else run_ours)(args, rank, world, device)
    finally:
        if group:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
