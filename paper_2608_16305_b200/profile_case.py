"""A small case of the training step for multi-pass profiler captures.

    python -m paper_2608_16305_b200.profile_case [--workload large] [--events 2000000] [--steps 4]

Builds the named workload's configuration with fewer events (same node count, feature width and dtype, d, k, heads
and batch size, so every kernel of a step has the launch configuration of the full-size run, while the device
holds a few hundred MB instead of the bench's 18.6 GB feature table) and runs a few consecutive mid-epoch training
steps in the 16-bit split mode without graph replay, so that a profiler sees one launch per kernel.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import trainer as T
from . import workload as wl


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="large", choices=sorted(wl.CONFIGS))
    ap.add_argument("--events", type=int, default=2_000_000)
    ap.add_argument("--steps", type=int, default=4)
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.workload]
    if args.events < cfg.num_events:
        cfg = wl.scaled(cfg, num_events=args.events)
    stream = wl.make_stream(cfg)
    efeat = wl.edge_feature_table_torch(cfg, "cuda")
    b0 = cfg.num_batches // 2
    dw = T.DeviceWorkload(stream, device="cuda", efeat=efeat, batches=range(b0 - 1, b0 + args.steps + 2))
    tr = T.Trainer(dw, wl.make_weights(cfg.d, cfg.d_e, cfg.seed), math_mode=B.TGNN_MATH_F16X3)
    tr.lib.set_graph_replay(False)
    with torch.cuda.stream(tr.stream):
        for b in range(b0, b0 + args.steps):
            tr.step(b)
    torch.cuda.synchronize()
    status = tr.lib.status()
    print("status", status)
    if status != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
