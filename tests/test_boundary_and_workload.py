"""CPU-side checks: the C-ABI library builds, loads and exports every symbol the
header declares; the synthetic workload generator has the structure the recipe
states; the multi-process timing aggregation works over gloo."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2608_16305_b200 import workload as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2608_16305_b200 import binding, build
    build.build_library()
    header = open(os.path.join(ROOT, "include", "tgnn.h")).read()
    declared = set(re.findall(r"TGNN_API\s+[\w\s\*]+?\b(tgnn_\w+)\s*\(", header))
    assert len(declared) >= 20
    assert declared == set(binding.EXPORTS)
    lib = binding.load_library()
    for name in declared:
        assert hasattr(lib, name), name


def test_param_layout_matches_between_header_order_and_counts():
    from paper_2608_16305_b200 import binding
    for name, want in [("tiny", 25537), ("wiki", 307401), ("lastfm", 221401), ("large", 314401)]:
        c = wl.CONFIGS[name]
        cfg = binding.make_config(c.num_nodes, c.d, c.d_e, c.k, c.heads)
        lay = binding.param_layout(cfg)
        assert lay["total"] == want == sum(int(np.prod(s)) for s in wl.param_shapes(c.d, c.d_e).values())
        offs = [lay[n] for n in binding.PARAM_NAMES]
        assert offs == sorted(offs) and offs[0] == 0
        # W_k and W_v (and b_k, b_v) are adjacent so the key/value projection is one [2d, d_kv] matrix
        assert lay["w_v"] == lay["w_k"] + c.d * c.d_kv and lay["b_v"] == lay["b_k"] + c.d


def test_oracle_and_library_agree_on_the_parameter_layout(oracle):
    from paper_2608_16305_b200 import binding
    c = wl.CONFIGS["wiki"]
    a = binding.param_layout(binding.make_config(c.num_nodes, c.d, c.d_e, c.k, c.heads))
    b = oracle.param_layout(oracle.make_config(c.num_nodes, c.d, c.d_e, c.k, c.heads))
    assert a == b


def test_invalid_configs_are_rejected_on_the_host():
    from paper_2608_16305_b200 import binding
    lib = binding.load_library()
    import ctypes as C
    assert lib.tgnn_param_count(C.byref(binding.make_config(100, 30, 16, 10, 2))) == -1    # d % 4
    assert lib.tgnn_param_count(C.byref(binding.make_config(100, 32, 15, 10, 2))) == -1    # odd d_e
    assert lib.tgnn_param_count(C.byref(binding.make_config(100, 32, 16, 40, 2))) == -1    # k > 32
    assert lib.tgnn_param_count(C.byref(binding.make_config(100, 32, 16, 10, 3))) == -1    # d % heads
    assert lib.tgnn_last_error(None) == b"null context"


def test_stream_structure():
    for name in ("tiny", "wiki"):
        c = wl.CONFIGS[name]
        s = wl.make_stream(c)
        assert len(s.t) == c.num_events and (np.diff(s.t) >= 0).all()
        assert abs(np.diff(s.t).mean() - 1.0) < 0.02                          # Exp(1) gaps
        if c.num_src:
            assert s.src.max() < c.num_src <= s.dst.min() and s.dst.max() < c.num_nodes
            assert s.neg.min() >= c.num_src
        else:
            assert (s.src != s.dst).all()
        top = np.bincount(np.concatenate([s.src, s.dst])).max() / (2 * c.num_events)
        assert 0.05 < top < 0.3                                               # a Zipf hub
        # T-CSR: every event appears under both endpoints, slices sorted by (ts, eid)
        assert s.indptr[-1] == 2 * c.num_events
        for n in (0, 1, int(s.dst[0]), c.num_nodes - 1):
            lo, hi = s.indptr[n], s.indptr[n + 1]
            e = s.eid[lo:hi]
            assert ((s.src[e] == n) | (s.dst[e] == n)).all()
            assert np.array_equal(s.ts[lo:hi], s.t[e])
            key = list(zip(s.ts[lo:hi], e))
            assert key == sorted(key)
            assert hi - lo == (s.src == n).sum() + (s.dst == n).sum()


def test_mixed_batches_follow_the_replay_recipe():
    c = wl.scaled(wl.CONFIGS["reddit"], num_events=6000)
    s = wl.make_stream(c)
    for b in range(c.num_batches):
        mb = wl.mixed_batch(s, b)
        tar = mb.eid[mb.is_aux == 0]
        rep = mb.eid[mb.is_aux == 1]
        assert np.array_equal(tar, np.arange(b * c.batch, min((b + 1) * c.batch, c.num_events)))
        assert len(rep) == (0 if b == 0 else round(c.replay_frac * c.batch))
        assert len(set(rep.tolist())) == len(rep)                              # deduplicated
        if len(rep):
            assert rep.min() >= max(0, b - 5) * c.batch and rep.max() < b * c.batch
        key = list(zip(mb.t, mb.eid))
        assert key == sorted(key)                                             # sort_t of Eq. 5
        assert np.array_equal(mb.src, s.src[mb.eid]) and np.array_equal(mb.t, s.t[mb.eid])
    again = wl.mixed_batch(s, 3)
    assert np.array_equal(again.eid, wl.mixed_batch(s, 3).eid)                 # seeded


def test_edge_features_are_regenerable_and_standard_normal():
    x = wl.edge_feature_rows(11, np.arange(4000), 64)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert np.array_equal(x[123:130], wl.edge_feature_rows(11, np.arange(123, 130), 64))
    c = wl.scaled(wl.CONFIGS["tiny"], num_events=3000)
    assert np.array_equal(wl.edge_feature_table_torch(c, "cpu").numpy(), wl.edge_feature_table(c))
    cb = wl.scaled(wl.CONFIGS["large"], num_events=2000, num_nodes=100)
    tb = wl.edge_feature_table_torch(cb, "cpu").view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(tb, wl.edge_feature_table(cb))


def test_weights_follow_the_initialisation_recipe():
    w = wl.make_weights(100, 172, 5)
    assert not w["gru_b_i"].any() and not w["b_2"].any() and not w["time_b"].any()
    assert w["time_w"][0] == 1.0 and abs(w["time_w"][-1] - 1e-9) < 1e-15
    a = np.sqrt(6.0 / (300 + 472))
    assert np.abs(w["gru_w_i"]).max() <= a and np.abs(w["gru_w_i"]).max() > 0.99 * a


def test_two_rank_timing_aggregation_over_gloo():
    code = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, %r)
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=2,
                        init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"])
rank = dist.get_rank()
ms, units = bench.aggregate_over_ranks(10.0 * (rank + 1), 600 * (rank + 1), torch.device("cpu"))
assert ms == 20.0 and units == 1800, (ms, units)
dist.barrier()
print("ok", rank)
""" % ROOT
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE))
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err.decode()[-2000:]
        assert b"ok" in out


def test_jodie_layout_matches_the_oracles_and_tgn_layout_is_unchanged():
    from oracle import jodie as oj
    from paper_2608_16305_b200 import binding
    for name in ("tiny", "wiki", "lastfm"):
        c = wl.CONFIGS[name]
        cfg = binding.make_config(c.num_nodes, c.d, c.d_e, c.k, c.heads, model=binding.TGNN_MODEL_JODIE)
        lay, ref = binding.param_layout(cfg), oj.param_layout(c.d, c.d_e)
        assert lay == {k: ref[k] for k in lay}
        shapes = wl.param_shapes(c.d, c.d_e, "jodie")
        assert tuple(shapes) == binding.PARAM_NAMES_JODIE == oj.PARAM_NAMES
        assert sum(int(np.prod(s)) for s in shapes.values()) == lay["total"]
        w = wl.make_weights(c.d, c.d_e, c.seed, bias_scale=0.1, model="jodie")
        flat = binding.pack_params(cfg, w)
        assert np.array_equal(flat, oj.pack(c.d, c.d_e, w).astype(np.float32))
    with pytest.raises(binding.TgnnError):
        binding.param_layout(binding.make_config(100, 32, 16, 10, 2, model=7))
