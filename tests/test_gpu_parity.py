"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Integers, indices and masks must be
bit-exact; floats are compared teacher-forced per batch (the oracle starts each
step from the GPU's pre-step state) with

    err(x) = max|x_gpu - x_ref| / max(max|x_ref|, 1e-6)

<= 2e-3 for the TF32 tensor-core mode (<= 1e-2 with bf16 features), and a much
tighter 1e-4 for the fp32 FMA mode, per compared tensor: updated memory rows,
embeddings h, loss, gradient norm, every gradient tensor, the updated
parameters (the oracle's own Adam step on its own gradient), and the Adam
kernel by itself (the oracle's Adam fed with the GPU gradient, since Adam's
g/(|g|+eps) amplifies rounding noise of near-zero gradients without bound).
"""
import os
import numpy as np
import pytest
import torch

from paper_2608_16305_b200 import workload as wl

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "tf32": 2e-3, "tf32_bf16": 1e-2, "tf32fast": 2e-3, "tf32fast_bf16": 1e-2, "f16x3": 2e-3, "f16x3_bf16": 1e-2}
# ReLU's derivative jumps at zero.  A unit whose pre-activation is closer to zero than the kernel's
# arithmetic resolves may land on either side; for such units (|pre| <= GATE_EPS * max|pre|, nowhere
# else) the oracle differentiates the branch the kernel took.
GATE_EPS = {"fp32": 1e-5, "tf32": 2e-4, "tf32fast": 3e-3, "f16x3": 2e-4}
# How many units per step may take the kernel's branch against the oracle's own fp64 sign: a handful, or
# 2e-5 of the step's ReLU units on the big batches (measured: at most 3 units in any compared step of the
# five workloads, 1.2 M to 2 M units per step on the batch-4000 ones).
MAX_OVERRIDES = lambda units: max(10, int(2e-5 * units))
OVERRIDE_LOG = os.environ.get("TGNN_OVERRIDE_LOG")   # optional: append "what units overrides" per compared step


def relerr(gpu, ref):
    gpu, ref = np.asarray(gpu, np.float64), np.asarray(ref, np.float64)
    if ref.size == 0:
        return 0.0
    return float(np.abs(gpu - ref).max() / max(np.abs(ref).max(), 1e-6))


@pytest.fixture(scope="module")
def B():
    from paper_2608_16305_b200 import binding
    binding.load_library()
    return binding


def dev(a, dt=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dt is not None:
        t = t.to(dt)
    return t.cuda()


def orc_cfg(oracle, c, **kw):
    return oracle.make_config(c.num_nodes, c.d, c.d_e, c.k, c.heads, feat_bf16=c.feat_dtype == "bf16", **kw)


# ------------------------------------------------------------ set-up -------
class Rig:
    """A workload on the device plus a library context and an oracle configuration."""

    def __init__(self, B, oracle, cfg, math="fp32", batches=None, bias_scale=0.1, lr=1e-3, partition=None, model="tgn",
                 embed_aux=False):
        from paper_2608_16305_b200 import trainer
        self.B, self.oracle, self.cfg, self.math = B, oracle, cfg, math
        self.stream = wl.make_stream(cfg)
        efeat_dev = None
        self.compact = cfg.num_events * cfg.d_e > 2_000_000_000   # too big for a host copy: fetch rows per step
        if cfg.num_events * cfg.d_e > 20_000_000:      # big table: generate it on the device (bit-identical)
            efeat_dev = wl.edge_feature_table_torch(cfg, "cuda")
            if not self.compact:
                self.stream._efeat = self._to_host(efeat_dev)
        self.efeat_dev = efeat_dev
        if partition is None:
            self.dw = trainer.DeviceWorkload(self.stream, batches=batches, efeat=efeat_dev, embed_aux=embed_aux)
        else:   # (owner, P, p, K): worker p's mixed batches from the backward dependency scan
            self.dw = trainer.PartitionedWorkload(self.stream, *partition, efeat=efeat_dev, embed_aux=embed_aux)
        self.model = model
        self.weights = wl.make_weights(cfg.d, cfg.d_e, cfg.seed, bias_scale=bias_scale, model=model)
        mode = {"fp32": B.TGNN_MATH_FP32, "tf32": B.TGNN_MATH_TF32, "tf32fast": B.TGNN_MATH_TF32_FAST,
                "f16x3": B.TGNN_MATH_F16X3}[math]
        self.tr = trainer.Trainer(self.dw, self.weights, math_mode=mode, lr=lr, model=model)
        f32 = lambda x: float(np.float32(x))      # the library's configuration holds fp32 hyper-parameters
        self.ocfg = orc_cfg(oracle, cfg, lr=f32(lr), beta1=f32(0.9), beta2=f32(0.999), eps=f32(1e-8))
        self.graph = (self.stream.indptr, self.stream.nbr, self.stream.eid, self.stream.ts)
        self.efeat = self.stream.efeat() if (cfg.d_e and not self.compact) else None
        self.lay = B.param_layout(self.tr.tcfg)
        self.shapes = wl.param_shapes(cfg.d, cfg.d_e, model)
        key = math + ("_bf16" if cfg.feat_dtype == "bf16" and math != "fp32" else "")
        self.tol = TOL[key]

    def _to_host(self, t):
        host = t.cpu()
        return host.view(torch.int16).numpy().view(np.uint16) if self.cfg.feat_dtype == "bf16" else host.numpy()

    def snapshot(self):
        tr = self.tr
        torch.cuda.synchronize()
        return dict(memory=tr.memory.cpu().numpy().astype(np.float64), last_update=tr.last_update.cpu().numpy().copy(),
                    params=tr.params.cpu().numpy().astype(np.float64), m=tr.adam_m.cpu().numpy().astype(np.float64),
                    v=tr.adam_v.cpu().numpy().astype(np.float64), step=int(tr.step_count.item()))

    def upd_host(self, b):
        """Kept update events of batch b-1 as the oracle wants them (or None)."""
        if b <= self.dw.batches.start:
            return None
        mb = self.dw.mb_host[b - 1 - self.dw.batches.start]
        keep = self.dw.mb_keep[self.dw.mb_slice(b - 1)].cpu().numpy()
        return (mb.src, mb.dst, mb.t, mb.eid, keep)

    def gpu_gates(self, b):
        nq = len(self.dw.targets_host(b)[0])
        torch.cuda.synchronize()
        hg = torch.zeros((3 * nq, self.cfg.d), dtype=torch.uint8, device="cuda")
        dg = torch.zeros((2 * nq, self.cfg.d), dtype=torch.uint8, device="cuda")
        self.tr.lib.debug_get_gates(hg, dg)
        torch.cuda.synchronize()
        return hg.cpu().numpy(), dg.cpu().numpy()

    def oracle_step(self, pre, b, gates=None, loss_mask="workload", want_grads=True):
        o = self.oracle
        t_src, t_dst, t_neg, t_t = self.dw.targets_host(b)
        if isinstance(loss_mask, str):
            loss_mask = self.dw.loss_mask_host(b)
        self._last_mask = loss_mask
        nodes = np.concatenate([t_src, t_dst, t_neg])
        times = np.concatenate([t_t] * 3)
        if self.model == "jodie":
            from oracle import jodie as oj
            upd = self.upd_host(b)
            if upd is None:
                z = np.zeros(0, np.int32)
                upd = (z, z, np.zeros(0), z, None)
            hint = {} if gates is None else dict(hid_gate=gates[1], gate_eps=GATE_EPS[self.math])
            res = oj.step(self.ocfg, pre["params"], pre["memory"], pre["last_update"], self.efeat, upd,
                          (t_src, t_dst, t_neg, t_t), loss_mask, **hint)
            return res, (nodes, times)
        nb = o.sample_recent(*self.graph, nodes, times, self.cfg.k)
        upd = self.upd_host(b)
        if upd is None:
            z = np.zeros(0, np.int32)
            upd = (z, z, np.zeros(0), z, None)
        efeat = self.efeat
        roots = (nodes, times) + nb
        if self.compact:
            # the oracle indexes the feature table by event id: hand it only the rows this step touches,
            # with ids renumbered monotonically (the (t, eid) order of the reduction is unchanged)
            ids = np.unique(np.concatenate([np.asarray(upd[3], np.int64), nb[1][nb[1] >= 0].astype(np.int64)]))
            efeat = self._to_host(self.efeat_dev[torch.from_numpy(ids).cuda()])
            remap = lambda e: np.where(e >= 0, np.searchsorted(ids, np.maximum(e, 0)), -1).astype(np.int32)
            upd = (upd[0], upd[1], upd[2], remap(np.asarray(upd[3])), upd[4])
            roots = (nodes, times, nb[0], remap(nb[1]), nb[2], nb[3])
        kw = {}
        if gates is not None:
            kw = dict(h_gate=gates[0], hid_gate=gates[1], gate_eps=GATE_EPS[self.math])
        res = o.loss_and_grads(self.ocfg, pre["params"], pre["memory"], pre["last_update"], efeat, upd,
                               roots, len(t_src), loss_mask, want_grads=want_grads, **kw)
        return res, roots

    def check_step(self, b, pre, res, what=""):
        """Compare the GPU's post-step state with the oracle's result from `pre`."""
        tr, o, tol = self.tr, self.oracle, self.tol
        torch.cuda.synchronize()
        assert tr.lib.status() == 0
        mem = tr.memory.cpu().numpy()
        lu = tr.last_update.cpu().numpy()
        assert np.array_equal(lu, res.last_update_post), f"{what} last_update"
        untouched = np.ones(self.cfg.num_nodes, bool)
        untouched[res.uniq] = False
        assert np.array_equal(mem[untouched], pre["memory"][untouched].astype(np.float32)), f"{what} untouched rows"
        e = relerr(mem[res.uniq], res.memory_post[res.uniq])
        assert e <= tol, f"{what} memory rows err {e}"
        e = abs(float(tr.loss.item()) - res.loss) / max(abs(res.loss), 1e-6)
        assert e <= tol, f"{what} loss {tr.loss.item()} vs {res.loss}"
        self.check_without_hints(b, pre, res, what)
        g = torch.zeros_like(tr.params)
        tr.lib.debug_get_grads(g)
        g = g.cpu().numpy().astype(np.float64)
        self.check_grads(g, res, what, params=pre["params"])
        e = abs(float(tr.gradnorm.item()) - res.gradnorm) / max(res.gradnorm, 1e-6)
        assert e <= tol, f"{what} gradnorm {tr.gradnorm.item()} vs {res.gradnorm}"
        self.check_adam(g, pre, what)
        self.check_updated_params(pre, res, what)

    def check_without_hints(self, b, pre, res, what=""):
        """The part of the step that needs no ReLU hint -- embeddings, loss, memory rows -- against an oracle
        run that takes every branch by its own fp64 sign; and a bound on how many units of the hinted run
        followed the kernel instead of that sign."""
        tr, tol = self.tr, self.tol
        n_h = res.h.size
        units = n_h + (2 * n_h) // 3
        ov = getattr(res, "gate_overrides", (0, 0))
        if OVERRIDE_LOG:
            with open(OVERRIDE_LOG, "a") as f:
                f.write(f"{what} {self.math} units {units} overrides {ov[0]} {ov[1]}\n")
        assert sum(ov) <= MAX_OVERRIDES(units), f"{what} {ov} of {units} ReLU units took the kernel's branch"
        if self.model == "jodie":
            return
        plain, _ = self.oracle_step(pre, b, None, loss_mask=self._last_mask, want_grads=False)
        h = torch.zeros(res.h.shape, dtype=torch.float32, device="cuda")
        tr.lib.debug_get_embeddings(h)
        torch.cuda.synchronize()
        e = relerr(h.cpu().numpy(), plain.h)
        assert e <= tol, f"{what} embeddings vs unhinted oracle err {e}"
        e = abs(float(tr.loss.item()) - plain.loss) / max(abs(plain.loss), 1e-6)
        assert e <= tol, f"{what} loss {tr.loss.item()} vs unhinted oracle {plain.loss}"
        assert np.array_equal(plain.memory_post, res.memory_post)      # the update never sees a hint

    def b2_term_scale(self, params, res):
        """Sum of the absolute values of the terms whose signed sum is d loss / d b_2 (Eq. 13 through the two
        scores of every target event): sum_j w_j (sigmoid(-s_pos_j) + sigmoid(s_neg_j)), from the oracle's own
        embeddings and the step's parameters."""
        lay, d = self.lay, self.cfg.d
        h = np.asarray(res.h, np.float64)
        nq = h.shape[0] // 3
        W1 = params[lay["w_1"]:lay["w_1"] + 2 * d * d].reshape(d, 2 * d)
        b1, w2, b2 = params[lay["b_1"]:lay["b_1"] + d], params[lay["w_2"]:lay["w_2"] + d], params[lay["b_2"]]
        score = lambda a, b: np.maximum(np.concatenate([a, b], 1) @ W1.T + b1, 0.0) @ w2 + b2
        sp, sn = score(h[:nq], h[nq:2 * nq]), score(h[:nq], h[2 * nq:])
        m = np.ones(nq) if self._last_mask is None else (np.asarray(self._last_mask) != 0).astype(np.float64)
        if m.sum() == 0:
            return 0.0
        sig = lambda x: 1.0 / (1.0 + np.exp(-x))
        return float((m * (sig(-sp) + sig(sn))).sum() / m.sum())

    def check_grads(self, g, res, what="", params=None):
        """A gradient (fp64 copy of the GPU's) against the oracle's, tensor by tensor:
        max|gpu - ref| / max(max|ref|, 1e-6)."""
        tol = self.tol
        for name in self.B.param_names(self.tr.tcfg):
            sl = slice(self.lay[name], self.lay[name] + int(np.prod(self.shapes[name])))
            floor = 1e-6
            if name == "b_2" and params is not None:
                # A single number: the difference of two sums of per-event terms (positive pairs pull it down,
                # negative pairs push it up) that nearly cancel once the scores are balanced, so it has no largest
                # entry of its own to be measured against.  Each term is held to the tolerance, hence the sum to
                # the tolerance times the sum of the terms' magnitudes: that sum is the scale here.
                floor = self.b2_term_scale(params, res)
            if name == "b_k":
                # b_k's gradient is identically zero in exact arithmetic (softmax is shift invariant, so the
                # logit gradients of a root sum to zero); what both sides hold is rounding residue of sums
                # whose terms are as large as the other gradients.  This one tensor is measured on the scale
                # of the gradient as a whole: floor = 1e-3 x largest entry.
                floor = 1e-3 * np.abs(res.grads).max()
            e = float(np.abs(g[sl] - res.grads[sl]).max() / max(np.abs(res.grads[sl]).max(), floor, 1e-6))
            assert e <= tol, f"{what} grad {name} err {e}"

    def check_updated_params(self, pre, res, what=""):
        """The updated parameters against the oracle's own Adam step on the oracle's own gradient.
        Two measures.  (1) The update itself, in units of the learning rate, element by element against what
        the gradient tolerance can move it by: with dg <= tol * max|g_tensor| entering
        m_hat / (sqrt(v_hat) + eps), the update moves by at most (1 - beta1) / (1 - beta1^t) * dg /
        (sqrt(v_hat) + eps) through the first moment and by as much again through the second, so elements
        whose second moment is well away from eps are checked tightly at every step and an element with a
        vanishing gradient history is not checked by this measure (the fed-gradient check covers the kernel's
        arithmetic for those).  (2) The contract's metric on each updated tensor, max|p_gpu - p_ref| /
        max|p_ref|, from step 50 on: in the first steps Adam's normalisation turns every near-zero gradient
        entry into a full +-lr move of either sign, and the zero-initialised bias tensors are then no larger
        than the moves themselves.  b_k is left out of (2): its gradient is rounding residue on both sides
        (it is identically zero in exact arithmetic), so its updates are +-lr noise on both sides at any
        step."""
        tr, o, c = self.tr, self.oracle, self.ocfg
        if res.grads is None:
            return
        p_ref, m_ref, v_ref, st = o.adam(c, res.grads, pre["params"], pre["m"], pre["v"], pre["step"])
        p_gpu = tr.params.cpu().numpy().astype(np.float64)
        bc1, bc2 = 1.0 - c.beta1 ** st, 1.0 - c.beta2 ** st
        denom = np.sqrt(v_ref / bc2) + c.eps
        for name in self.B.param_names(self.tr.tcfg):
            sl = slice(self.lay[name], self.lay[name] + int(np.prod(self.shapes[name])))
            if pre["step"] >= 50 and name != "b_k":
                e = relerr(p_gpu[sl], p_ref[sl])
                assert e <= self.tol, f"{what} updated {name} err {e}"
            gmax = np.abs(res.grads[sl]).max()
            if name == "b_k":
                gmax = max(gmax, 1e-3 * np.abs(res.grads).max())
            if name == "b_2":
                gmax = max(gmax, self.b2_term_scale(pre["params"], res))   # the scale its gradient is held to
            allowed = 2.0 * (1.0 - c.beta1) / bc1 * self.tol * max(gmax, 1e-6) / denom[sl] + 1e-4
            moved = np.abs((p_gpu[sl] - pre["params"][sl]) - (p_ref[sl] - pre["params"][sl])) / c.lr
            worst = float((moved / allowed).max())
            assert worst <= 1.0, f"{what} update of {name}: {worst:.2f} x the bound the gradient tolerance allows"

    def check_adam(self, g, pre, what=""):
        """The GPU's parameter update against the oracle's Adam fed with the gradient g the GPU applied."""
        tr, o = self.tr, self.oracle
        p_ref, m_ref, v_ref, st = o.adam(self.ocfg, g, pre["params"], pre["m"], pre["v"], pre["step"])
        assert int(tr.step_count.item()) == st
        upd_gpu = tr.params.cpu().numpy().astype(np.float64) - pre["params"]
        e = np.abs(upd_gpu - (p_ref - pre["params"])).max() / self.ocfg.lr
        assert e <= 1e-3, f"{what} adam update err {e} (units of lr)"
        assert relerr(tr.adam_m.cpu().numpy(), m_ref) <= 1e-6 and relerr(tr.adam_v.cpu().numpy(), v_ref) <= 1e-6


def same_relu_decisions(ra, rb, b, rows_a=None):
    """Whether two contexts took the same branch at every ReLU of step b (rows_a: boolean mask over ra's scored
    events when ra scores more events than rb).  Two runs from the same state differ in the last bits of the
    forward pass (atomic summation order); a unit whose pre-activation is that close to zero can then be
    differentiated on either branch, which moves cancellation-heavy gradient sums by far more than rounding.
    Both gradients are correct; they are only comparable when the decisions agree."""
    ga, gb = ra.gpu_gates(b), rb.gpu_gates(b)
    if rows_a is not None:
        m = np.asarray(rows_a, bool)
        ga = (ga[0][np.concatenate([m, m, m])], ga[1][np.concatenate([m, m])])
    return all(np.array_equal(x, y) for x, y in zip(ga, gb))


TINY = wl.CONFIGS["tiny"]


@pytest.fixture(scope="module")
def tiny_rig(B, oracle):
    return Rig(B, oracle, TINY)


# ------------------------------------------------------------ step (0) -----
@pytest.mark.parametrize("case", ["uniform", "hub", "mixed", "one", "ragged"])
def test_prune_mask_bit_exact(B, oracle, case):
    rng = np.random.default_rng(21)
    N = 5000
    if case == "uniform":
        n = 600
        src, dst = rng.permutation(N)[:n], rng.permutation(N)[:n]
    elif case == "hub":
        n = 4000
        src, dst = np.zeros(n, np.int64), rng.integers(1, N, n)
    elif case == "one":
        n, src, dst = 1, np.array([7]), np.array([7])
    else:
        n = 1337 if case == "ragged" else 4800
        p = 1.0 / np.arange(1, N + 1) ** 1.3
        p /= p.sum()
        src, dst = rng.choice(N, n, p=p), rng.choice(N, n, p=p)
    eid = rng.permutation(10 * n)[:n]
    aux = (rng.random(n) < 0.3).astype(np.uint8)
    lib = B.Tgnn(B.make_config(N, 32, 16, 10, 2, max_events=5000, max_roots=3000))
    d_src, d_dst, d_eid, d_aux = dev(src, torch.int32), dev(dst, torch.int32), dev(eid, torch.int32), dev(aux)
    keep = torch.zeros(n, dtype=torch.uint8, device="cuda")
    heavy = torch.zeros(1, dtype=torch.int32, device="cuda")
    for force, q32, bidx in [(-1, 1 << 31, 0), (-1, 1 << 31, 5), (1, 1 << 30, 2), (1, 0xFFFFFFFF, 1), (0, 1 << 31, 3)]:
        k_ref, h_ref = oracle.prune_mask(N, src, dst, eid, aux, force_heavy=force, drop_q32=q32, seed=99, batch_idx=bidx)
        lib.prune_mask(d_src, d_dst, d_eid, d_aux, keep, heavy, force_heavy=force, drop_q32=q32, seed=99, batch_idx=bidx)
        assert int(heavy.item()) == h_ref
        assert np.array_equal(keep.cpu().numpy(), k_ref)
        assert k_ref[aux == 0].all()                         # targets are never pruned
    lib.close()


# ------------------------------------------------------------ step (1) -----
def test_sample_recent_bit_exact_tiny_stream(tiny_rig):
    r = tiny_rig
    s = r.stream
    rng = np.random.default_rng(22)
    nodes = np.concatenate([s.src, s.dst, s.neg[:5000], rng.integers(0, TINY.num_nodes, 3001).astype(np.int32)])
    times = np.concatenate([s.t, s.t, s.t[:5000], rng.uniform(-1, s.t[-1] + 5, 3001)])
    _check_sample(r.tr.lib, r.oracle, r.graph, nodes, times, TINY.k)


def test_sample_recent_long_slices_and_ties(B, oracle):
    # one hub with ~40k entries (several 32-way rounds), integer timestamps (ties), queries on and between ties
    rng = np.random.default_rng(23)
    N, E = 50, 40000
    src = np.where(rng.random(E) < 0.9, 0, rng.integers(0, N, E)).astype(np.int32)
    dst = rng.integers(1, N, E).astype(np.int32)
    t = np.cumsum(rng.integers(0, 3, E)).astype(np.float64)
    g = wl.build_tcsr(src, dst, t, N)
    lib = B.Tgnn(B.make_config(N, 32, 16, 10, 2))
    lib.set_graph(*[dev(a) for a in g])
    nodes = rng.integers(0, N, 4099).astype(np.int32)
    nodes[::3] = 0
    times = rng.integers(-1, int(t[-1]) + 3, 4099).astype(np.float64) + rng.choice([0.0, 0.5], 4099)
    _check_sample(lib, oracle, g, nodes, times, 10)
    lib.close()


def _check_sample(lib, oracle, graph, nodes, times, k):
    n = len(nodes)
    nb = torch.full((n, k), 77, dtype=torch.int32, device="cuda")
    ne = torch.full((n, k), 77, dtype=torch.int32, device="cuda")
    nt = torch.full((n, k), 7.0, dtype=torch.float64, device="cuda")
    nc = torch.full((n,), 77, dtype=torch.int32, device="cuda")
    lib.sample_recent(dev(nodes, torch.int32), dev(times, torch.float64), nb, ne, nt, nc)
    ref = oracle.sample_recent(*graph, nodes, times, k)
    for got, want in zip((nb, ne, nt, nc), ref):
        assert np.array_equal(got.cpu().numpy(), want)


# ----------------------------------------------------- steps (2)-(4) -------
def _state_for_parts(r, seed=24):
    """Random non-trivial state uploaded into the rig's trainer."""
    rng = np.random.default_rng(seed)
    c = r.cfg
    mem = (rng.normal(size=(c.num_nodes, c.d)) * 0.5).astype(np.float32)
    lu = (rng.random(c.num_nodes) * r.stream.t[2000]).astype(np.float64)
    r.tr.memory.copy_(dev(mem))
    r.tr.last_update.copy_(dev(lu))
    return mem, lu


def test_time_encoding_over_the_whole_argument_range(B):
    """Phi(dt) from the message builder for time differences from 0 to 5e7 (the large workload's stream
    length) under the workloads' frequencies 1 .. 1e-9 and random phases: the kernel's own range reduction
    followed by the hardware cosine against cos of the same fp32 argument in fp64."""
    c = wl.scaled(TINY, d_e=0)
    from paper_2608_16305_b200 import trainer
    dw = trainer.DeviceWorkload(wl.make_stream(c))
    W = wl.make_weights(c.d, c.d_e, c.seed, bias_scale=0.0)
    rng = np.random.default_rng(8)
    W["time_b"] = (rng.random(c.d) * 6.0 - 3.0).astype(np.float32)
    tr = trainer.Trainer(dw, W)
    n, calls = dw.max_mixed, 24                     # the context's batch capacity, many batches
    dt = np.concatenate([[0.0, 1e-3, 3.14159265, 6.2831853, 5e7], rng.random(n * calls - 5) * 10.0 ** rng.uniform(0, 7.7, n * calls - 5)])
    src = torch.arange(n, dtype=torch.int32, device="cuda") % c.num_nodes
    dst = (src + 1) % c.num_nodes
    eid = torch.zeros(n, dtype=torch.int32, device="cuda")
    tr.last_update.zero_()
    parts = []
    for i in range(calls):
        msg = torch.zeros((2 * n, c.d_msg), dtype=torch.float32, device="cuda")
        node = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
        tr.lib.build_messages(src, dst, dev(dt[i * n:(i + 1) * n].astype(np.float64)), eid, None, msg, node)
        torch.cuda.synchronize()
        parts.append(msg.cpu().numpy()[:, 2 * c.d + c.d_e:])
    phi = np.concatenate(parts)
    # the argument is one fused multiply-add in fp32: w * dt + b rounded once
    arg = (W["time_w"].astype(np.float64)[None, :] * np.repeat(dt, 2).astype(np.float32).astype(np.float64)[:, None]
           + W["time_b"].astype(np.float64)[None, :]).astype(np.float32).astype(np.float64)
    assert np.abs(arg).max() > 4e7
    assert np.abs(phi - np.cos(arg)).max() <= 2e-6


def test_messages_reduction_and_gru_by_parts(tiny_rig):
    r, o, c = tiny_rig, tiny_rig.oracle, TINY
    tr = r.tr
    mem, lu = _state_for_parts(r)
    P = tr.params.cpu().numpy().astype(np.float64)
    mb = r.dw.mb_host[10]
    n = mb.n
    rng = np.random.default_rng(25)
    keep = (rng.random(n) < 0.85).astype(np.uint8)
    sl = r.dw.mb_slice(10)
    d_src, d_dst, d_t, d_eid = r.dw.mb_src[sl], r.dw.mb_dst[sl], r.dw.mb_t[sl], r.dw.mb_eid[sl]
    d_keep = dev(keep)
    msg = torch.zeros((2 * n, c.d_msg), dtype=torch.float32, device="cuda")
    node = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    tr.lib.build_messages(d_src, d_dst, d_t, d_eid, d_keep, msg, node)
    msg_ref, node_ref = o.build_messages(r.ocfg, P, mem, lu, r.efeat, mb.src, mb.dst, mb.t, mb.eid, keep)
    assert np.array_equal(node.cpu().numpy(), node_ref)
    got = msg.cpu().numpy()
    assert np.array_equal(got[:, :2 * c.d + c.d_e], msg_ref[:, :2 * c.d + c.d_e].astype(np.float32))   # pure gathers
    assert np.abs(got[:, 2 * c.d + c.d_e:] - msg_ref[:, 2 * c.d + c.d_e:]).max() <= 2e-6                # cos in fp32
    # reduction
    uniq = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    win = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    tr.lib.reduce_latest(node, d_t, d_eid, uniq, win, nu)
    u_ref, w_ref = o.reduce_latest(node_ref, mb.t, mb.eid, c.num_nodes)
    U = int(nu.item())
    assert U == len(u_ref)
    assert np.array_equal(uniq[:U].cpu().numpy(), u_ref) and np.array_equal(win[:U].cpu().numpy(), w_ref)
    # GRU from the materialised rows, then (fresh state) from virtual rows: same result
    mem_ref, lu_ref = o.memory_update(r.ocfg, P, msg_ref, mb.t, u_ref, w_ref, mem, lu)
    for virtual in (False, True):
        tr.memory.copy_(dev(mem))
        tr.last_update.copy_(dev(lu))
        if virtual:
            tr.lib.build_messages(d_src, d_dst, d_t, d_eid, d_keep, None, node)
            tr.lib.reduce_latest(node, d_t, d_eid, uniq, win, nu)
        tr.lib.memory_update(None if virtual else msg, uniq, win, nu)
        got_m, got_lu = tr.memory.cpu().numpy(), tr.last_update.cpu().numpy()
        assert np.array_equal(got_lu, lu_ref)
        assert relerr(got_m[u_ref], mem_ref[u_ref]) <= r.tol
        rest = np.setdiff1d(np.arange(c.num_nodes), u_ref)
        assert np.array_equal(got_m[rest], mem[rest])


@pytest.mark.parametrize("case", ["ties_unsorted", "hub", "sorted_hub", "all_dropped", "empty"])
def test_reduce_latest_bit_exact(B, oracle, case):
    rng = np.random.default_rng(26)
    N = 3000
    lib = B.Tgnn(B.make_config(N, 32, 16, 10, 2, max_events=6000, max_roots=3000))
    if case == "empty":
        n = 0
    elif case in ("hub", "sorted_hub"):
        n = 5200
    else:
        n = 777
    src = rng.integers(0, N, n).astype(np.int32)
    dst = rng.integers(0, N, n).astype(np.int32)
    if case in ("hub", "sorted_hub"):
        src[rng.random(n) < 0.6] = 5
        dst[rng.random(n) < 0.3] = 5
    t = rng.integers(0, 40, n).astype(np.float64) - (3.0 if case == "ties_unsorted" else 0.0)   # ties, unsorted, some negative
    eid = rng.permutation(3 * n + 1)[:n].astype(np.int32)
    if case == "sorted_hub":          # a batch sorted by (t, eid), as mixed batches are: the shared-memory fast path
        t, eid = np.sort(t), np.sort(eid)
    node = np.stack([src, dst], 1).reshape(-1).astype(np.int32)
    drop = np.repeat(rng.random(n) < (1.0 if case == "all_dropped" else 0.2), 2)
    node[drop] = -1
    u_ref, w_ref = oracle.reduce_latest(node, t, eid, N)
    uniq = torch.zeros(max(2 * n, 1), dtype=torch.int32, device="cuda")
    win = torch.zeros(max(2 * n, 1), dtype=torch.int32, device="cuda")
    nu = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    for rep in range(2):                                     # second call: the scratch tables were left clean
        lib.reduce_latest(dev(node), dev(t), dev(eid), uniq, win, nu)
        U = int(nu.item())
        assert U == len(u_ref)
        assert np.array_equal(uniq[:U].cpu().numpy(), u_ref) and np.array_equal(win[:U].cpu().numpy(), w_ref)
    lib.close()


# ------------------------------------------------------------ step (5) -----
def test_embed_by_parts(tiny_rig):
    r, o, c = tiny_rig, tiny_rig.oracle, TINY
    tr = r.tr
    mem, _ = _state_for_parts(r, seed=27)
    P = tr.params.cpu().numpy().astype(np.float64)
    s = r.stream
    q = slice(6000, 6190)
    nodes = np.concatenate([s.src[q], s.dst[q], s.neg[q], s.src[:7]])       # ragged count, early events with cnt < k
    times = np.concatenate([s.t[q]] * 3 + [s.t[:7]])
    nb = o.sample_recent(*r.graph, nodes, times, c.k)
    assert (nb[3] == 0).any() and (nb[3] == c.k).any()
    h = torch.zeros((len(nodes), c.d), dtype=torch.float32, device="cuda")
    tr.lib.embed(dev(nodes), dev(times), dev(nb[0]), dev(nb[1]), dev(nb[2]), dev(nb[3]), h)
    h_ref = o.embed(r.ocfg, P, mem, r.efeat, nodes, times, *nb)
    assert relerr(h.cpu().numpy(), h_ref) <= r.tol
    # the call recorded an embedding of 577 rows: a backward with a mismatching n_q is rejected on the host
    rc = tr.lib.call_raw("tgnn_backward_step", 200, None, None, None, None)
    assert rc == B_ESHAPE


B_ESHAPE = -2


# ------------------------------------------------- whole step, teacher-forced
def _run_epoch_checks(rig, steps, check_at):
    for b in steps:
        pre = rig.snapshot() if b in check_at else None
        rig.tr.step(b)
        if pre is not None:
            res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b))
            rig.check_step(b, pre, res, what=f"[{rig.cfg.name} batch {b}]")


@pytest.mark.parametrize("math", ["fp32", "tf32", "f16x3"])
def test_tiny_epoch_teacher_forced(B, oracle, math):
    rig = Rig(B, oracle, TINY, math=math)
    nb = TINY.num_batches
    _run_epoch_checks(rig, range(nb), {0, 1, 2, 3, 10, 37, nb // 2, nb - 2, nb - 1})
    assert rig.tr.lib.kernel_launches() > 0


def test_tiny_default_init_zero_biases(B, oracle):
    rig = Rig(B, oracle, TINY, bias_scale=0.0)
    _run_epoch_checks(rig, range(0, 6), {0, 1, 5})


def _scaled(name, events, **kw):
    c = wl.CONFIGS[name]
    return wl.scaled(c, num_events=events, **kw)


@pytest.mark.parametrize("math", ["fp32", "tf32", "f16x3"])
@pytest.mark.parametrize("name,events,at", [
    ("wiki", 6000, {1, 5, 9}),          # 172-d features, d = 100: ragged tiles everywhere
    ("reddit", 9000, {2, 8, 14}),       # replay events + pruning
    ("lastfm", 24000, {1, 3, 5}),       # no edge features, heavy skew, batch 4000
])
def test_scaled_configs_teacher_forced(B, oracle, name, events, at, math):
    rig = Rig(B, oracle, _scaled(name, events), math=math)
    _run_epoch_checks(rig, range(rig.cfg.num_batches), at)
    if rig.cfg.prune:
        heavy = rig.dw.heavy.cpu().numpy()
        keep = rig.dw.mb_keep.cpu().numpy()
        aux = rig.dw.mb_aux.cpu().numpy()
        assert keep[aux == 0].all()
        # pruning really happened on heavy batches and only there
        for i, b in enumerate(rig.dw.batches):
            s = rig.dw.mb_slice(b)
            mb = rig.dw.mb_host[i]
            k_ref, h_ref = rig.oracle.prune_mask(rig.cfg.num_nodes, mb.src, mb.dst, mb.eid, mb.is_aux, seed=rig.cfg.seed,
                                                 batch_idx=b)
            assert h_ref == heavy[i] and np.array_equal(keep[s], k_ref)


def test_rebinding_state_after_graph_replay_has_started(B, oracle):
    """A recorded step graph has the state pointers baked into its kernel arguments.  After tgnn_set_state with
    other buffers the library must record new graphs: the step runs on the new buffers (parity with the oracle
    from their contents) and never touches the old ones (poisoned here)."""
    rig = Rig(B, oracle, _scaled("wiki", 6000), math="tf32")
    tr = rig.tr
    for b in range(4):                       # from the third call on, steps of this shape replay a graph
        tr.step(b)
    torch.cuda.synchronize()
    old = (tr.memory, tr.last_update, tr.params, tr.adam_m, tr.adam_v, tr.step_count)
    new = tuple(x.clone() for x in old)
    tr.memory, tr.last_update, tr.params, tr.adam_m, tr.adam_v, tr.step_count = new
    tr.lib.set_state(*new)
    for x in old[:5]:
        x.fill_(float("nan"))
    old[5].fill_(-12345)
    for b in range(4, 8):                    # plain launches, capture, then replay on the new buffers
        pre = rig.snapshot()
        tr.step(b)
        res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b))
        rig.check_step(b, pre, res, what=f"[rebound state, batch {b}]")
    assert all(bool(torch.isnan(x).all()) for x in old[:5]) and int(old[5].item()) == -12345


@pytest.mark.parametrize("math", ["fp32", "tf32"])
@pytest.mark.parametrize("d,batch", [
    (160, 150),   # W_1 no longer fits in shared memory: the head runs as separate projection kernels
    (100, 150),   # fused head, last group of 4 events ragged (150 = 37 * 4 + 2)
    (32, 2501),   # fused head walking several groups per block; odd batch
])
def test_head_paths_wide_and_ragged(B, oracle, math, d, batch):
    c = wl.scaled(wl.CONFIGS["wiki"], num_events=4 * batch, num_nodes=1200, num_src=1000, d=d, batch=batch)
    rig = Rig(B, oracle, c, math=math)
    _run_epoch_checks(rig, range(4), {1, 3})


@pytest.mark.parametrize("math", ["fp32", "tf32", "f16x3"])
def test_bf16_feature_table(B, oracle, math):
    c = wl.scaled(wl.CONFIGS["large"], num_events=20000, num_nodes=3000, batch=1000)
    rig = Rig(B, oracle, c, math=math)
    _run_epoch_checks(rig, range(8), {1, 4, 7})


def test_adaptive_controller_drives_pruning(B, oracle):
    """Algorithm 2 end to end: the library's controller decides H_r from the batch times it is fed, a heavy
    batch loses every pure replay event (Eq. 10-11) and nothing else, the next step's memory update uses
    exactly the kept events, and the decisions equal the oracle controller's on the same measurements."""
    from oracle import controller as oc
    rig = Rig(B, oracle, _scaled("reddit", 9000))
    alpha, beta, tau_g, tau_c, K = 0.1, 0.1, 1.6, 1.5, 3
    ctl = B.Controller(alpha, beta, tau_g, tau_c, K)
    ref = oc.ControllerOracle(alpha, beta, tau_g, tau_c, K)
    nb = rig.cfg.num_batches
    times = [1.0] * nb
    times[3] = 4.0          # a straggling batch: the one after it runs in heavy-load mode
    times[9] = 3.0
    heavy_seen = []
    for b in range(nb):
        pre = rig.snapshot() if b in (4, 5, 10) else None
        log = rig.tr.step_adaptive(b, ctl, batch_time=times[b])
        bd, s, h = ref.begin_batch(b)
        assert (log["boundary"], log["sync"], log["heavy"]) == (bd, -1 if s is None else s, h), b
        ref.end_batch(log["g"], times[b])
        assert ctl.state() == (ref.g_bar, ref.g_last, ref.c_bar, ref.c_prev)
        heavy_seen.append(h)
        torch.cuda.synchronize()
        mb = rig.dw.mb_host[b]
        keep = rig.dw.mb_keep[rig.dw.mb_slice(b)].cpu().numpy()
        k_ref, _ = oracle.prune_mask(rig.cfg.num_nodes, mb.src, mb.dst, mb.eid, mb.is_aux, seed=rig.cfg.seed, batch_idx=b,
                                     force_heavy=h, drop_q32=0xFFFFFFFF)
        assert np.array_equal(keep, k_ref), b
        assert np.array_equal(keep, (mb.is_aux == 0) if h else np.ones_like(keep)), b
        if pre is not None:   # steps 5 and 10 update memory from the pruned batches 4 and 9... and 4 from the unpruned 3
            res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b))
            rig.check_step(b, pre, res, what=f"[adaptive batch {b}]")
    assert heavy_seen[4] == 1 and heavy_seen[10] == 1 and sum(heavy_seen) == 2
    assert any(m.is_aux.any() for m in rig.dw.mb_host[4:5])   # the heavy batch did have replay events to lose


@pytest.mark.parametrize("p", [0, 2])
def test_partitioned_worker_steps_on_scanned_mixed_batches(B, oracle, p):
    """Worker p of a 3-way node partition trains on the mixed batches that the backward dependency scan
    (Algorithm 1) built on the device: its targets are the source-owned events (variable count per batch),
    the memory update replays targets and auxiliary events alike, and each step matches the oracle."""
    cfg = _scaled("reddit", 7200)
    owner = (np.arange(cfg.num_nodes) * 2654435761 % 2 ** 32 % 3).astype(np.int32)
    rig = Rig(B, oracle, cfg, math="tf32", partition=(owner, 3, p, 4))
    dw = rig.dw
    src, dst = rig.stream.src, rig.stream.dst
    for b in range(cfg.num_batches):
        mb = dw.mb_host[b]
        assert np.array_equal(owner[src[mb.eid]] != p, mb.is_aux == 1)           # the event-type mask is the ownership test
        assert np.array_equal(dw.targets_host(b)[0], mb.src[mb.is_aux == 0])     # targets = the non-auxiliary events, in order
        assert np.all(np.diff(mb.t) >= 0)                                        # timestamp order (Eq. 5)
    assert sum(int(m.is_aux.sum()) for m in dw.mb_host) > 0
    _run_epoch_checks(rig, range(cfg.num_batches), {1, 4, 7, cfg.num_batches - 1})


# ------------------------------------------------- gradient synchronisation across workers
def test_deferred_gradient_then_apply_equals_the_fused_step(B, oracle):
    """With gradient synchronisation on, a step leaves its complete gradient in the context's buffer and
    touches neither parameters nor Adam state; tgnn_apply_gradient then finishes it.  Against a second
    context that runs the fused step from the same state: same gradient, same loss, same norm; the applied
    update is the oracle's Adam on scale x the buffer.  Steps are replayed as CUDA graphs from the third on."""
    cfg = _scaled("reddit", 9000)
    a = Rig(B, oracle, cfg, math="tf32")
    b = Rig(B, oracle, cfg, math="tf32")
    b.tr.lib.set_grad_sync(True)
    names = ("memory", "last_update", "params", "adam_m", "adam_v", "step_count")
    for step in range(8):
        for name in names:
            getattr(b.tr, name).copy_(getattr(a.tr, name))
        pre = b.snapshot()
        a.tr.step(step)
        b.tr.step(step)
        torch.cuda.synchronize()
        assert np.array_equal(b.tr.params.cpu().numpy(), pre["params"].astype(np.float32))
        assert int(b.tr.step_count.item()) == pre["step"] and np.array_equal(b.tr.adam_m.cpu().numpy(), pre["m"].astype(np.float32))
        ga = torch.zeros_like(a.tr.params)
        a.tr.lib.debug_get_grads(ga)
        gb = b.tr.lib.grad_buffer()
        assert gb.numel() == ga.numel()
        assert abs(float(b.tr.loss.item()) - float(a.tr.loss.item())) <= 1e-5 * abs(float(a.tr.loss.item()))
        if same_relu_decisions(a, b, step):
            assert relerr(gb.cpu().numpy(), ga.cpu().numpy()) <= 1e-4
            assert abs(float(b.tr.gradnorm.item()) - float(a.tr.gradnorm.item())) <= 1e-4 * float(a.tr.gradnorm.item())
        assert relerr(b.tr.memory.cpu().numpy(), a.tr.memory.cpu().numpy()) <= 1e-5
        # a new step while the gradient is pending is refused on the host
        with pytest.raises(B.TgnnError) as ei:
            b.tr.lib.train_step(None, None, None, None, None, *b.dw.targets(step), None, b.tr.loss, b.tr.gradnorm)
        assert ei.value.code == B.TGNN_ESTATE
        scale = 1.0 if step % 2 == 0 else 0.5
        g_local = gb.cpu().numpy().astype(np.float64)
        b.tr._run(lambda: b.tr.lib.apply_gradient(scale, b.tr.gradnorm))
        torch.cuda.synchronize()
        g_applied = b.tr.lib.grad_buffer().cpu().numpy().astype(np.float64)
        assert np.array_equal(g_applied, g_local * scale)                     # the product is stored (exact for 1 and 1/2)
        want = np.sqrt(np.sum(g_applied * g_applied))
        assert abs(float(b.tr.gradnorm.item()) - want) <= 1e-6 * want
        b.check_adam(g_applied, pre, what=f"[deferred step {step}]")
        with pytest.raises(B.TgnnError):
            b.tr.lib.apply_gradient(1.0, b.tr.gradnorm)                       # nothing pending any more
    with pytest.raises(B.TgnnError):
        a.tr.lib.apply_gradient(1.0, a.tr.gradnorm)                           # fused mode has nothing to apply
    # back to the fused form: the next step applies Adam by itself again
    b.tr.lib.set_grad_sync(False)
    st = int(b.tr.step_count.item())
    b.tr.step(8)
    torch.cuda.synchronize()
    assert int(b.tr.step_count.item()) == st + 1


def test_two_emulated_workers_with_synchronised_gradient_match_oracle(B, oracle):
    """Two workers of a 2-way node partition on one device, run one after the other: each steps on its
    scanned mixed batch up to the gradient, the all-reduce is written out (both buffers receive the sum),
    each applies the mean.  Local gradients match the oracle's per worker, g_r matches the norm of the
    oracle's mean gradient and is the same number on both, the update is Adam on the mean, and the two
    replicas of the parameters stay bitwise identical."""
    from oracle import refresh as orf
    cfg = _scaled("reddit", 7200)
    owner = (np.arange(cfg.num_nodes) * 2654435761 % 2 ** 32 % 2).astype(np.int32)
    rigs = [Rig(B, oracle, cfg, math="tf32", partition=(owner, 2, p, 4)) for p in range(2)]
    for r in rigs:
        r.tr.lib.set_grad_sync(True)
    check = {1, 4, 9, cfg.num_batches - 1}
    for b in range(cfg.num_batches):
        pres = [r.snapshot() for r in rigs] if b in check else None
        for r in rigs:
            r.tr.step(b)
        bufs = [r.tr.lib.grad_buffer() for r in rigs]
        local = [x.clone() for x in bufs]
        losses = [float(r.tr.loss.item()) for r in rigs]
        total = bufs[0] + bufs[1]
        for r, buf in zip(rigs, bufs):
            buf.copy_(total)
            r.tr._run(lambda r=r: r.tr.lib.apply_gradient(0.5, r.tr.gradnorm))
        torch.cuda.synchronize()
        for name in ("params", "adam_m", "adam_v", "step_count"):
            assert torch.equal(getattr(rigs[0].tr, name), getattr(rigs[1].tr, name)), (b, name)
        assert float(rigs[0].tr.gradnorm.item()) == float(rigs[1].tr.gradnorm.item())
        if pres is not None:
            res = [r.oracle_step(pre, b, r.gpu_gates(b))[0] for r, pre in zip(rigs, pres)]
            for p, r in enumerate(rigs):
                r.check_grads(local[p].cpu().numpy().astype(np.float64), res[p], what=f"[worker {p} batch {b}]",
                              params=pres[p]["params"])
                assert abs(losses[p] - res[p].loss) <= r.tol * max(abs(res[p].loss), 1e-6)
                assert relerr(r.tr.memory.cpu().numpy()[res[p].uniq], res[p].memory_post[res[p].uniq]) <= r.tol
            mean, g = orf.synchronised_gradient([x.grads for x in res])
            assert abs(float(rigs[0].tr.gradnorm.item()) - g) <= rigs[0].tol * g
            applied = bufs[0].cpu().numpy().astype(np.float64)
            assert np.array_equal(applied, (total * 0.5).cpu().numpy().astype(np.float64))
            for r, pre in zip(rigs, pres):
                r.check_adam(applied, pre, what=f"[synchronised batch {b}]")


def test_distributed_step_of_a_single_worker_runs_refresh_decisions_and_applies_its_own_gradient(B, oracle):
    """Trainer.step_distributed without a process group: the controller's boundary decisions are taken, the
    refresh callback runs exactly at the executed boundaries with the window index, the gradient hook sees
    the context's buffer, and the step equals the fused step of a second context."""
    cfg = _scaled("reddit", 9000)
    a = Rig(B, oracle, cfg, math="tf32")
    b = Rig(B, oracle, cfg, math="tf32")
    b.tr.lib.set_grad_sync(True)
    ctl = B.Controller(alpha=0.1, beta=0.1, tau_g=1.6, tau_c=1e9, K=3)

    class Probe:
        def __init__(self):
            self.calls = []

        def run(self, q, memory, last_update):
            self.calls.append(q)
    probe, seen, logs = Probe(), [], []

    def reduce(buf):
        seen.append(buf.data_ptr())
        return 1
    for step in range(10):
        for name in ("memory", "last_update", "params", "adam_m", "adam_v", "step_count"):
            getattr(b.tr, name).copy_(getattr(a.tr, name))
        pre = b.snapshot()
        a.tr.step(step, force_heavy=0)
        logs.append(b.tr.step_distributed(step, ctl, refresh=probe, reduce_gradient=reduce, batch_time=1.0))
        torch.cuda.synchronize()
        if same_relu_decisions(a, b, step):
            assert abs(float(b.tr.gradnorm.item()) - float(a.tr.gradnorm.item())) <= 1e-4 * float(a.tr.gradnorm.item())
        b.check_adam(b.tr.lib.grad_buffer().cpu().numpy().astype(np.float64), pre, what=f"[step {step}]")
    assert [l["boundary"] for l in logs] == [1 if r % 3 == 0 else 0 for r in range(10)]
    assert probe.calls == [l["r"] // 3 for l in logs if l["boundary"] and l["sync"]] and 0 in probe.calls
    assert len(set(seen)) == 1 and len(seen) == 10


# ------------------------------------------------- masked loss (Eq. 12-13)
@pytest.mark.parametrize("model", ["tgn", "jodie"])
@pytest.mark.parametrize("mask_kind", ["random", "none_set", "one_set"])
def test_masked_loss_with_caller_mask(B, oracle, model, mask_kind):
    """The step under an arbitrary target mask: masked events add nothing to the loss or to any gradient,
    the mean runs over the unmasked ones, and a mask with no event set gives loss 0, a zero gradient and an
    Adam step on a zero gradient (the memory update of the previous batch still happens)."""
    rig = Rig(B, oracle, TINY, model=model)
    tr, dw = rig.tr, rig.dw
    rng = np.random.default_rng(5)
    for b in range(4):
        nq = len(dw.targets_host(b)[0])
        mask = {"random": (rng.random(nq) < 0.4), "none_set": np.zeros(nq, bool),
                "one_set": np.arange(nq) == nq // 3}[mask_kind].astype(np.uint8)
        pre = rig.snapshot()
        u = dw.mb_slice(b - 1) if b > 0 else None
        upd = (dw.mb_src[u], dw.mb_dst[u], dw.mb_t[u], dw.mb_eid[u], dw.mb_keep[u]) if b > 0 else (None,) * 5
        m_dev = torch.from_numpy(mask).cuda()
        tr._run(lambda: tr.lib.train_step(*upd, *dw.targets(b), m_dev, tr.loss, tr.gradnorm))
        res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b), loss_mask=mask)
        rig.check_step(b, pre, res, what=f"[{model} {mask_kind} batch {b}]")
        if mask_kind == "none_set":
            assert float(tr.loss.item()) == 0.0 and float(tr.gradnorm.item()) == 0.0


@pytest.mark.parametrize("math", ["fp32", "tf32"])
def test_every_event_scored_under_the_target_mask(B, oracle, math):
    """embed_aux: every event of the mixed batch is a root (auxiliary events too, the costing in which replay
    events pay the forward pass) and Eq. 13 weighs auxiliary events 0.  Each step matches the oracle on the
    same roots and mask, and loss and gradient norm equal those of the target-only path from the same state."""
    cfg = _scaled("reddit", 9000)
    rig = Rig(B, oracle, cfg, math=math, embed_aux=True)
    ref = Rig(B, oracle, cfg, math=math)
    assert rig.tr.tcfg.embed_aux == 1 and rig.dw.max_targets == cfg.max_mixed
    for b in range(cfg.num_batches):
        mb = rig.dw.mb_host[b]
        assert len(rig.dw.targets_host(b)[0]) == mb.n and int(rig.dw.loss_mask_host(b).sum()) == int((mb.is_aux == 0).sum())
        for name in ("memory", "last_update", "params", "adam_m", "adam_v", "step_count"):
            getattr(ref.tr, name).copy_(getattr(rig.tr, name))
        pre = rig.snapshot() if b in {1, 6, 13} else None
        rig.tr.step(b)
        ref.tr.step(b)
        torch.cuda.synchronize()
        if pre is not None:
            res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b))
            rig.check_step(b, pre, res, what=f"[embed_aux batch {b}]")
        tol = 1e-5 if math == "fp32" else 1e-4
        assert abs(float(rig.tr.loss.item()) - float(ref.tr.loss.item())) <= tol * abs(float(ref.tr.loss.item())), b
        if same_relu_decisions(rig, ref, b, rows_a=rig.dw.loss_mask_host(b)):
            assert abs(float(rig.tr.gradnorm.item()) - float(ref.tr.gradnorm.item())) <= 10 * tol * float(ref.tr.gradnorm.item()), b
        assert np.array_equal(rig.tr.last_update.cpu().numpy(), ref.tr.last_update.cpu().numpy())
    assert sum(int(m.is_aux.sum()) for m in rig.dw.mb_host) > 0


def test_partitioned_worker_scoring_every_event(B, oracle):
    """The scanned mixed batches of one worker with every event scored: roots and mask come from the
    device-built batch (the negatives by event id), and the steps match the oracle."""
    cfg = _scaled("reddit", 7200)
    owner = (np.arange(cfg.num_nodes) * 2654435761 % 2 ** 32 % 3).astype(np.int32)
    rig = Rig(B, oracle, cfg, math="tf32", partition=(owner, 3, 1, 4), embed_aux=True)
    for b in range(cfg.num_batches):
        mb = rig.dw.mb_host[b]
        s, d, n, t = rig.dw.targets_host(b)
        assert np.array_equal(s, mb.src) and np.array_equal(n, rig.stream.neg[mb.eid])
        assert np.array_equal(rig.dw.loss_mask_host(b), 1 - mb.is_aux)
    _run_epoch_checks(rig, range(cfg.num_batches), {2, 5, cfg.num_batches - 1})



@pytest.mark.parametrize("math", ["fp32", "tf32"])
@pytest.mark.parametrize("name,events,at", [
    ("tiny", 4000, {0, 1, 2, 7, 19}),
    ("wiki", 6000, {1, 5, 9}),
    ("reddit", 9000, {2, 8, 14}),       # replay events + pruning
    ("lastfm", 24000, {1, 3, 5}),       # no edge features, batch 4000
])
def test_jodie_variant_teacher_forced(B, oracle, name, events, at, math):
    """The paper's second model: recurrent-cell memory update and time-projected embedding, same head, loss and Adam."""
    from oracle import jodie as oj
    rig = Rig(B, oracle, _scaled(name, events), math=math, model="jodie")
    lay = oj.param_layout(rig.cfg.d, rig.cfg.d_e)
    assert all(rig.lay[n] == lay[n] for n in oj.PARAM_NAMES) and rig.lay["total"] == lay["total"]
    _run_epoch_checks(rig, range(rig.cfg.num_batches), at)
    assert rig.tr.lib.kernel_launches() > 0


def test_jodie_by_parts_and_wide_model(B, oracle):
    """Entry point by entry point (no whole-step call), a model too wide for the fused head, and the embedding alone."""
    from oracle import jodie as oj
    c = wl.scaled(wl.CONFIGS["wiki"], num_events=1200, num_nodes=1200, num_src=1000, d=160, batch=300)
    rig = Rig(B, oracle, c, math="tf32", model="jodie")
    _run_epoch_checks(rig, range(4), {1, 3})
    # the embedding entry point with the neighbor arrays left out
    tr, s = rig.tr, rig.stream
    nodes = dev(np.concatenate([s.src[:50], s.dst[:50]]), torch.int32)
    times = dev(np.full(100, s.t[-1] + 3.5), torch.float64)
    h = torch.zeros((100, c.d), dtype=torch.float32, device="cuda")
    tr.lib.embed(nodes, times, None, None, None, None, h)
    torch.cuda.synchronize()
    W = oj.unpack(c.d, c.d_e, tr.params.cpu().numpy().astype(np.float64))
    mem, lu = tr.memory.cpu().numpy().astype(np.float64), tr.last_update.cpu().numpy()
    n = nodes.cpu().numpy()
    dt = (times.cpu().numpy() - lu[n]).astype(np.float32).astype(np.float64)
    assert relerr(h.cpu().numpy(), oj.time_projection(mem[n], dt, W["proj_w"], W["proj_b"])) <= 1e-6


def test_host_buffer_entry_point_matches_device_path(B, oracle):
    a = Rig(B, oracle, TINY)
    b = Rig(B, oracle, TINY)
    loss = torch.zeros(1).pin_memory()
    gn = torch.zeros(1).pin_memory()
    for step in range(4):
        a.tr.step(step)
        b.tr.prune(step)
        q = b.dw.target_slice(step)
        s = b.stream
        pin = lambda x: torch.from_numpy(np.ascontiguousarray(x)).pin_memory()
        upd = b.upd_host(step)
        upd = tuple(pin(x) for x in upd) if upd is not None else (None,) * 5
        b.tr.lib.train_step_host(*upd, pin(s.src[q]), pin(s.dst[q]), pin(s.neg[q]), pin(s.t[q]), None, loss, gn)
        torch.cuda.synchronize()
        assert abs(float(loss.item()) - float(a.tr.loss.item())) <= 1e-5 * abs(float(loss.item()))
        assert abs(float(gn.item()) - float(a.tr.gradnorm.item())) <= 1e-5 * abs(float(gn.item()))
    # atomics make float sums order-dependent: compare within rounding, not bitwise
    assert relerr(b.tr.memory.cpu().numpy(), a.tr.memory.cpu().numpy()) <= 2e-3
    assert relerr(b.tr.params.cpu().numpy(), a.tr.params.cpu().numpy()) <= 2e-3


@pytest.mark.parametrize("embed_aux", [False, True])
def test_streaming_host_entry_point_matches_device_path(B, oracle, embed_aux):
    # replay + pruning workload: the streaming call keeps each batch (and its prune mask) on the device for the
    # next call, so agreement over several steps checks the slot hand-over and the mask as well; with every
    # event scored the call also builds the roots and the target mask of the whole mixed batch
    cfg = _scaled("reddit", 9000)
    a = Rig(B, oracle, cfg, math="tf32", embed_aux=embed_aux)
    b = Rig(B, oracle, cfg, math="tf32", embed_aux=embed_aux)
    loss = torch.zeros(1).pin_memory()
    gn = torch.zeros(1).pin_memory()
    for step in range(cfg.num_batches):
        # two training runs drift apart chaotically (atomics order -> rounding -> Adam), so the second run is
        # put on the first one's state before every step; its previous batch and prune mask remain its own
        for name in ("memory", "last_update", "params", "adam_m", "adam_v", "step_count"):
            getattr(b.tr, name).copy_(getattr(a.tr, name))
        torch.cuda.synchronize()
        a.tr.step(step)
        b.tr.step_host(step, b.tr.host_batch(step), loss, gn)
        torch.cuda.synchronize()
        assert abs(float(loss.item()) - float(a.tr.loss.item())) <= 1e-5 * abs(float(loss.item())), step
        if same_relu_decisions(a, b, step):
            assert abs(float(gn.item()) - float(a.tr.gradnorm.item())) <= 1e-4 * abs(float(gn.item())), step
        assert np.array_equal(b.tr.last_update.cpu().numpy(), a.tr.last_update.cpu().numpy())   # same events kept
        assert relerr(b.tr.memory.cpu().numpy(), a.tr.memory.cpu().numpy()) <= 1e-5
    assert a.dw.heavy.sum().item() > 0


# ------------------------------------------------------------ errors -------
def test_argument_errors_are_reported_not_launched(B):
    lib = B.Tgnn(B.make_config(100, 32, 16, 10, 2, max_events=64, max_roots=96))
    z = torch.zeros(200, dtype=torch.int32, device="cuda")
    zt = torch.zeros(200, dtype=torch.float64, device="cuda")
    zu = torch.zeros(200, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TgnnError) as e:
        lib.sample_recent(z[:10], zt[:10], z, z, zt, z)                    # graph not set
    assert e.value.code == B.TGNN_ESTATE
    with pytest.raises(B.TgnnError) as e:
        lib.prune_mask(z[:100], z[:100], z[:100], zu[:100], zu, z)         # over capacity
    assert e.value.code == B.TGNN_ECAPACITY and "max_events" in str(e.value)
    with pytest.raises(B.TgnnError) as e:
        lib.backward_step(10, None, None, None)                            # nothing embedded
    assert e.value.code == B.TGNN_ESTATE
    assert lib.call_raw("tgnn_prune_mask", None, None, None, None, 5, -1, 0, 0, 0, None, None, None) == B.TGNN_EINVAL
    bad = B.make_config(100, 30, 16, 10, 2)                                  # d not a multiple of 4
    with pytest.raises(B.TgnnError):
        B.Tgnn(bad)
    assert lib.status() == 0
    lib.close()


def test_indices_beyond_the_graph_are_reported_and_never_used(B, oracle):
    """Every gather and scatter checks its indices.  An update event that names a node beyond the graph or a
    feature row beyond the table is reported through the status word (TGNN_EBOUNDS) and treated exactly as if its
    keep flag were 0: the step's result equals, bit for bit, that of a second context given the same batch with
    those events masked out.  A root beyond the graph and a node count beyond the capacity are reported too, and
    nothing outside the arrays involved is touched."""
    cfg = _scaled("wiki", 6000)
    a = Rig(B, oracle, cfg, math="fp32")
    a.tr.lib.set_graph_replay(False)
    for step in range(3):
        a.tr.step(step)
    torch.cuda.synchronize()
    N, E = cfg.num_nodes, cfg.num_events
    u = a.dw.mb_slice(2)
    src, dst, t, eid = (x[u].clone() for x in (a.dw.mb_src, a.dw.mb_dst, a.dw.mb_t, a.dw.mb_eid))
    keep = torch.ones(src.numel(), dtype=torch.uint8, device="cuda")
    bad_src, bad_dst, bad_eid = src.clone(), dst.clone(), eid.clone()
    bad_src[3] = N + 7
    bad_dst[11] = 1 << 30
    bad_eid[5] = E + 3
    masked = keep.clone()
    masked[[3, 5, 11]] = 0
    q = a.dw.targets(3)
    state = (a.tr.memory, a.tr.last_update, a.tr.params, a.tr.adam_m, a.tr.adam_v, a.tr.step_count)
    saved = [x.clone() for x in state]
    a.tr.lib.train_step(bad_src, bad_dst, t, bad_eid, keep, *q, None, a.tr.loss, a.tr.gradnorm)
    torch.cuda.synchronize()
    assert a.tr.lib.status() == B.TGNN_EBOUNDS
    got = [x.clone() for x in state] + [a.tr.loss.clone()]
    a.tr.lib.clear_status()
    for x, y in zip(state, saved):
        x.copy_(y)
    a.tr.lib.train_step(src, dst, t, eid, masked, *q, None, a.tr.loss, a.tr.gradnorm)
    torch.cuda.synchronize()
    assert a.tr.lib.status() == 0
    assert torch.equal(got[1], a.tr.last_update)                                  # the same nodes were updated
    assert relerr(got[0].cpu().numpy(), a.tr.memory.cpu().numpy()) <= 1e-6        # (atomic summation order differs)
    assert abs(float(got[6].item()) - float(a.tr.loss.item())) <= 1e-6 * abs(float(a.tr.loss.item()))
    a.tr.lib.clear_status()
    # a root beyond the graph: reported, the step completes with finite numbers
    qs, qd, qn, qt = (x.clone() for x in a.dw.targets(4))
    qd[7] = N
    v = a.dw.mb_slice(3)
    a.tr.lib.train_step(a.dw.mb_src[v], a.dw.mb_dst[v], a.dw.mb_t[v], a.dw.mb_eid[v], None, qs, qd, qn, qt, None, a.tr.loss,
                        a.tr.gradnorm)
    torch.cuda.synchronize()
    assert a.tr.lib.status() == B.TGNN_EBOUNDS
    assert bool(torch.isfinite(a.tr.loss).all()) and bool(torch.isfinite(a.tr.memory).all())
    a.tr.lib.clear_status()
    # a device-side node count beyond the capacity of the arrays it describes: clamped and reported
    lib = a.tr.lib
    n = 40
    node = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    lib.build_messages(src[:n], dst[:n], t[:n], eid[:n], None, None, node)
    uniq = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    win = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib.reduce_latest(node, t[:n], eid[:n], uniq, win, nu)
    before = a.tr.memory.clone()
    nu.fill_(1_000_000)
    lib.memory_update(None, uniq, win, nu)
    torch.cuda.synchronize()
    assert lib.status() == B.TGNN_EBOUNDS
    touched = torch.zeros(N, dtype=torch.bool, device="cuda")
    touched[uniq.long()] = True
    assert torch.equal(a.tr.memory[~touched], before[~touched])


# ------------------------------------------ full-size workloads, bench launch configuration
# The same teacher-forced comparison at the full sizes of the named workloads, driven the way bench.py drives
# it: tensor-core mode, the whole step replayed as a CUDA graph on a capturable stream.  The oracle
# needs seconds per step at these sizes, so only a few sampled steps are compared; every other step
# still has to keep the device status clean.
def _full_size(B, oracle, cfg, check_at, last, math="tf32"):
    rig = Rig(B, oracle, cfg, math=math, batches=range(0, last + 1), bias_scale=0.0, lr=1e-4)
    for b in range(last + 1):
        pre = rig.snapshot() if b in check_at else None
        rig.tr.step(b)
        if pre is not None:
            res, _ = rig.oracle_step(pre, b, rig.gpu_gates(b))
            rig.check_step(b, pre, res, what=f"[{cfg.name} full size, batch {b}]")
    torch.cuda.synchronize()
    assert rig.tr.lib.status() == 0
    return rig


@pytest.mark.slow
@pytest.mark.parametrize("math", ["tf32", "f16x3"])
def test_wiki_full_size_graph_replay(B, oracle, math):
    cfg = wl.CONFIGS["wiki"]
    rig = _full_size(B, oracle, cfg, {0, 1, 2, 150, cfg.num_batches - 1}, cfg.num_batches - 1, math=math)
    # the last batch is ragged (160000 = 266 * 600 + 400): a different shape signature was captured
    assert cfg.num_events % cfg.batch != 0
    assert rig.tr.lib.kernel_launches() > 30 * cfg.num_batches


@pytest.mark.slow
@pytest.mark.parametrize("math", ["tf32", "f16x3"])
def test_reddit_full_size_replay_and_pruning(B, oracle, math):
    cfg = wl.CONFIGS["reddit"]
    rig = _full_size(B, oracle, cfg, {3, 400}, 400, math=math)
    heavy = rig.dw.heavy.cpu().numpy()
    keep = rig.dw.mb_keep.cpu().numpy()
    aux = rig.dw.mb_aux.cpu().numpy()
    assert keep[aux == 0].all() and 0 < heavy.sum() and (keep[aux == 1] == 0).any()


@pytest.mark.slow
@pytest.mark.parametrize("math", ["tf32", "f16x3"])
def test_lastfm_full_size_hub_contention(B, oracle, math):
    cfg = wl.CONFIGS["lastfm"]
    rig = _full_size(B, oracle, cfg, {2, 60}, 60, math=math)
    top = np.bincount(np.concatenate([rig.stream.src, rig.stream.dst])).max() / (2 * cfg.num_events)
    assert top > 0.3                       # one node takes a third of all endpoint slots


@pytest.mark.slow
@pytest.mark.parametrize("math", ["tf32", "f16x3"])
def test_large_full_size_bf16(B, oracle, math):
    # 17,000 nodes, 50 M events, 18.6 GB of bf16 edge features resident in HBM (generated on the device),
    # batch 4,000, 20 % replay with pruning; about a minute of host set-up (T-CSR over 10^8 entries).  The
    # feature table is too big for a host copy, so the oracle gets the rows each compared step touches.
    cfg = wl.CONFIGS["large"]
    last = cfg.num_batches - 1
    rig = _full_size(B, oracle, cfg, {5, last}, last, math=math)
    assert rig.compact and rig.efeat_dev.numel() * 2 > 18e9
