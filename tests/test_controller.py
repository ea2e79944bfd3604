"""Adaptive runtime controller (Eq. 6-9, Algorithm 2): the oracle against hand-worked values, closed forms
and brute force; then the library's host-side implementation against the oracle through the C ABI."""
import ctypes as C
import os

import numpy as np
import pytest

from oracle import controller as oc

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    rows, params = [], None
    with open(os.path.join(HERE, "golden", "controller_worked.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            v = line.split()
            if params is None:
                params = (float(v[0]), float(v[1]), float(v[2]), float(v[3]), int(v[4]))
            else:
                rows.append((int(v[0]), float(v[1]), float(v[2]), int(v[3]), int(v[4]), int(v[5]), float(v[6]), float(v[7])))
    return params, rows


def test_oracle_hand_worked_example():
    (alpha, beta, tau_g, tau_c, K), rows = _golden()
    got = oc.run(alpha, beta, tau_g, tau_c, K, [r[1] for r in rows], [r[2] for r in rows])
    for (r, _, _, b, s, h, gb, cb), (gb_, s_, h_, gbar, cbar) in zip(rows, got):
        assert gb_ == b, r
        assert (s_ if s_ is not None else -1) == s, r
        assert h_ == h, r
        assert gbar == gb and cbar == cb, r   # dyadic: exact


def test_oracle_ema_closed_form_and_bounds():
    rng = np.random.default_rng(5)
    for alpha in (0.1, 0.37, 0.9):
        g = rng.uniform(0.5, 3.0, size=60)
        out = oc.run(alpha, alpha, 1.6, 0.5, 6, g, g)
        for r in (0, 1, 7, 59):
            w = alpha * (1 - alpha) ** (r - np.arange(1, r + 1))
            closed = (1 - alpha) ** r * g[0] + float(np.dot(w, g[1:r + 1]))
            assert abs(out[r][3] - closed) <= 1e-12 * closed
            assert g[:r + 1].min() - 1e-15 <= out[r][3] <= g[:r + 1].max() + 1e-15
    # a constant sequence is a fixed point, whatever the factor
    assert all(o[3] == 2.5 for o in oc.run(0.3, 0.3, 1.6, 0.5, 6, [2.5] * 20, [2.5] * 20))


def test_oracle_restart_from_zero_average():
    out = oc.run(0.25, 0.25, 1.6, 0.5, 3, [0.0, 0.0, 5.0, 1.0], [0.0, 7.0, 0.0, 0.0])
    assert [o[3] for o in out] == [0.0, 0.0, 5.0, 0.25 * 1.0 + 0.75 * 5.0]
    assert [o[4] for o in out] == [0.0, 7.0, 5.25, 3.9375]
    # while the average is 0 nothing is skipped and nothing is heavy
    assert out[0][1] == 1 and all(o[2] == 0 for o in out[:2])


def test_oracle_decision_special_cases():
    n, K = 40, 4
    const = [3.0] * n
    out = oc.run(0.1, 0.1, 1.6, 0.5, K, const, const)
    assert out[0][:3] == (1, 1, 0)                                    # r = 0: refresh, not heavy
    assert [o[0] for o in out] == [1 if r % K == 0 else 0 for r in range(n)]
    assert all(o[1] is None for r, o in enumerate(out) if r % K)
    assert all(o[1] == 0 for r, o in enumerate(out) if r % K == 0 and r > 0)   # stable norm: skipped (tau_g > 1)
    assert all(o[2] == 1 for o in out[1:])                            # tau_c = 0.5 < 1: a steady time is "heavy"
    assert all(o[2] == 0 for o in oc.run(0.1, 0.1, 1.6, 1.0, K, const, const))  # strict inequality at tau_c = 1
    assert all(o[1] == 1 for o in oc.run(0.1, 0.1, 1.0, 0.5, K, const, const) if o[1] is not None)  # strict at tau_g = 1
    # a spike in the gradient norm forces the next boundary's refresh; a spike in time makes the next batch heavy
    g = [1.0] * 8 + [50.0] + [1.0] * 7
    o2 = oc.run(0.1, 0.1, 1.6, 2.0, 1, g, g)
    assert [o[1] for o in o2[1:]] == [0] * 8 + [1] + [0] * 6
    assert [o[2] for o in o2] == [0] * 9 + [1] + [0] * 6


def test_oracle_decisions_by_brute_force():
    """Recompute every decision from the closed-form averages of the prefix (no running state)."""
    rng = np.random.default_rng(11)
    alpha, beta, tau_g, tau_c, K = 0.2, 0.35, 1.3, 1.1, 5
    g = rng.lognormal(0.0, 0.6, size=200)
    c = rng.lognormal(0.0, 0.4, size=200)
    out = oc.run(alpha, beta, tau_g, tau_c, K, g, c)

    def avg(x, f, r):  # average after batch r
        w = f * (1 - f) ** (r - np.arange(1, r + 1))
        return (1 - f) ** r * x[0] + float(np.dot(w, x[1:r + 1]))

    margin = 1e-9
    for r in range(1, 200):
        gb, cb = avg(g, alpha, r - 1), avg(c, beta, r - 1)
        if abs(c[r - 1] - tau_c * cb) > margin:
            assert out[r][2] == int(c[r - 1] > tau_c * cb), r
        if r % K == 0 and abs(g[r - 1] - tau_g * gb) > margin:
            assert out[r][1] == int(not g[r - 1] < tau_g * gb), r


# ---- the library's controller through the C ABI (host code: runs without a GPU) -----------------------
@pytest.fixture(scope="module")
def B():
    from paper_2608_16305_b200 import binding
    binding.load_library()
    return binding


def test_library_controller_matches_oracle(B):
    rng = np.random.default_rng(3)
    for alpha, beta, tau_g, tau_c, K in [(0.1, 0.1, 1.6, 0.5, 6), (0.5, 0.25, 1.2, 1.3, 1), (0.9, 0.05, 1.01, 1.0, 7)]:
        g = rng.lognormal(0.0, 0.8, size=500)
        c = rng.lognormal(0.0, 0.5, size=500)
        g[rng.integers(0, 500, 20)] = 0.0          # restarts
        c[:3] = 0.0
        ctl = B.Controller(alpha, beta, tau_g, tau_c, K)
        ref = oc.ControllerOracle(alpha, beta, tau_g, tau_c, K)
        for r in range(500):
            got = ctl.begin_batch(r)
            b, s, h = ref.begin_batch(r)
            assert got == (b, -1 if s is None else s, h), r
            ctl.end_batch(float(g[r]), float(c[r]))
            ref.end_batch(float(g[r]), float(c[r]))
            assert ctl.state() == (ref.g_bar, ref.g_last, ref.c_bar, ref.c_prev), r   # same fp64 operations: exact


def test_library_controller_hand_worked_and_errors(B):
    (alpha, beta, tau_g, tau_c, K), rows = _golden()
    ctl = B.Controller(alpha, beta, tau_g, tau_c, K)
    for r, g, c, b, s, h, gb, cb in rows:
        assert ctl.begin_batch(r) == (b, s, h)
        ctl.end_batch(g, c)
        st = ctl.state()
        assert st[0] == gb and st[2] == cb
    for bad in [(0.0, 0.1, 1.6, 0.5, 6), (0.1, 1.5, 1.6, 0.5, 6), (0.1, 0.1, -1.0, 0.5, 6), (0.1, 0.1, 1.6, 0.5, 0),
                (float("nan"), 0.1, 1.6, 0.5, 6)]:
        with pytest.raises(B.TgnnError):
            B.Controller(*bad)
    with pytest.raises(B.TgnnError):
        ctl.begin_batch(-1)
    with pytest.raises(B.TgnnError):
        ctl.end_batch(float("nan"), 1.0)
    with pytest.raises(B.TgnnError):
        ctl.end_batch(1.0, -2.0)
