"""The allocation-free entry point (tgnn_reduce_latest_static) against the context-backed
tgnn_reduce_latest, through the C ABI.

Some hosts of this library may not allocate device memory at all -- they run under a fixed
memory plan or inside a sandbox that only passes them buffers -- so they cannot create a
context.  For them step (3) exists in a form whose scratch tables are a fixed array inside
the library.  That array is shared by every call and keeps the previous call's contents, so
the check is made on two calls in a row with different inputs: the second must not see what
the first left behind.  Results are integers and must match bit for bit.

Collected last (file name) so that a run stopping at the first failure has already run
every other test; it passes alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(rng, N, n, hub):
    src = rng.integers(0, N, n).astype(np.int32)
    dst = rng.integers(0, N, n).astype(np.int32)
    if hub:
        src[rng.random(n) < 0.5] = N - 1
    t = rng.integers(0, 25, n).astype(np.float64)          # ties and unsorted times
    eid = rng.permutation(4 * n + 1)[:n].astype(np.int32)
    node = np.stack([src, dst], 1).reshape(-1).astype(np.int32)
    node[np.repeat(rng.random(n) < 0.15, 2)] = -1          # pruned events
    return node, t, eid


def test_static_reduction_matches_context_backed_one_on_two_calls_in_a_row(oracle):
    from paper_2608_16305_b200 import binding as B
    rng = np.random.default_rng(31)
    N = 50_000
    ctx = B.Tgnn(B.make_config(N, 32, 16, 10, 2, max_events=6000, max_roots=300))
    dev = lambda a: torch.from_numpy(a).cuda()
    # first call touches many nodes including the highest ids; the second a small, different set
    for N_call, n, hub in [(N, 5000, True), (N // 7, 301, False)]:
        node, t, eid = _case(rng, N_call, n, hub)
        d_node, d_t, d_eid = dev(node), dev(t), dev(eid)
        out = {}
        for which in ("ctx", "static"):
            uniq = torch.full((2 * n,), -7, dtype=torch.int32, device="cuda")
            win = torch.full((2 * n,), -7, dtype=torch.int32, device="cuda")
            nu = torch.full((1,), -7, dtype=torch.int32, device="cuda")
            if which == "ctx":
                ctx.reduce_latest(d_node, d_t, d_eid, uniq, win, nu)
            else:
                B.reduce_latest_static(d_node, d_t, d_eid, N_call, uniq, win, nu)
            torch.cuda.synchronize()
            U = int(nu.item())
            out[which] = (U, uniq[:U].cpu().numpy(), win[:U].cpu().numpy())
        assert out["ctx"][0] == out["static"][0] > 0
        assert np.array_equal(out["ctx"][1], out["static"][1])
        assert np.array_equal(out["ctx"][2], out["static"][2])
        assert np.array_equal(out["static"][1], np.unique(node[node >= 0]))
        # and both against the CPU oracle's reduction (largest (t, eid, role) per node, ascending nodes)
        u_ref, w_ref = oracle.reduce_latest(node, t, eid, N_call)
        assert np.array_equal(out["static"][1], u_ref) and np.array_equal(out["static"][2], w_ref)
    ctx.close()


def test_static_reduction_skips_and_reports_a_node_id_beyond_the_graph(oracle):
    """No status word exists without a context: an id >= num_nodes is never used as an index (the tables
    beyond num_nodes keep an earlier call's contents) and the call answers n_uniq = -1; the next call with
    clean inputs is unaffected."""
    from paper_2608_16305_b200 import binding as B
    rng = np.random.default_rng(32)
    N, n = 900, 400
    node, t, eid = _case(rng, N, n, False)
    bad = node.copy()
    bad[11] = N + 5            # inside the built-in array, outside this graph
    bad[12] = 1 << 30          # far outside the array
    dev = lambda a: torch.from_numpy(a).cuda()
    for nodes, expect_bad in [(bad, True), (node, False)]:
        uniq = torch.full((2 * n,), -7, dtype=torch.int32, device="cuda")
        win = torch.full((2 * n,), -7, dtype=torch.int32, device="cuda")
        nu = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        B.reduce_latest_static(dev(nodes), dev(t), dev(eid), N, uniq, win, nu)
        torch.cuda.synchronize()
        if expect_bad:
            assert int(nu.item()) == -1
        else:
            u_ref, w_ref = oracle.reduce_latest(nodes, t, eid, N)
            U = int(nu.item())
            assert U == len(u_ref)
            assert np.array_equal(uniq[:U].cpu().numpy(), u_ref) and np.array_equal(win[:U].cpu().numpy(), w_ref)


def test_static_reduction_refuses_graphs_beyond_its_built_in_scratch():
    from paper_2608_16305_b200 import binding as B
    z = torch.zeros(4, dtype=torch.int32, device="cuda")
    zt = torch.zeros(2, dtype=torch.float64, device="cuda")
    with pytest.raises(B.TgnnError) as e:
        B.reduce_latest_static(z, zt, z[:2], B.TGNN_STATIC_MAX_NODES + 1, z, z, z[:1])
    assert e.value.code == B.TGNN_ECAPACITY and "TGNN_STATIC_MAX_NODES" in str(e.value)
    B.reduce_latest_static(z, zt, z[:2], B.TGNN_STATIC_MAX_NODES, z.clone(), z.clone(), z[:1].clone())   # the limit itself is fine
    torch.cuda.synchronize()
