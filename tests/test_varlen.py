"""One prefix length per example (mate_plan_varlen): the paper's inputs pair a question or passage of
varying length with a table (Section 3 defines the set Q per example).  The examples of a batch are
independent, so the expected values are the oracle's results example by example, each with its own |Q|."""
import numpy as np
import pytest

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def batch(N=700, H=4, d=64, dtype="bf16", seed=3):
    """Four examples with different prefix lengths, table shapes and amounts of tail padding."""
    rng = np.random.default_rng(seed)
    prefix = [0, 37, 130, 300]
    shapes = [(9, 6), (20, 3), (5, 11), (12, 4)]
    rows, cols = [], []
    for P, (nr, nc) in zip(prefix, shapes):
        cells = [(r, c, int(rng.integers(1, 7))) for r in range(1, nr + 1) for c in range(1, nc + 1)]
        while P + sum(c[2] for c in cells) > N:
            cells.pop()
        r_, c_ = tables.custom_structure(P, cells, N)
        rows.append(r_)
        cols.append(c_)
    rows, cols = np.concatenate(rows), np.concatenate(cols)
    cfg = tables.TableConfig("varlen", len(prefix), H, H // 2, d, N, 0, 0, 0, "uniform", 1, 1, dtype, 0.5)
    vals = tables.make_values(cfg, N, seed + 1)
    return cfg, rows, cols, prefix, vals


def make_plan(rows, cols, prefix, hv, radius=0):
    import torch
    import paper_2109_04312_b200 as m
    return m, m.mate_plan_varlen(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), prefix, hv, radius)


@pytest.mark.parametrize("radius", [0, 9])
def test_varlen_plan_is_the_oracles_plan_example_by_example(radius):
    cfg, rows, cols, prefix, _ = batch()
    hv = tables.head_view(cfg)
    m, plan = make_plan(rows, cols, prefix, hv, radius)
    pairs = plan.useful_pairs()
    for view, ids in ((0, rows), (1, cols)):
        max_id = max(int(ids.max()), 0)
        perm, inv, seg = plan.get(view)
        for b, P in enumerate(prefix):
            operm, oinv, oseg = oracle.plan(rows[b:b + 1], cols[b:b + 1], P, view, max_id)
            assert np.array_equal(perm[b:b + 1], operm) and np.array_equal(inv[b:b + 1], oinv)
            assert np.array_equal(seg[b:b + 1], oseg)
    for b, P in enumerate(prefix):
        assert np.array_equal(pairs[b:b + 1], oracle.useful_pairs(rows[b:b + 1], cols[b:b + 1], P, hv, radius=radius))
    plan.destroy()


def test_equal_prefix_lengths_give_the_plain_plan():
    import torch
    cfg, rows, cols, info, _ = hp.make_case("bert")
    hv = tables.head_view(cfg)
    m, p1 = make_plan(rows, cols, [cfg.P] * cfg.B, hv)
    p0 = m.mate_plan(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, hv)
    for view in (0, 1):
        for a, b in zip(p0.get(view), p1.get(view)):
            assert np.array_equal(a, b)
    assert np.array_equal(p0.useful_pairs(), p1.useful_pairs())
    p0.destroy()
    p1.destroy()


def test_varlen_rejects_bad_prefix_lengths():
    import torch
    import paper_2109_04312_b200 as m
    rows = torch.tensor([[0, 0, 1, 1], [0, 1, 1, 2]], dtype=torch.int32).cuda()
    cols = torch.tensor([[0, 0, 1, 2], [0, 1, 2, 1]], dtype=torch.int32).cuda()

    def status(prefix):
        try:
            m.mate_plan_varlen(rows, cols, prefix, [0, 1]).destroy()
        except m.MateError as e:
            return e.status
        return 0

    assert status([2, 1]) == 0
    assert status([2, 5]) == -1   # longer than the sequence
    assert status([2, -1]) == -1
    assert status([2, 2]) == -1   # a non-zero id inside the second example's prefix
    assert status([3, 1]) == -1   # the same for the first example


@pytest.mark.parametrize("radius", [0, 9])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_varlen_forward_backward_parity(impl_idx, radius):
    import torch
    cfg, rows, cols, prefix, vals = batch()
    hv = tables.head_view(cfg)
    m, plan = make_plan(rows, cols, prefix, hv, radius)
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    scale = 1.0 / np.sqrt(cfg.d)
    atol, rtol = hp.tol(cfg.dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    gO, gL = hp.to_np(O), LSE.cpu().numpy().astype(np.float64)
    grads = [hp.to_np(g) for g in (dQ, dK, dV)]
    for b, P in enumerate(prefix):
        sl = slice(b, b + 1)
        ex = {n: vals[n][sl] for n in vals}
        oO, oL = oracle.fwd(ex["Q"], ex["K"], ex["V"], rows[sl], cols[sl], P, hv, scale, radius=radius)
        og = oracle.bwd(ex["Q"], ex["K"], ex["V"], ex["dO"], rows[sl], cols[sl], P, hv, scale, radius=radius)
        valid = np.broadcast_to((rows[sl] >= 0)[:, None, :], oL.shape)
        hp.assert_close(gO[sl], oO, atol, rtol, "O of example %d" % b)
        hp.assert_close(gL[sl][valid], oL[valid], atol, rtol, "LSE of example %d" % b)
        assert np.all(gO[sl][~valid] == 0)
        for nm, g, o in zip(("dQ", "dK", "dV"), grads, og):
            hp.assert_close(g[sl], o, atol, rtol, "%s of example %d" % (nm, b))
    plan.destroy()


@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_varlen_degenerate_examples(impl_idx):
    """A batch whose examples are: only padding, only a prefix that fills the sequence, no prefix at
    all, and a prefix followed by padding only."""
    import torch
    N, H, d = 300, 2, 64
    r0 = np.full((1, N), -1, np.int32)
    r1 = np.zeros((1, N), np.int32)
    r2, c2 = tables.custom_structure(0, [(r, c, 2) for r in range(1, 11) for c in range(1, 8)], N)
    r3 = np.full((1, N), -1, np.int32)
    r3[0, :17] = 0
    rows = np.concatenate([r0, r1, r2, r3])
    cols = np.concatenate([r0, r1, c2, r3])
    prefix = [0, N, 0, 17]
    cfg = tables.TableConfig("degenerate", 4, H, 1, d, N, 0, 0, 0, "uniform", 1, 1, "bf16", 0.5)
    vals = tables.make_values(cfg, N, 11)
    hv = tables.head_view(cfg)
    m, plan = make_plan(rows, cols, prefix, hv)
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    scale = 0.125
    atol, rtol = hp.tol("bf16")
    Q, K, V, dO = (hp.to_dev(vals[n], "bf16") for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    gO, grads = hp.to_np(O), [hp.to_np(g) for g in (dQ, dK, dV)]
    for b, P in enumerate(prefix):
        sl = slice(b, b + 1)
        ex = {n: vals[n][sl] for n in vals}
        oO, _ = oracle.fwd(ex["Q"], ex["K"], ex["V"], rows[sl], cols[sl], P, hv, scale)
        og = oracle.bwd(ex["Q"], ex["K"], ex["V"], ex["dO"], rows[sl], cols[sl], P, hv, scale)
        hp.assert_close(gO[sl], oO, atol, rtol, "O of example %d" % b)
        for nm, g, o in zip(("dQ", "dK", "dV"), grads, og):
            hp.assert_close(g[sl], o, atol, rtol, "%s of example %d" % (nm, b))
    assert np.all(gO[0] == 0) and all(np.all(g[0] == 0) for g in grads)  # the all-padding example
    plan.destroy()

