"""The bucketed, approximate form of the paper's Section 3.1 / Appendix D (global part G = the prefix,
buckets of R positions in every head's own order, a token sees its bucket and the two next to it,
restricted to its own row or column).  CPU pins of the oracle's pattern and GPU parity of the plan,
the forward and the backward with such a plan."""
import numpy as np
import pytest

import oracle
from tests import helpers as hp
from tests.test_oracle_pins import brute_fwd, brute_sets, rand_qkv, small_table
from workloads import tables


def brute_bucketed_sets(row_ids, col_ids, P, view, R, G=None):
    """Token by token, from the text: order the tokens (prefix first, then by row / column number,
    ties by position, padding last); the first G positions of that order (default: the prefix) are
    global -- they see everything and everything sees them; what follows is cut into buckets of R,
    and such a token keeps of the exact set A_k the global tokens and the tokens whose bucket is its
    own or next to it."""
    ids = row_ids if view == 0 else col_ids
    N = len(ids)
    G = P if G is None else max(G, P)
    exact = brute_sets(row_ids, col_ids, P, view)
    order = sorted(range(N), key=lambda k: ((0, 0) if k < P else ((1, ids[k]) if ids[k] >= 0 else (2, 0)), k))
    pos = {k: t for t, k in enumerate(order)}
    valid = [j for j in range(N) if ids[j] >= 0]
    glob = set(j for j in valid if pos[j] < G)
    bucket = {k: (pos[k] - G) // R for k in valid if pos[k] >= G}
    sets = []
    for k in range(N):
        if ids[k] < 0:
            sets.append(set())
        elif k in glob:
            sets.append(set(valid))
        else:
            sets.append(glob | set(j for j in exact[k] if j not in glob and abs(bucket[j] - bucket[k]) <= 1))
    return sets


@pytest.mark.parametrize("seed", [0, 1])
@pytest.mark.parametrize("R,G", [(2, 5), (3, 7), (1, 4), (4, 30)])
def test_bucketed_mask_with_a_global_section_longer_than_the_prefix(seed, R, G):
    # Section 3.1: the first G tokens of a head's order attend to and from everything, G >= |Q|; with
    # G > |Q| the table tokens that come first in the head's order are global too
    rows, cols, n = small_table(seed, P=3, n_rows=3, n_cols=3, max_len=3, pad=2)
    for view in (0, 1):
        M = oracle.mask(rows[0], cols[0], 3, view, radius=R, global_len=G)
        sets = brute_bucketed_sets(list(rows[0]), list(cols[0]), 3, view, R, G)
        for k in range(n):
            assert set(np.nonzero(M[k])[0].tolist()) == sets[k], (view, k)
        assert np.array_equal(M, M.T)
        assert np.all(oracle.mask(rows[0], cols[0], 3, view, radius=R) <= M) or G > 3   # more global tokens, other buckets
    # G = |Q| is the plain bucketed pattern; G below |Q| reads as |Q|
    assert np.array_equal(oracle.mask(rows[0], cols[0], 3, 0, radius=R, global_len=3), oracle.mask(rows[0], cols[0], 3, 0, radius=R))
    assert np.array_equal(oracle.mask(rows[0], cols[0], 3, 0, radius=R, global_len=1), oracle.mask(rows[0], cols[0], 3, 0, radius=R))


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("R", [1, 2, 3, 5])
def test_bucketed_mask_equals_brute_force(seed, R):
    rows, cols, n = small_table(seed, P=3, n_rows=3, n_cols=3, max_len=3, pad=2)
    for view in (0, 1):
        M = oracle.mask(rows[0], cols[0], 3, view, radius=R)
        sets = brute_bucketed_sets(list(rows[0]), list(cols[0]), 3, view, R)
        for k in range(n):
            assert set(np.nonzero(M[k])[0].tolist()) == sets[k], (view, k)
        # symmetric, every valid token sees itself, never more than the exact pattern
        assert np.array_equal(M, M.T)
        exact = oracle.mask(rows[0], cols[0], 3, view)
        assert np.all(M <= exact)
        valid = rows[0] >= 0
        assert np.all(np.diag(M)[valid] == 1)


def test_large_radius_is_the_exact_pattern():
    # The paper notes that with the question inside G and R long enough to hold a whole row or column
    # the bucketed implementation computes what the mask-based one does.
    rows, cols, n = small_table(5, P=4, n_rows=4, n_cols=3, max_len=3, pad=3)
    for view, ids in ((0, rows[0]), (1, cols[0])):
        table = ids[4:]
        longest = int(max(np.bincount(table[table >= 0])))
        exact = oracle.mask(rows[0], cols[0], 4, view)
        assert np.array_equal(oracle.mask(rows[0], cols[0], 4, view, radius=longest), exact)
        assert np.array_equal(oracle.mask(rows[0], cols[0], 4, view, radius=1000), exact)
        if longest > 2:  # a radius well below a third of the longest segment must lose pairs
            assert oracle.mask(rows[0], cols[0], 4, view, radius=max(1, longest // 4)).sum() < exact.sum()


def test_bucketed_forward_equals_brute_force_loops():
    rows, cols, n = small_table(3, P=2, n_rows=3, n_cols=2, max_len=3, pad=1)
    Q, K, V = rand_qkv(7, 1, 2, n, 4)
    hv = np.asarray([0, 1], np.uint8)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, 2, hv, 0.7, radius=2)
    for h, view in ((0, 0), (1, 1)):
        sets = brute_bucketed_sets(list(rows[0]), list(cols[0]), 2, view, 2)
        bO, bL = brute_fwd(Q[0, h], K[0, h], V[0, h], sets, 0.7)
        np.testing.assert_allclose(O[0, h], bO, rtol=1e-12, atol=1e-12)
        valid = rows[0] >= 0
        np.testing.assert_allclose(LSE[0, h][valid], np.asarray(bL)[valid], rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------------------------------ GPU

def _plan(cfg, rows, cols, R):
    import torch
    import paper_2109_04312_b200 as m
    return m, m.mate_plan_bucketed(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P,
                                   tables.head_view(cfg), R, max(int(rows.max()), 0), max(int(cols.max()), 0))


@pytest.mark.gpu
@pytest.mark.parametrize("name,R", [("bert", 42), ("bert", 5), ("medium", 42), ("skew", 42)])
def test_bucketed_plan_counts_the_oracles_pairs(name, R):
    cfg, rows, cols, info, _ = hp.make_case(name)
    m, plan = _plan(cfg, rows, cols, R)
    assert np.array_equal(plan.useful_pairs(), oracle.useful_pairs(rows, cols, cfg.P, tables.head_view(cfg), radius=R))
    # the order itself does not depend on the radius
    for view, ids in ((0, rows), (1, cols)):
        perm, inv, seg = plan.get(view)
        operm, oinv, oseg = oracle.plan(rows, cols, cfg.P, view, max(int(ids.max()), 0))
        assert np.array_equal(perm, operm) and np.array_equal(inv, oinv) and np.array_equal(seg, oseg)
    plan.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name,R", [("bert", 42), ("bert", 5), ("bert", 1), ("medium", 42), ("medium", 7), ("skew", 42)])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_bucketed_forward_backward_parity(name, R, impl_idx):
    import torch
    cfg, rows, cols, info, vals = hp.make_case(name)
    m, plan = _plan(cfg, rows, cols, R)
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    hv = tables.head_view(cfg)
    scale = 1.0 / np.sqrt(cfg.d)
    atol, rtol = hp.tol(cfg.dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    oO, oLSE = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale, radius=R)
    odQ, odK, odV = oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale, radius=R)
    valid = np.broadcast_to((rows >= 0)[:, None, :], oLSE.shape)
    hp.assert_close(hp.to_np(O), oO, atol, rtol, "O")
    hp.assert_close(LSE.cpu().numpy().astype(np.float64)[valid], oLSE[valid], atol, rtol, "LSE")
    for nm, g, o in (("dQ", dQ, odQ), ("dK", dK, odK), ("dV", dV, odV)):
        hp.assert_close(hp.to_np(g), o, atol, rtol, nm)
    plan.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name,G,R", [("bert", 116, 42), ("bert", 70, 5), ("bert", 512, 42), ("medium", 300, 42),
                                      ("skew", 500, 42)])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_global_section_longer_than_the_prefix(name, G, R, impl_idx):
    # Section 3.1 / Appendix A.2: G = 116, R = 42 with a shorter question: the table tokens at the first
    # G - |Q| positions of every head's own order are global
    import torch
    import paper_2109_04312_b200 as m
    cfg, rows, cols, info, vals = hp.make_case(name)
    assert cfg.P < G
    hv = tables.head_view(cfg)
    plan = m.mate_plan_bucketed_global(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, G, hv, R)
    assert np.array_equal(plan.useful_pairs(),
                          oracle.useful_pairs(rows, cols, cfg.P, hv, radius=R, global_len=G))   # bit exact
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    scale = 1.0 / np.sqrt(cfg.d)
    atol, rtol = hp.tol(cfg.dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    oO, oLSE = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale, radius=R, global_len=G)
    want = oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale, radius=R, global_len=G)
    valid = np.broadcast_to((rows >= 0)[:, None, :], oLSE.shape)
    hp.assert_close(hp.to_np(O), oO, atol, rtol, "O")
    hp.assert_close(LSE.cpu().numpy().astype(np.float64)[valid], oLSE[valid], atol, rtol, "LSE")
    for nm, g, o in zip(("dQ", "dK", "dV"), (dQ, dK, dV), want):
        hp.assert_close(hp.to_np(g), o, atol, rtol, nm)
    plan.destroy()


@pytest.mark.gpu
def test_global_section_arguments():
    import torch
    import paper_2109_04312_b200 as m
    cfg, rows, cols, info, _ = hp.make_case("bert")
    r, c = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    hv = tables.head_view(cfg)
    for G, R in ((cfg.P - 1, 42), (cfg.N + 1, 42), (116, 0)):      # below the prefix, beyond N, no radius
        with pytest.raises(m.MateError) as e:
            m.mate_plan_bucketed_global(r, c, cfg.P, G, hv, R)
        assert e.value.status == -1
    # G = |Q| is the plain bucketed plan
    p0 = m.mate_plan_bucketed(r, c, cfg.P, hv, 42)
    p1 = m.mate_plan_bucketed_global(r, c, cfg.P, cfg.P, hv, 42)
    assert np.array_equal(p0.useful_pairs(), p1.useful_pairs())
    p0.destroy()
    p1.destroy()
