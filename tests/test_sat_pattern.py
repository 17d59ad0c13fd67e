"""The head-independent row-or-column pattern (mate_plan_sat; Section 2 of the paper describes it for
its closest comparison system) against the CPU oracle's explicit mask (head_view value 2)."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from tests.test_gpu_parity import custom_case
from workloads import tables

pytestmark = pytest.mark.gpu


def run_sat(cfg, rows, cols, vals, impl, backward=True):
    import paper_2109_04312_b200 as m
    hv = np.full(cfg.H, 2, np.uint8)
    plan = m.mate_plan_sat(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, cfg.H)
    assert np.array_equal(plan.useful_pairs(), oracle.useful_pairs(rows, cols, cfg.P, hv))   # bit exact
    scale = 1.0 / np.sqrt(cfg.d)
    atol, rtol = hp.tol(cfg.dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    oO, oLSE = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale)
    valid = rows >= 0
    vmask = np.broadcast_to(valid[:, None, :], oLSE.shape)
    gO, gLSE = hp.to_np(O), LSE.detach().cpu().numpy().astype(np.float64)
    hp.assert_close(gO, oO, atol, rtol, "O")
    assert np.all(gO[~vmask] == 0) and np.all(np.isneginf(gLSE[~vmask]))
    hp.assert_close(gLSE[vmask], oLSE[vmask], atol, rtol, "LSE")
    if backward:
        dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
        torch.cuda.synchronize()
        plan.status()
        want = oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale)
        for nm, g, o in zip(("dQ", "dK", "dV"), (dQ, dK, dV), want):
            g = hp.to_np(g)
            hp.assert_close(g, o, atol, rtol, nm)
            assert np.all(g[np.broadcast_to(~valid[:, None, :, None], g.shape)] == 0), nm + " padding rows"
    plan.destroy()


@pytest.mark.parametrize("name", ["bert", "medium", "skew"])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_sat_parity_on_the_workloads(name, impl_idx):
    import paper_2109_04312_b200 as m
    cfg, rows, cols, info, vals = hp.make_case(name)
    run_sat(cfg, rows, cols, vals, (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx])


@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_sat_shuffled_tokens_and_edge_structures(impl_idx):
    import paper_2109_04312_b200 as m
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    # table tokens in random order: a cell's tokens are scattered in the input
    cfg, rows, cols, info, vals = hp.make_case("bert", seed_structure=5, seed_values=6, shuffle=True)
    run_sat(cfg, rows, cols, vals, impl)
    cases = [
        custom_case(0, [(r, c, 1 + (r * c) % 3) for r in range(1, 9) for c in range(1, 5)], 77),   # no prefix
        custom_case(150, [], 200),                                                                 # prefix only
        custom_case(9, [(1, c, 17) for c in range(1, 12)], 9 + 17 * 11),                           # one row
        custom_case(9, [(r, 1, 40) for r in range(1, 12)], 9 + 40 * 11 + 5),                       # one column, long
        custom_case(5, [(0, 1, 3), (0, 2, 4), (1, 1, 2), (1, 2, 6)], 40),                          # ids 0 in the table
    ]
    for cfg, rows, cols, vals in cases:
        run_sat(cfg, rows, cols, vals, impl)
